// Helpers shared by the tensor-core conv kernels.
#pragma once
#include "rtn_internal.cuh"
#include "rtn_tcgen05.cuh"

namespace rtn {
namespace conv_detail {

// channel (within a group of 16) held by byte e of a 16-byte chunk: tc::unpack32's order
// (0,4,8,12, 2,6,10,14, 1,5,9,13, 3,7,11,15)
__host__ __device__ constexpr int perm16(int e)
{
    return 4 * (e & 3) + ((e >> 2) == 0 ? 0 : (e >> 2) == 1 ? 2 : (e >> 2) == 2 ? 1 : 3);
}

// x / d for x*d < 2^32 (d >= 1): floor(x * ceil(2^32 / d) / 2^32)
struct FastDiv {
    uint32_t d, m;
};
inline FastDiv make_fastdiv(uint32_t d)
{
    FastDiv f;
    f.d = d;
    f.m = d <= 1 ? 0u : (uint32_t)(((uint64_t(1) << 32) + d - 1) / d);
    return f;
}
__device__ __forceinline__ uint32_t fdiv(uint32_t x, FastDiv f) { return f.d <= 1 ? x : __umulhi(x, f.m); }

// Bounded wait that also gives up at once when another thread of the CTA has already timed out.
__device__ __forceinline__ bool wait_or_die(uint64_t* bar, uint32_t parity, unsigned* status,
                                            volatile int* dead)
{
    if (tc::mbar_try_wait(bar, parity)) return true;
    for (uint32_t i = 0; i < tc::kWaitPolls; ++i) {
        if (tc::mbar_try_wait(bar, parity)) return true;
        if (*dead) return false;
    }
    *dead = 1;
    atomicOr(status, kStatusWaitTimeout);
    return false;
}

// Sixteen fp32 values -> sixteen int8 codes {-1,0,+1} in four words (byte e of the chunk = v[e]).
// Branch-free: p = (v > hi), n = (v < lo) as 1.0f / 0.0f, then (1.5*2^23 + p) - n is a float whose
// low mantissa byte is the two's-complement code; PRMT gathers the four low bytes of a word.  The
// two comparisons never both hold: the set-up replaces t_lo by the float just above t_hi when
// t_lo > t_hi, which keeps "+1 is tested first" (then -1 exactly when v <= t_hi).
template <bool kPerLayer>
__device__ __forceinline__ uint4 codes16(const float (&v)[16], const float* lo, const float* hi, int c0,
                                         float lo0, float hi0)
{
    uint32_t t[16];
    #pragma unroll
    for (int e = 0; e < 16; ++e) {
        const float l = kPerLayer ? lo0 : lo[c0 + perm16(e)];
        const float h = kPerLayer ? hi0 : hi[c0 + perm16(e)];
        const float pos = v[e] > h ? 1.0f : 0.0f;
        const float neg = v[e] < l ? 1.0f : 0.0f;
        t[e] = __float_as_uint((12582912.0f + pos) - neg);
    }
    uint32_t w[4];
    #pragma unroll
    for (int k = 0; k < 4; ++k)
        w[k] = __byte_perm(__byte_perm(t[4 * k], t[4 * k + 1], 0x0040),
                           __byte_perm(t[4 * k + 2], t[4 * k + 3], 0x0040), 0x5410);
    return make_uint4(w[0], w[1], w[2], w[3]);
}

}  // namespace conv_detail
}  // namespace rtn
