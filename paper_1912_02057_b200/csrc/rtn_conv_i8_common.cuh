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
        if ((i & 15u) == 15u && *dead) return false;        // a look at the flag now and then keeps the poll short
    }
    *dead = 1;
    atomicOr(status, kStatusWaitTimeout);
    return false;
}

// Filters of rows n_base .. n_base + ld - 1: bit planes (Table 1) in global memory -> int8 in shared memory,
// sW[(tap * Cp/16 + 16-channel chunk) * ld + row][16 B] in tc::unpack32's byte order.  Row `ones_row` (relative to
// n_base; -1 for none) becomes all +1 (it makes the tensor core produce the activation code sum), rows at or past
// N become 0.  Item = (row, packed block of four 32-channel words of each plane): two 16-byte loads instead of
// eight 4-byte ones.  Consecutive lanes take consecutive rows, so the shared-memory stores are conflict-free; the
// loads of a warp then fall in 32 different lines, which the load unit takes one line at a time, and that, with
// every CTA of the grid asking for the same few lines, is what this step's time is made of: a quarter of the load
// instructions is a quarter of the time.  kBatch items' loads are in flight per thread.
template <int kBatch>
__device__ __forceinline__ void expand_filter_rows(const uint8_t* w_packed, uint4* sW, int T, int cwords, int ld,
                                                   FastDiv div_ld, FastDiv div_cw, int n_base, int N, int ones_row,
                                                   int tid, int nthreads)
{
    const int nwords = T * cwords;                     // 32-channel words per plane and row
    const int nblocks = (nwords + 3) / 4;              // packed blocks per row
    const int nchunk = 2 * cwords;
    const uint4* Wp = reinterpret_cast<const uint4*>(w_packed);
    const int items = nblocks * ld;
    for (int base = tid; base < items; base += kBatch * nthreads) {
        uint4 nz[kBatch], sg[kBatch];
        #pragma unroll
        for (int u = 0; u < kBatch; ++u) {
            const int i = base + u * nthreads;
            nz[u] = make_uint4(0u, 0u, 0u, 0u); sg[u] = nz[u];
            if (i < items) {
                const int wb = (int)fdiv((uint32_t)i, div_ld), r = i - wb * ld;
                const int n = n_base + r;
                if (r == ones_row) {
                    nz[u] = make_uint4(~0u, ~0u, ~0u, ~0u); sg[u] = nz[u];
                } else if (n < N) {
                    const uint4* blk = Wp + ((int64_t)n * nblocks + wb) * 2;
                    nz[u] = __ldg(blk);
                    sg[u] = __ldg(blk + 1);
                }
            }
        }
        #pragma unroll
        for (int u = 0; u < kBatch; ++u) {
            const int i = base + u * nthreads;
            if (i < items) {
                const int wb = (int)fdiv((uint32_t)i, div_ld), r = i - wb * ld;
                const uint32_t nzw[4] = {nz[u].x, nz[u].y, nz[u].z, nz[u].w};
                const uint32_t sgw[4] = {sg[u].x, sg[u].y, sg[u].z, sg[u].w};
                #pragma unroll
                for (int j = 0; j < 4; ++j) {
                    const int wd = 4 * wb + j;
                    if (wd < nwords) {
                        const int t = (int)fdiv((uint32_t)wd, div_cw), cw = wd - t * cwords;
                        uint32_t o[8];
                        tc::unpack32(nzw[j], sgw[j], o);
                        uint4* dst = sW + ((int64_t)(t * nchunk + 2 * cw) * ld + r);
                        dst[0] = make_uint4(o[0], o[1], o[2], o[3]);
                        dst[ld] = make_uint4(o[4], o[5], o[6], o[7]);
                    }
                }
            }
        }
    }
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

// Epilogue constant c3 of output channel n at a border pixel under value-zero padding: S_w and K
// run over the taps inside the image only.  Kept out of line: borders are rare, the code is long.  The
// layer's geometry comes by value: a reference to the kernel's parameter struct would make the compiler
// keep a copy of it in local memory.
struct BorderGeom {
    const int32_t* w_sum;
    const float* w_scale;
    const float* w_offset;
    int n_wparam, N, C, H, W, kw, stride, pad, T;
    float a_offset;
};
__device__ __forceinline__ BorderGeom border_geom(const ConvArgs& a, int T)
{
    BorderGeom g;
    g.w_sum = a.w_sum; g.w_scale = a.ep.w_scale; g.w_offset = a.ep.w_offset; g.n_wparam = (int)a.ep.n_wparam;
    g.N = a.N; g.C = a.C; g.H = a.H; g.W = a.W; g.kw = a.kw; g.stride = a.stride; g.pad = a.pad; g.T = T;
    g.a_offset = a.ep.a_offset_val;
    return g;
}
__device__ __noinline__ inline float border_c3_by_value(BorderGeom g, int ho, int wo, int n_inside, int n)
{
    int s_w = 0;
    for (int t = 0; t < g.T; ++t) {
        const int h = ho * g.stride - g.pad + t / g.kw, v = wo * g.stride - g.pad + t % g.kw;
        if (h >= 0 && h < g.H && v >= 0 && v < g.W) s_w += g.w_sum[(1 + t) * g.N + n];
    }
    const double ws = g.w_scale[g.n_wparam == 1 ? 0 : n];
    const double wo_ = g.w_offset[g.n_wparam == 1 ? 0 : n];
    return (float)((double)g.a_offset * (ws * (double)s_w + (double)g.C * n_inside * wo_));
}
__device__ __forceinline__ float border_c3(const ConvArgs& a, int T, int ho, int wo, int n_inside, int n)
{
    return border_c3_by_value(border_geom(a, T), ho, wo, n_inside, n);
}
// Element j (runtime index) of a register array, without sending the array to local memory.
__device__ __forceinline__ uint32_t pick16(const uint32_t (&v)[16], int j)
{
    uint32_t r = v[0];
    #pragma unroll
    for (int k = 1; k < 16; ++k) r = (j == k) ? v[k] : r;
    return r;
}
__device__ __forceinline__ void put16(float (&y)[16], int j, float val)
{
    #pragma unroll
    for (int k = 0; k < 16; ++k) y[k] = (j == k) ? val : y[k];
}

// The hand-over epilogue (NextLayerArgs) for one pixel and one block of 16 output channels n0..n0+15:
//   y = phi(c1*S_xw + c2*S_x + c3) + skip;  out <- y;  nzb, sgb <- Eq. 3 codes of y (16 bits per plane,
//   computed when want_codes; the caller assembles them into words of the packed pixel row).
// v: the block's accumulators; sC: {c1, c2, c3, 0} and sT: {t_lo, t_hi} of the next layer, both for
// column n0 (columns past N hold zeros and (-inf, +inf): they code to 0).  o0: offset of (b, n0, ho, wo)
// in the NCHW tensors.  Straight-line over the 16 columns: every load of a step is issued before its
// first use (the skip values of 16 channels are 16 independent trips to memory).
__device__ __forceinline__ void next_layer_block16(const ConvArgs& a, const NextLayerArgs& f, const uint32_t (&v)[16],
                                                   const float4* sC, const float2* sT, float fsx, bool border,
                                                   int T, int ho, int wo, int n_inside, int n0, int64_t o0,
                                                   int64_t ostride, bool want_codes, uint32_t& nzb, uint32_t& sgb)
{
    const bool full = n0 + 16 <= a.N;
    float y[16];
    #pragma unroll
    for (int j = 0; j < 16; ++j) {
        const float4 c = sC[j];
        y[j] = fmaf(c.x, (float)(int)v[j], fmaf(c.y, fsx, c.z));
    }
    if (border) {
        // value-zero padding at an image border: S_w and K over inside taps only
        #pragma unroll 1
        for (int j = 0; j < 16; ++j) {
            const int n = n0 + j;
            if (n >= a.N) break;
            const float4 c = sC[j];
            const float c3 = border_c3(a, T, ho, wo, n_inside, n);
            put16(y, j, fmaf(c.x, (float)(int)pick16(v, j), fmaf(c.y, fsx, c3)));
        }
    }
    if (f.relu) {
        #pragma unroll
        for (int j = 0; j < 16; ++j) y[j] = fmaxf(y[j], 0.f);          // (a NaN becomes 0 either way)
    }
    if (f.skip != nullptr) {
        float sk[16];
        #pragma unroll
        for (int j = 0; j < 16; ++j)
            sk[j] = (full || n0 + j < a.N) ? __ldg(f.skip + o0 + (int64_t)j * ostride) : 0.f;
        #pragma unroll
        for (int j = 0; j < 16; ++j) y[j] += sk[j];
    }
    if (a.out != nullptr) {
        #pragma unroll
        for (int j = 0; j < 16; ++j)
            if (full || n0 + j < a.N) a.out[o0 + (int64_t)j * ostride] = y[j];
    }
    if (a.dbg_acc != nullptr) {
        #pragma unroll
        for (int j = 0; j < 16; ++j)
            if (full || n0 + j < a.N) a.dbg_acc[o0 + (int64_t)j * ostride] = (int)v[j];
    }
    nzb = 0; sgb = 0;                          // one bit per column and plane
    if (want_codes) {
        // The bits of a plane are summed as powers of two in fp32 (exact below 2^24): a comparison that yields
        // 1.0f / 0.0f and one FMA per value and plane, against a predicate, a select and an OR each.  +1 is tested
        // first: the sign plane is "y > t_hi" alone, and a value that is both above t_hi and below t_lo (possible
        // only when t_lo > t_hi) has its non-zero bit set by either comparison.
        float above0 = 0.f, above1 = 0.f, below0 = 0.f, below1 = 0.f;
        #pragma unroll
        for (int j = 0; j < 16; j += 2) {
            const float2 t0 = sT[j], t1 = sT[j + 1];
            above0 = fmaf(y[j] > t0.y ? 1.f : 0.f, (float)(1u << j), above0);
            below0 = fmaf(y[j] < t0.x ? 1.f : 0.f, (float)(1u << j), below0);
            above1 = fmaf(y[j + 1] > t1.y ? 1.f : 0.f, (float)(2u << j), above1);
            below1 = fmaf(y[j + 1] < t1.x ? 1.f : 0.f, (float)(2u << j), below1);
        }
        sgb = (uint32_t)(above0 + above1);
        nzb = sgb | (uint32_t)(below0 + below1);
    }
}

// The hand-over step for TWO pixels of a thread and one block of 16 output channels, all of which exist (layers
// without border classes): every constant and threshold pair is fetched once and serves both pixels, and the two
// pixels' arithmetic interleaves, which is what an epilogue bound by the round trips of its loads needs.
// v0, v1: the block's accumulators of the two pixels; o0_0, o0_1: offsets of (b, n0, ho, wo) of each pixel; sk0, sk1: when
// not null, where channel n0 of each pixel's skip value sits in shared memory (channel n0 + j is j * sk_stride floats on);
// ok0, ok1: the pixel exists (nothing is read or written for one that does not).
template <bool kSk = false>
__device__ __forceinline__ void next_layer_block16_pair(const ConvArgs& a, const NextLayerArgs& f,
                                                        const uint32_t (&v0)[16], const uint32_t (&v1)[16],
                                                        const float4* sC, const float2* sT, float fsx0, float fsx1,
                                                        bool ok0, bool ok1, int64_t o0_0, int64_t o0_1, int64_t ostride,
                                                        bool want_codes, uint32_t& nzb0, uint32_t& sgb0,
                                                        uint32_t& nzb1, uint32_t& sgb1,
                                                        const float* sk0 = nullptr, const float* sk1 = nullptr,
                                                        int sk_stride = 0)
{
    nzb0 = sgb0 = nzb1 = sgb1 = 0;
    #pragma unroll
    for (int h = 0; h < 16; h += 8) {
        float y0[8], y1[8];
        #pragma unroll
        for (int j = 0; j < 8; ++j) {
            const float4 c = sC[h + j];
            y0[j] = fmaf(c.x, (float)(int)v0[h + j], fmaf(c.y, fsx0, c.z));
            y1[j] = fmaf(c.x, (float)(int)v1[h + j], fmaf(c.y, fsx1, c.z));
        }
        if (f.relu) {
            #pragma unroll
            for (int j = 0; j < 8; ++j) { y0[j] = fmaxf(y0[j], 0.f); y1[j] = fmaxf(y1[j], 0.f); }
        }
        if (f.skip != nullptr) {
            float s0[8], s1[8];
            #pragma unroll
            if constexpr (kSk) {
                // staged in shared memory by the kernel's producer warp (sk_stride floats between channels)
                #pragma unroll
                for (int j = 0; j < 8; ++j) {
                    s0[j] = ok0 ? sk0[(h + j) * sk_stride] : 0.f;
                    s1[j] = ok1 ? sk1[(h + j) * sk_stride] : 0.f;
                }
            } else {
                #pragma unroll
                for (int j = 0; j < 8; ++j) {
                    s0[j] = ok0 ? __ldg(f.skip + o0_0 + (int64_t)(h + j) * ostride) : 0.f;
                    s1[j] = ok1 ? __ldg(f.skip + o0_1 + (int64_t)(h + j) * ostride) : 0.f;
                }
            }
            #pragma unroll
            for (int j = 0; j < 8; ++j) { y0[j] += s0[j]; y1[j] += s1[j]; }
        }
        if (a.out != nullptr) {
            #pragma unroll
            for (int j = 0; j < 8; ++j) {
                if (ok0) a.out[o0_0 + (int64_t)(h + j) * ostride] = y0[j];
                if (ok1) a.out[o0_1 + (int64_t)(h + j) * ostride] = y1[j];
            }
        }
        if (a.dbg_acc != nullptr) {
            #pragma unroll
            for (int j = 0; j < 8; ++j) {
                if (ok0) a.dbg_acc[o0_0 + (int64_t)(h + j) * ostride] = (int)v0[h + j];
                if (ok1) a.dbg_acc[o0_1 + (int64_t)(h + j) * ostride] = (int)v1[h + j];
            }
        }
        if (want_codes) {
            float ab0 = 0.f, be0 = 0.f, ab1 = 0.f, be1 = 0.f;          // bits summed as powers of two (exact)
            #pragma unroll
            for (int j = 0; j < 8; ++j) {
                const float2 t = sT[h + j];
                const float bit = (float)(1u << (h + j));
                ab0 = fmaf(y0[j] > t.y ? 1.f : 0.f, bit, ab0);
                be0 = fmaf(y0[j] < t.x ? 1.f : 0.f, bit, be0);
                ab1 = fmaf(y1[j] > t.y ? 1.f : 0.f, bit, ab1);
                be1 = fmaf(y1[j] < t.x ? 1.f : 0.f, bit, be1);
            }
            const uint32_t s0 = (uint32_t)ab0, s1 = (uint32_t)ab1;
            sgb0 |= s0; nzb0 |= s0 | (uint32_t)be0;
            sgb1 |= s1; nzb1 |= s1 | (uint32_t)be1;
        }
    }
}

// Zero codes for the columns from n_begin (a multiple of 16) to the end of a packed pixel row.
__device__ __forceinline__ void zero_fill_packed_row(uint8_t* out_row, int n_begin, int packed_cols)
{
    for (int n0 = n_begin; n0 < packed_cols; n0 += 16) {
        uint8_t* dst = out_row + (n0 >> 7) * kBlockBytes + ((n0 & 127) >> 3);
        *reinterpret_cast<uint16_t*>(dst) = 0;
        *reinterpret_cast<uint16_t*>(dst + 16) = 0;
    }
}

}  // namespace conv_detail
}  // namespace rtn
