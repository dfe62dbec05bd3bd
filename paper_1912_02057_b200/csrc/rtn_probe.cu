// Peak probes: the two non-memory ceilings the contraction kernels are measured against, as committed code.
//   probe_i8_kernel    one CTA per SM issues tcgen05.mma kind::i8 (M = 128, N = 256 or a given column count,
//                      K = 32) back to back on operands that stay in shared memory: int8 tensor-pipe rate, nothing
//                      else in the way.
//   probe_popc_kernel  every thread runs the inner product of Eq. 9 (AND, XOR-AND, two popcounts, two adds per
//                      32 code pairs) on registers only: issue rate of the bit-plane kernels' instruction mix.
// Both write the SM-clock cycles each CTA spent in its loop; the caller times the launch with events as well.
#include "rtn_internal.cuh"
#include "rtn_tcgen05.cuh"

namespace rtn {

namespace {

constexpr int kProbeM = 128, kProbeN = 256, kProbeK = 32;
constexpr int kProbeThreads = 128;
constexpr int kPopcThreads = 1024;
constexpr int kPopcTile = 8;            // 8 x 8 word pairs per round and thread

__device__ __forceinline__ uint32_t mix(uint32_t v)
{
    v ^= v >> 16; v *= 0x7feb352du; v ^= v >> 15; v *= 0x846ca68bu; v ^= v >> 16;
    return v;
}

__global__ void __launch_bounds__(kProbeThreads, 1)
probe_i8_kernel(uint32_t n_cols, uint32_t n_mma, long long* cycles, unsigned* status)
{
    // [K chunk of 16 B][row][16 B]: the K-major no-swizzle operand layout of the contraction kernels
    __shared__ __align__(128) uint8_t sA[2 * kProbeM * 16];
    __shared__ __align__(128) uint8_t sB[2 * kProbeN * 16];
    __shared__ uint64_t done;
    __shared__ uint32_t slot;
    const int warp = threadIdx.x >> 5;
    // ternary codes as int8, pseudo-random (all-zero operands would draw less power than real ones)
    for (int i = threadIdx.x; i < (int)sizeof(sA) / 4; i += kProbeThreads) {
        const uint32_t r = mix(i * 2654435761u + blockIdx.x);
        reinterpret_cast<uint32_t*>(sA)[i] = __byte_perm(0x0100FF00u, 0u, r & 0x3333u);
    }
    for (int i = threadIdx.x; i < (int)sizeof(sB) / 4; i += kProbeThreads) {
        const uint32_t r = mix(i * 2246822519u + 77u * blockIdx.x);
        reinterpret_cast<uint32_t*>(sB)[i] = __byte_perm(0x0100FF00u, 0u, r & 0x3333u);
    }
    if (warp == 0) tc::tmem_alloc(&slot, kProbeN);            // (the largest column count)
    if (threadIdx.x == 32) {
        tc::mbar_init(&done, 1);
        tc::mbar_init_fence();
    }
    tc::fence_smem_to_async_proxy();
    tc::tc_fence_before_sync();
    __syncthreads();
    tc::tc_fence_after_sync();
    const uint32_t tmem = slot;
    if (threadIdx.x == 0) {
        const uint64_t a_desc = tc::smem_desc_kmajor(tc::smem_addr(sA), kProbeM * 16, 128);
        const uint64_t b_desc = tc::smem_desc_kmajor(tc::smem_addr(sB), n_cols * 16, 128);
        const uint32_t idesc = tc::idesc_i8(kProbeM, n_cols);
        const long long t0 = clock64();
        tc::mma_i8_ss(tmem, a_desc, b_desc, idesc, false);
        for (uint32_t i = 1; i < n_mma; ++i) tc::mma_i8_ss_acc(tmem, a_desc, b_desc, idesc);
        tc::mma_commit(&done);
        tc::mbar_wait(&done, 0, status);
        cycles[blockIdx.x] = clock64() - t0;
    }
    tc::tc_fence_before_sync();
    __syncthreads();
    if (warp == 0) tc::tmem_dealloc(tmem, kProbeN);
}

__global__ void __launch_bounds__(kPopcThreads, 1)
probe_popc_kernel(uint32_t rounds, long long* cycles, int* sink)
{
    uint32_t xn[kPopcTile], xs[kPopcTile], wn[kPopcTile], ws[kPopcTile];
    const uint32_t id = blockIdx.x * kPopcThreads + threadIdx.x;
    #pragma unroll
    for (int i = 0; i < kPopcTile; ++i) {
        xn[i] = mix(id * 4u * kPopcTile + i);
        xs[i] = mix(id * 4u * kPopcTile + kPopcTile + i);
        wn[i] = mix(id * 4u * kPopcTile + 2 * kPopcTile + i);
        ws[i] = mix(id * 4u * kPopcTile + 3 * kPopcTile + i);
    }
    int both = 0, differ = 0;
    __syncthreads();
    const long long t0 = clock64();
    for (uint32_t r = 0; r < rounds; ++r) {
        #pragma unroll
        for (int i = 0; i < kPopcTile; ++i) {
            #pragma unroll
            for (int j = 0; j < kPopcTile; ++j) {
                const uint32_t c = wn[i] & xn[j];               // both codes non-zero
                both += __popc(c);
                differ += __popc((ws[i] ^ xs[j]) & c);          // ... and of opposite sign
            }
        }
        #pragma unroll
        for (int i = 0; i < kPopcTile; ++i) { wn[i] += 0x9E3779B9u; ws[i] += 0x7F4A7C15u; }     // new operand words
    }
    __syncthreads();
    if (threadIdx.x == 0) cycles[blockIdx.x] = clock64() - t0;
    if (both - 2 * differ == 0x7FFFFFFF) *sink = 1;            // keeps the loop alive; never true
}

// Plain copy, 16 bytes per thread and trip: what a kernel that only moves a layer's input and output can reach at
// that size (launch ramp and tail included), the yardstick for the HBM-bound conv shapes.
__global__ void __launch_bounds__(1024, 2)
probe_copy_kernel(const uint4* __restrict__ src, uint4* __restrict__ dst, size_t n16)
{
    const size_t stride = (size_t)gridDim.x * blockDim.x;
    for (size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < n16; i += stride) dst[i] = src[i];
}

}  // namespace

}  // namespace rtn

extern "C" {

int64_t rtn_probe_ctas(void) { return rtn::device_sm_count(); }

int64_t rtn_probe_i8_ops_per_mma(void) { return 2ll * rtn::kProbeM * rtn::kProbeN * rtn::kProbeK; }

int64_t rtn_probe_popc_ops_per_round(void)
{
    return 2ll * 32 * rtn::kPopcTile * rtn::kPopcTile * rtn::kPopcThreads;
}

rtn_status rtn_probe_peak_i8(int64_t n_mma, int64_t* cycles, void* stream)
{
    return rtn_probe_i8_rate(rtn::kProbeN, n_mma, cycles, stream);
}

rtn_status rtn_probe_i8_rate(int64_t n_cols, int64_t n_mma, int64_t* cycles, void* stream)
{
    if (cycles == nullptr) return RTN_ERR_NULL;
    if (n_mma < 1 || n_mma > (1 << 22)) return RTN_ERR_SHAPE;
    if (n_cols < 16 || n_cols > rtn::kProbeN || n_cols % 16 != 0) return RTN_ERR_SHAPE;
    if (reinterpret_cast<uintptr_t>(cycles) % 8 != 0) return RTN_ERR_ALIGN;
    unsigned* word = rtn::device_status_word();      // receives a time-out of the final (bounded) wait
    if (word == nullptr) return RTN_ERR_CUDA;
    rtn::probe_i8_kernel<<<(unsigned)rtn::device_sm_count(), rtn::kProbeThreads, 0, static_cast<cudaStream_t>(stream)>>>(
        (uint32_t)n_cols, (uint32_t)n_mma, reinterpret_cast<long long*>(cycles), word);
    return cudaGetLastError() == cudaSuccess ? RTN_OK : RTN_ERR_CUDA;
}

rtn_status rtn_probe_copy(const void* src, void* dst, int64_t bytes, void* stream)
{
    if (src == nullptr || dst == nullptr) return RTN_ERR_NULL;
    if (bytes <= 0 || bytes % 16 != 0) return RTN_ERR_SHAPE;
    if (reinterpret_cast<uintptr_t>(src) % 16 != 0 || reinterpret_cast<uintptr_t>(dst) % 16 != 0) return RTN_ERR_ALIGN;
    rtn::probe_copy_kernel<<<(unsigned)(2 * rtn::device_sm_count()), 1024, 0, static_cast<cudaStream_t>(stream)>>>(
        static_cast<const uint4*>(src), static_cast<uint4*>(dst), (size_t)bytes / 16);
    return cudaGetLastError() == cudaSuccess ? RTN_OK : RTN_ERR_CUDA;
}

rtn_status rtn_probe_peak_popc(int64_t rounds, int64_t* cycles, int32_t* sink, void* stream)
{
    if (cycles == nullptr || sink == nullptr) return RTN_ERR_NULL;
    if (rounds < 1 || rounds > (1 << 24)) return RTN_ERR_SHAPE;
    if (reinterpret_cast<uintptr_t>(cycles) % 8 != 0 || reinterpret_cast<uintptr_t>(sink) % 4 != 0) return RTN_ERR_ALIGN;
    rtn::probe_popc_kernel<<<(unsigned)rtn::device_sm_count(), rtn::kPopcThreads, 0, static_cast<cudaStream_t>(stream)>>>(
        (uint32_t)rounds, reinterpret_cast<long long*>(cycles), sink);
    return cudaGetLastError() == cudaSuccess ? RTN_OK : RTN_ERR_CUDA;
}

}  // extern "C"
