// Packing kernels: weight codes -> bit planes (+ code sums), and fp32 activations ->
// ternary codes (Eq. 3) -> bit planes (Table 1) with the per-row code sum S_x.
#include "rtn_internal.cuh"

namespace rtn {

// ---------------------------------------------------------------------------------------------
// Weights.  One thread builds one 32-code word pair of one filter row.
// Row order (kh, kw, c) with the channel rounded up to 32, so a word never straddles two taps.
// ---------------------------------------------------------------------------------------------
__global__ void pack_weights_kernel(const int8_t* __restrict__ w, int64_t N, int64_t C, int kh,
                                    int kw, uint8_t* __restrict__ packed, int32_t* __restrict__ w_sum,
                                    unsigned* status)
{
    const int T = kh * kw;
    const int64_t cwords = (C + 31) / 32;              // words per tap
    const int64_t words = (int64_t)T * cwords;         // words per row that hold codes
    const int64_t row_words = ((words + 3) / 4) * 4;   // words per plane per row, block padded
    const int64_t total = N * row_words;
    for (int64_t idx = blockIdx.x * (int64_t)blockDim.x + threadIdx.x; idx < total;
         idx += (int64_t)gridDim.x * blockDim.x) {
        const int64_t n = idx / row_words;
        const int64_t wd = idx % row_words;
        uint32_t nz = 0, sg = 0;
        bool bad = false;
        int t = 0;
        if (wd < words) {
            t = (int)(wd / cwords);
            const int64_t c0 = (wd % cwords) * 32;
            const int8_t* src = w + (n * C) * T + t;   // + c*T
            #pragma unroll 4
            for (int i = 0; i < 32; ++i) {
                const int64_t c = c0 + i;
                if (c < C) {
                    const int v = src[c * T];
                    bad |= (v < -1) | (v > 1);
                    nz |= (uint32_t)(v != 0) << i;
                    sg |= (uint32_t)(v > 0) << i;
                }
            }
        }
        uint8_t* row = packed + n * (row_words / 4) * kBlockBytes;
        uint32_t* blk = reinterpret_cast<uint32_t*>(row + (wd / 4) * kBlockBytes);
        blk[wd % 4] = nz;
        blk[4 + (wd % 4)] = sg;
        if (bad) atomicOr(status, kStatusBadWeightCode);
        const int s = __popc(nz & sg) - __popc(nz & ~sg);
        if (s != 0) {
            atomicAdd(&w_sum[n], s);
            atomicAdd(&w_sum[(int64_t)(1 + t) * N + n], s);
        }
    }
}

cudaError_t launch_pack_weights(const int8_t* w, int64_t N, int64_t C, int kh, int kw,
                                uint8_t* packed, int32_t* w_sum, unsigned* status, cudaStream_t s)
{
    const int T = kh * kw;
    cudaError_t e = cudaMemsetAsync(w_sum, 0, sizeof(int32_t) * (size_t)(1 + T) * (size_t)N, s);
    if (e != cudaSuccess) return e;
    const int64_t words = (int64_t)T * ((C + 31) / 32);
    const int64_t total = N * (((words + 3) / 4) * 4);
    const int threads = 256;
    int64_t blocks = (total + threads - 1) / threads;
    if (blocks > 148 * 64) blocks = 148 * 64;
    pack_weights_kernel<<<(unsigned)blocks, threads, 0, s>>>(w, N, C, kh, kw, packed, w_sum, status);
    return cudaGetLastError();
}

// ---------------------------------------------------------------------------------------------
// Activations [M][K] fp32.  One warp walks one row, one 128-code block per step: lane l reads
// a[k0 + l + 32 j], j = 0..3 (four coalesced 128-byte requests), and __ballot_sync over the
// comparison results is word j of the plane -- bit l of word j is code k0 + 32 j + l, which is
// the packed format's bit order.  Lanes 0..7 then write the block's eight words (32 bytes).
// ---------------------------------------------------------------------------------------------
template <bool kPerK>
__global__ void __launch_bounds__(256)
ternarize_pack_kernel(const float* __restrict__ a, int64_t M, int64_t K,
                      const float* __restrict__ t_lo, const float* __restrict__ t_hi,
                      uint8_t* __restrict__ packed, int32_t* __restrict__ a_sum)
{
    const int lane = threadIdx.x & 31;
    const int64_t warp = (blockIdx.x * (int64_t)blockDim.x + threadIdx.x) >> 5;
    const int64_t nwarps = ((int64_t)gridDim.x * blockDim.x) >> 5;
    const int64_t nblk = (K + kBlockCodes - 1) / kBlockCodes;
    const float lo0 = t_lo[0], hi0 = t_hi[0];

    for (int64_t m = warp; m < M; m += nwarps) {
        const float* row = a + m * K;
        uint32_t* dst = reinterpret_cast<uint32_t*>(packed + m * nblk * kBlockBytes);
        int sum = 0;
        for (int64_t b0 = 0; b0 < nblk; b0 += 2) {
            // two blocks per trip: eight independent loads in flight per lane
            float v[8];
            float lo[8], hi[8];
            #pragma unroll
            for (int j = 0; j < 8; ++j) {
                const int64_t k = b0 * kBlockCodes + j * 32 + lane;
                const bool in = k < K;
                v[j] = in ? __ldg(row + k) : 0.0f;
                if (kPerK) {
                    lo[j] = in ? __ldg(t_lo + k) : 0.0f;
                    hi[j] = in ? __ldg(t_hi + k) : 0.0f;
                } else {
                    lo[j] = lo0; hi[j] = hi0;
                }
                if (!in) { lo[j] = -1.0f; hi[j] = 1.0f; }     // padding codes to 0
            }
            uint32_t mine = 0;       // lane q < 8 keeps word q of block b0, lane 8+q of block b0+1
            #pragma unroll
            for (int j = 0; j < 8; ++j) {
                bool nz, pos;
                ternarize(v[j], lo[j], hi[j], nz, pos);
                const uint32_t wn = __ballot_sync(0xffffffffu, nz);
                const uint32_t wp = __ballot_sync(0xffffffffu, pos);
                sum += __popc(wp) - __popc(wn & ~wp);
                const int blk = j >> 2, q = j & 3;
                if (lane == blk * 8 + q) mine = wn;
                if (lane == blk * 8 + 4 + q) mine = wp;
            }
            const int64_t blk = b0 + (lane >> 3);
            if (lane < 16 && blk < nblk) dst[blk * 8 + (lane & 7)] = mine;
        }
        if (a_sum != nullptr && lane == 0) a_sum[m] = sum;
    }
}

cudaError_t launch_ternarize_pack(const float* a, int64_t M, int64_t K, const float* t_lo,
                                  const float* t_hi, int64_t n_thr, uint8_t* packed, int32_t* a_sum,
                                  cudaStream_t s)
{
    const int threads = 256;
    int64_t blocks = (M + 7) / 8;
    if (blocks > 148 * 32) blocks = 148 * 32;
    if (n_thr == 1)
        ternarize_pack_kernel<false><<<(unsigned)blocks, threads, 0, s>>>(a, M, K, t_lo, t_hi, packed, a_sum);
    else
        ternarize_pack_kernel<true><<<(unsigned)blocks, threads, 0, s>>>(a, M, K, t_lo, t_hi, packed, a_sum);
    return cudaGetLastError();
}

}  // namespace rtn
