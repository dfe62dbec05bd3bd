// The paper's comparison workload: 2-bit quaternary weights and activations (Table 1, last column: bits
// (b1, b2) stand for 2 b1 + b2), dot product in the DoReFa-Net pattern the section "Efficient
// Computation Pattern" describes: AND between each bit plane of the two inputs, popcount, power-of-two
// shifts, four partial sums:
//
//   x.w = 4 bC(X1 and W1) + 2 bC(X1 and W2) + 2 bC(X2 and W1) + bC(X2 and W2)
//
// Same packed format as the ternary operands (plane 1 = first bit, plane 2 = second bit) and the same
// tiling as the ternary bit-plane GEMM, so that the two can be timed against each other: per 32 values
// and output the ternary pattern costs 2 popcounts (Eq. 9), this one 4.
#include "rtn_internal.cuh"

namespace rtn {

// values [rows][K] in {0,1,2,3} -> packed rows.  One warp per (row, block of 128 values).
__global__ void pack_quaternary_kernel(const uint8_t* __restrict__ q, int64_t rows, int64_t K,
                                       uint8_t* __restrict__ packed, unsigned* status)
{
    const int64_t nblk = (K + kBlockCodes - 1) / kBlockCodes;
    const int64_t warp = ((int64_t)blockIdx.x * blockDim.x + threadIdx.x) >> 5;
    const int lane = threadIdx.x & 31;
    if (warp >= rows * nblk) return;
    const int64_t row = warp / nblk, blk = warp % nblk;
    uint32_t* dst = reinterpret_cast<uint32_t*>(packed + (row * nblk + blk) * kBlockBytes);
    #pragma unroll
    for (int w = 0; w < 4; ++w) {
        const int64_t k = blk * kBlockCodes + w * 32 + lane;
        const unsigned v = k < K ? q[row * K + k] : 0u;
        if (v > 3u) atomicOr(status, kStatusBadWeightCode);
        const uint32_t b1 = __ballot_sync(0xffffffffu, (v & 2u) != 0u);
        const uint32_t b2 = __ballot_sync(0xffffffffu, (v & 1u) != 0u);
        if (lane == 0) { dst[w] = b1; dst[4 + w] = b2; }
    }
}

template <int TM, int TN>
__global__ void __launch_bounds__(256)
gemm_quaternary_kernel(const uint8_t* __restrict__ a_packed, const uint8_t* __restrict__ w_packed,
                       int64_t M, int64_t N, int64_t K, int32_t* __restrict__ out)
{
    constexpr int BM = 16 * TM, BN = 16 * TN, KB = 2;      // KB packed blocks (256 values) per stage
    __shared__ uint4 sA[KB][2][BM];                        // [block][plane][row]
    __shared__ uint4 sB[KB][2][BN];

    const int tid = threadIdx.x;
    const int tx = tid & 15, ty = tid >> 4;
    const int64_t m0 = (int64_t)blockIdx.x * BM, n0 = (int64_t)blockIdx.y * BN;
    const int64_t nblk = (K + kBlockCodes - 1) / kBlockCodes;
    const uint4* __restrict__ A = reinterpret_cast<const uint4*>(a_packed);
    const uint4* __restrict__ Wp = reinterpret_cast<const uint4*>(w_packed);

    // four counters per output, as the circuit keeps four partial sums
    int c11[TM][TN], c12[TM][TN], c21[TM][TN], c22[TM][TN];
    #pragma unroll
    for (int i = 0; i < TM; ++i)
        #pragma unroll
        for (int j = 0; j < TN; ++j) { c11[i][j] = 0; c12[i][j] = 0; c21[i][j] = 0; c22[i][j] = 0; }

    for (int64_t kb0 = 0; kb0 < nblk; kb0 += KB) {
        __syncthreads();
        for (int i = tid; i < KB * 2 * (BM + BN); i += 256) {
            const int b = i / (2 * (BM + BN));
            int r = i % (2 * (BM + BN));
            const bool isA = r < 2 * BM;
            if (!isA) r -= 2 * BM;
            const int rows = isA ? BM : BN;
            const int plane = r / rows, row = r % rows;
            const int64_t grow = (isA ? m0 : n0) + row;
            const int64_t kb = kb0 + b;
            uint4 v = make_uint4(0, 0, 0, 0);
            if (kb < nblk && grow < (isA ? M : N))
                v = __ldg((isA ? A : Wp) + (grow * nblk + kb) * 2 + plane);
            if (isA) sA[b][plane][row] = v; else sB[b][plane][row] = v;
        }
        __syncthreads();
        #pragma unroll
        for (int b = 0; b < KB; ++b) {
            uint4 x1[TM], x2[TM], w1[TN], w2[TN];
            #pragma unroll
            for (int i = 0; i < TM; ++i) { x1[i] = sA[b][0][ty + 16 * i]; x2[i] = sA[b][1][ty + 16 * i]; }
            #pragma unroll
            for (int j = 0; j < TN; ++j) { w1[j] = sB[b][0][tx + 16 * j]; w2[j] = sB[b][1][tx + 16 * j]; }
            #pragma unroll
            for (int i = 0; i < TM; ++i)
                #pragma unroll
                for (int j = 0; j < TN; ++j) {
                    c11[i][j] += (__popc(x1[i].x & w1[j].x) + __popc(x1[i].y & w1[j].y)) +
                                 (__popc(x1[i].z & w1[j].z) + __popc(x1[i].w & w1[j].w));
                    c12[i][j] += (__popc(x1[i].x & w2[j].x) + __popc(x1[i].y & w2[j].y)) +
                                 (__popc(x1[i].z & w2[j].z) + __popc(x1[i].w & w2[j].w));
                    c21[i][j] += (__popc(x2[i].x & w1[j].x) + __popc(x2[i].y & w1[j].y)) +
                                 (__popc(x2[i].z & w1[j].z) + __popc(x2[i].w & w1[j].w));
                    c22[i][j] += (__popc(x2[i].x & w2[j].x) + __popc(x2[i].y & w2[j].y)) +
                                 (__popc(x2[i].z & w2[j].z) + __popc(x2[i].w & w2[j].w));
                }
        }
    }
    // shifts and the final additions, once per output
    #pragma unroll
    for (int i = 0; i < TM; ++i) {
        const int64_t m = m0 + ty + 16 * i;
        if (m >= M) continue;
        #pragma unroll
        for (int j = 0; j < TN; ++j) {
            const int64_t n = n0 + tx + 16 * j;
            if (n >= N) continue;
            out[m * N + n] = (c11[i][j] << 2) + (c12[i][j] << 1) + (c21[i][j] << 1) + c22[i][j];
        }
    }
}

cudaError_t launch_pack_quaternary(const uint8_t* q, int64_t rows, int64_t K, uint8_t* packed, unsigned* status,
                                   cudaStream_t s)
{
    const int64_t warps = rows * blocks_of(K);
    const int64_t blocks = (warps * 32 + 255) / 256;
    if (blocks > 0x7fffffff) return cudaErrorInvalidConfiguration;
    pack_quaternary_kernel<<<(unsigned)blocks, 256, 0, s>>>(q, rows, K, packed, status);
    return cudaGetLastError();
}

cudaError_t launch_gemm_quaternary(const uint8_t* a, const uint8_t* w, int64_t M, int64_t N, int64_t K, int32_t* out,
                                   cudaStream_t s)
{
    auto ctas = [&](int64_t t) { return ((M + t - 1) / t) * ((N + t - 1) / t); };
    if (ctas(64) >= device_sm_count()) {
        dim3 grid((unsigned)((M + 63) / 64), (unsigned)((N + 63) / 64));
        gemm_quaternary_kernel<4, 4><<<grid, 256, 0, s>>>(a, w, M, N, K, out);
    } else if (ctas(32) >= device_sm_count()) {
        dim3 grid((unsigned)((M + 31) / 32), (unsigned)((N + 31) / 32));
        gemm_quaternary_kernel<2, 2><<<grid, 256, 0, s>>>(a, w, M, N, K, out);
    } else {
        dim3 grid((unsigned)((M + 15) / 16), (unsigned)((N + 15) / 16));
        gemm_quaternary_kernel<1, 1><<<grid, 256, 0, s>>>(a, w, M, N, K, out);
    }
    return cudaGetLastError();
}

}  // namespace rtn
