// Packed ternary GEMM, bit-plane variant: Eq. 9 evaluated with AND / XOR / popcount on the
// packed planes, int32 accumulators, affine epilogue fused.
//
//   S_xw = bC(c) - 2 bC((W2 xor A2) and c),   c = W1 and A1            (Eq. 9)
//
// A CTA of 16x16 threads owns a (16 TM) x (16 TN) output tile; a thread owns TM x TN outputs
// (rows ty + 16 i, columns tx + 16 j).  Per 32 codes and output: 1 AND, 1 LOP3, 2 POPC and two
// integer adds into separate counters for bC(c) and bC(d), as the paper's circuit keeps two
// counters; the shift and the subtraction happen once, in the epilogue.
#include "rtn_internal.cuh"

namespace rtn {

template <int TM, int TN>
__global__ void __launch_bounds__(256)
gemm_popc_kernel(const GemmArgs g)
{
    constexpr int BM = 16 * TM, BN = 16 * TN, KB = 2;      // KB packed blocks (256 codes) per stage
    __shared__ uint4 sA[KB][2][BM];                        // [block][plane][row]
    __shared__ uint4 sB[KB][2][BN];

    const int tid = threadIdx.x;
    const int tx = tid & 15, ty = tid >> 4;
    const int64_t m0 = (int64_t)blockIdx.x * BM, n0 = (int64_t)blockIdx.y * BN;
    const int64_t nblk = (g.K + kBlockCodes - 1) / kBlockCodes;
    const uint4* __restrict__ A = reinterpret_cast<const uint4*>(g.a_packed);   // 2 uint4 per block
    const uint4* __restrict__ Wp = reinterpret_cast<const uint4*>(g.w_packed);

    int cnt_c[TM][TN], cnt_d[TM][TN];
    #pragma unroll
    for (int i = 0; i < TM; ++i)
        #pragma unroll
        for (int j = 0; j < TN; ++j) { cnt_c[i][j] = 0; cnt_d[i][j] = 0; }

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
            if (kb < nblk && grow < (isA ? g.M : g.N))
                v = __ldg((isA ? A : Wp) + (grow * nblk + kb) * 2 + plane);
            if (isA) sA[b][plane][row] = v; else sB[b][plane][row] = v;
        }
        __syncthreads();
        #pragma unroll
        for (int b = 0; b < KB; ++b) {
            uint4 a1[TM], a2[TM], w1[TN], w2[TN];
            #pragma unroll
            for (int i = 0; i < TM; ++i) { a1[i] = sA[b][0][ty + 16 * i]; a2[i] = sA[b][1][ty + 16 * i]; }
            #pragma unroll
            for (int j = 0; j < TN; ++j) { w1[j] = sB[b][0][tx + 16 * j]; w2[j] = sB[b][1][tx + 16 * j]; }
            #pragma unroll
            for (int i = 0; i < TM; ++i)
                #pragma unroll
                for (int j = 0; j < TN; ++j) {
                    const uint32_t c0 = a1[i].x & w1[j].x, c1 = a1[i].y & w1[j].y;
                    const uint32_t c2 = a1[i].z & w1[j].z, c3 = a1[i].w & w1[j].w;
                    const uint32_t d0 = (a2[i].x ^ w2[j].x) & c0, d1 = (a2[i].y ^ w2[j].y) & c1;
                    const uint32_t d2 = (a2[i].z ^ w2[j].z) & c2, d3 = (a2[i].w ^ w2[j].w) & c3;
                    cnt_c[i][j] += (__popc(c0) + __popc(c1)) + (__popc(c2) + __popc(c3));
                    cnt_d[i][j] += (__popc(d0) + __popc(d1)) + (__popc(d2) + __popc(d3));
                }
        }
    }

    // Epilogue: shift, subtract, then the four-term affine form in double, rounded once.
    const EpilogueParams& ep = g.ep;
    #pragma unroll
    for (int i = 0; i < TM; ++i) {
        const int64_t m = m0 + ty + 16 * i;
        if (m >= g.M) continue;
        const double a_s = ep.a_scale[ep.n_aparam == 1 ? 0 : m];
        const double a_o = ep.a_offset[ep.n_aparam == 1 ? 0 : m];
        const int s_x = g.a_sum[m];
        #pragma unroll
        for (int j = 0; j < TN; ++j) {
            const int64_t n = n0 + tx + 16 * j;
            if (n >= g.N) continue;
            const int s_xw = cnt_c[i][j] - 2 * cnt_d[i][j];
            const double w_s = ep.w_scale[ep.n_wparam == 1 ? 0 : n];
            const double w_o = ep.w_offset[ep.n_wparam == 1 ? 0 : n];
            g.out[m * g.N + n] = epilogue_f64(s_xw, s_x, g.w_sum[n], (double)g.K, a_s, a_o, w_s, w_o);
            if (g.dbg_acc != nullptr) g.dbg_acc[m * g.N + n] = s_xw;
        }
    }
}

// Split-K for linear layers with few rows and columns and a long K (a batch of a few samples through a
// wide layer): too few 16x16 output tiles to fill the machine, so the K range is cut into slices and
// grid.z CTAs work on one tile.  The fp32 output buffer doubles as the int32 accumulator: zeroed,
// then every slice adds its exact partial S_xw with an integer atomic, then a second kernel applies the
// affine form in place.  No workspace, and the integers stay exact whatever the order of the additions.
__global__ void __launch_bounds__(256)
gemm_popc_splitk_kernel(const GemmArgs g, int blocks_per_slice)
{
    __shared__ uint4 sA[2][16], sB[2][16];                 // [plane][row] of one packed block
    const int tid = threadIdx.x;
    const int tx = tid & 15, ty = tid >> 4;
    const int64_t m0 = (int64_t)blockIdx.x * 16, n0 = (int64_t)blockIdx.y * 16;
    const int64_t nblk = (g.K + kBlockCodes - 1) / kBlockCodes;
    const int64_t kb_begin = (int64_t)blockIdx.z * blocks_per_slice;
    const int64_t kb_end = kb_begin + blocks_per_slice < nblk ? kb_begin + blocks_per_slice : nblk;
    const uint4* __restrict__ A = reinterpret_cast<const uint4*>(g.a_packed);
    const uint4* __restrict__ Wp = reinterpret_cast<const uint4*>(g.w_packed);
    int cnt_c = 0, cnt_d = 0;
    for (int64_t kb = kb_begin; kb < kb_end; ++kb) {
        __syncthreads();
        if (tid < 64) {
            const bool isA = tid < 32;
            const int plane = (tid >> 4) & 1, row = tid & 15;
            const int64_t grow = (isA ? m0 : n0) + row;
            uint4 v = make_uint4(0, 0, 0, 0);
            if (grow < (isA ? g.M : g.N)) v = __ldg((isA ? A : Wp) + (grow * nblk + kb) * 2 + plane);
            if (isA) sA[plane][row] = v; else sB[plane][row] = v;
        }
        __syncthreads();
        const uint4 a1 = sA[0][ty], a2 = sA[1][ty], w1 = sB[0][tx], w2 = sB[1][tx];
        const uint32_t c0 = a1.x & w1.x, c1 = a1.y & w1.y, c2 = a1.z & w1.z, c3 = a1.w & w1.w;
        cnt_c += (__popc(c0) + __popc(c1)) + (__popc(c2) + __popc(c3));
        cnt_d += (__popc((a2.x ^ w2.x) & c0) + __popc((a2.y ^ w2.y) & c1)) +
                 (__popc((a2.z ^ w2.z) & c2) + __popc((a2.w ^ w2.w) & c3));
    }
    const int64_t m = m0 + ty, n = n0 + tx;
    if (m < g.M && n < g.N && kb_begin < kb_end)
        atomicAdd(reinterpret_cast<int*>(g.out) + m * g.N + n, cnt_c - 2 * cnt_d);      // Eq. 9, this slice's share
}

__global__ void gemm_epilogue_inplace_kernel(const GemmArgs g)
{
    const int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= g.M * g.N) return;
    const int64_t m = i / g.N, n = i % g.N;
    const EpilogueParams& ep = g.ep;
    const int s_xw = reinterpret_cast<const int*>(g.out)[i];
    const double a_s = ep.a_scale[ep.n_aparam == 1 ? 0 : m], a_o = ep.a_offset[ep.n_aparam == 1 ? 0 : m];
    const double w_s = ep.w_scale[ep.n_wparam == 1 ? 0 : n], w_o = ep.w_offset[ep.n_wparam == 1 ? 0 : n];
    g.out[i] = epilogue_f64(s_xw, g.a_sum[m], g.w_sum[n], (double)g.K, a_s, a_o, w_s, w_o);
    if (g.dbg_acc != nullptr) g.dbg_acc[i] = s_xw;
}

// Slices of K for a shape (1 = no split): only when the 16x16 tiles are fewer than half the SMs and K has
// at least eight packed blocks; enough slices for about two CTAs per SM, at least two blocks each.
int gemm_popc_slices(int64_t M, int64_t N, int64_t K)
{
    const int64_t tiles = ((M + 15) / 16) * ((N + 15) / 16);
    const int64_t nblk = (K + kBlockCodes - 1) / kBlockCodes;
    const int sms = device_sm_count();
    if (tiles >= sms / 2 || nblk < 8) return 1;
    int64_t slices = (2 * sms + tiles - 1) / tiles;
    if (slices > nblk / 2) slices = nblk / 2;
    return slices < 2 ? 1 : (int)slices;
}

cudaError_t launch_gemm_popc(const GemmArgs& g, cudaStream_t s)
{
    const int slices = gemm_popc_slices(g.M, g.N, g.K);
    if (slices > 1) {
        const int64_t nblk = (g.K + kBlockCodes - 1) / kBlockCodes;
        const int per_slice = (int)((nblk + slices - 1) / slices);
        cudaError_t e = cudaMemsetAsync(g.out, 0, (size_t)g.M * g.N * sizeof(float), s);
        if (e != cudaSuccess) return e;
        dim3 grid((unsigned)((g.M + 15) / 16), (unsigned)((g.N + 15) / 16), (unsigned)((nblk + per_slice - 1) / per_slice));
        gemm_popc_splitk_kernel<<<grid, 256, 0, s>>>(g, per_slice);
        e = cudaGetLastError();
        if (e != cudaSuccess) return e;
        gemm_epilogue_inplace_kernel<<<(unsigned)((g.M * g.N + 255) / 256), 256, 0, s>>>(g);
        return cudaGetLastError();
    }
    auto ctas = [&](int64_t t) { return ((g.M + t - 1) / t) * ((g.N + t - 1) / t); };
    if (ctas(64) >= device_sm_count()) {
        dim3 grid((unsigned)((g.M + 63) / 64), (unsigned)((g.N + 63) / 64));
        gemm_popc_kernel<4, 4><<<grid, 256, 0, s>>>(g);
    } else if (ctas(32) >= device_sm_count()) {
        dim3 grid((unsigned)((g.M + 31) / 32), (unsigned)((g.N + 31) / 32));
        gemm_popc_kernel<2, 2><<<grid, 256, 0, s>>>(g);
    } else {
        dim3 grid((unsigned)((g.M + 15) / 16), (unsigned)((g.N + 15) / 16));
        gemm_popc_kernel<1, 1><<<grid, 256, 0, s>>>(g);
    }
    return cudaGetLastError();
}

}  // namespace rtn
