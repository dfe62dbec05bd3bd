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
    if (blocks > device_sm_count() * 64) blocks = device_sm_count() * 64;
    pack_weights_kernel<<<(unsigned)blocks, threads, 0, s>>>(w, N, C, kh, kw, packed, w_sum, status);
    return cudaGetLastError();
}

// ---------------------------------------------------------------------------------------------
// Activations [M][K] fp32.  A team of wpr warps (1, 2, 4 or 8 of the block's eight) walks one row, a warp
// four 128-code blocks per trip: lane l reads a[k0 + l + 32 j], j = 0..15 (sixteen coalesced 128-byte
// requests in flight), and __ballot_sync over the comparison results is word j & 3 of a plane of block
// j >> 2 -- bit l of that word is code k0 + 32 j + l, which is the packed format's bit order.  Lane
// 8 i + q then writes word q of block i (one 128-byte store).  Long rows are spread over the block's
// warps so that a row's loads are all in flight at once instead of trip after trip; the team's partial
// code sums meet in shared memory.
// ---------------------------------------------------------------------------------------------
template <bool kPerK>
__global__ void __launch_bounds__(256, 4)
ternarize_pack_kernel(const float* __restrict__ a, int64_t M, int64_t K,
                      const float* __restrict__ t_lo, const float* __restrict__ t_hi,
                      uint8_t* __restrict__ packed, int32_t* __restrict__ a_sum, int wpr)
{
    __shared__ int ssum[8];
    const int lane = threadIdx.x & 31, w = threadIdx.x >> 5;
    const int rpb = 8 / wpr, sub = w % wpr, rloc = w / wpr;      // rows per block and trip; place in the team; row slot
    const int64_t nblk = (K + kBlockCodes - 1) / kBlockCodes;
    const float lo0 = t_lo[0], hi0 = t_hi[0];
    if (threadIdx.x < 8) ssum[threadIdx.x] = 0;

    for (int64_t mb = (int64_t)blockIdx.x * rpb; mb < M; mb += (int64_t)gridDim.x * rpb) {    // the same for the whole block
        const int64_t m = mb + rloc;
        __syncthreads();                                          // ssum zeroed (start, or by the writer below)
        int sum = 0;
        if (m < M) {
            const float* row = a + m * K;
            uint32_t* dst = reinterpret_cast<uint32_t*>(packed + m * nblk * kBlockBytes);
            for (int64_t b0 = (int64_t)sub * 4; b0 < nblk; b0 += 4 * wpr) {
                float v[16];
                #pragma unroll
                for (int j = 0; j < 16; ++j) {
                    const int64_t k = b0 * kBlockCodes + j * 32 + lane;
                    v[j] = k < K ? __ldg(row + k) : 0.0f;
                }
                uint32_t mine = 0;       // lane 8 i + q keeps word q of block b0 + i
                #pragma unroll
                for (int j = 0; j < 16; ++j) {
                    const int64_t k = b0 * kBlockCodes + j * 32 + lane;
                    float lo = lo0, hi = hi0;
                    if (kPerK && k < K) { lo = __ldg(t_lo + k); hi = __ldg(t_hi + k); }
                    if (k >= K) { lo = -1.0f; hi = 1.0f; }        // padding codes to 0 (v = 0 there)
                    bool nz, pos;
                    ternarize(v[j], lo, hi, nz, pos);
                    const uint32_t wn = __ballot_sync(0xffffffffu, nz);
                    const uint32_t wp = __ballot_sync(0xffffffffu, pos);
                    sum += __popc(wp) - __popc(wn & ~wp);
                    const int blk = j >> 2, q = j & 3;
                    if (lane == blk * 8 + q) mine = wn;
                    if (lane == blk * 8 + 4 + q) mine = wp;
                }
                const int64_t blk = b0 + (lane >> 3);
                if (blk < nblk) dst[blk * 8 + (lane & 7)] = mine;
            }
        }
        if (a_sum == nullptr) continue;                           // (uniform)
        if (wpr == 1) {
            if (lane == 0 && m < M) a_sum[m] = sum;               // every lane holds the same sum (ballots)
            continue;
        }
        if (lane == 0 && sum != 0) atomicAdd(&ssum[rloc], sum);
        __syncthreads();
        if (sub == 0 && lane == 0) {
            if (m < M) a_sum[m] = ssum[rloc];
            ssum[rloc] = 0;
        }
    }
}

// The same for rows whose length is a multiple of 8 and whose data are 16-byte aligned: a lane reads EIGHT
// consecutive values (two float4) of a 256-code unit and builds the two plane bytes they make itself -- lane l of a
// unit holds byte l & 3 of word (l & 15) >> 2 of block l >> 4 -- so that the comparisons' results never go
// through a warp vote: a quarter of the scalar kernel's instructions per value, which is what bounds it (the
// scalar kernel issues ~19 instructions per 128 bytes read).  Two shuffles OR the four bytes of a word together,
// one more brings word q of block i to lane 8 i + q, which stores as before.  A trip is two units (four blocks).
template <bool kPerK>
__global__ void __launch_bounds__(256, 4)
ternarize_pack_vec_kernel(const float* __restrict__ a, int64_t M, int64_t K,
                          const float* __restrict__ t_lo, const float* __restrict__ t_hi,
                          uint8_t* __restrict__ packed, int32_t* __restrict__ a_sum, int wpr)
{
    __shared__ int ssum[8];
    const int lane = threadIdx.x & 31, w = threadIdx.x >> 5;
    const int rpb = 8 / wpr, sub = w % wpr, rloc = w / wpr;
    const int64_t nblk = (K + kBlockCodes - 1) / kBlockCodes;
    const float lo0 = t_lo[0], hi0 = t_hi[0];
    if (threadIdx.x < 8) ssum[threadIdx.x] = 0;
    // where this lane's word comes from after the OR: unit lane >> 4, quad (block of the unit, word of the plane)
    const int src = 4 * (((lane >> 3) & 1) * 4 + (lane & 3));

    for (int64_t mb = (int64_t)blockIdx.x * rpb; mb < M; mb += (int64_t)gridDim.x * rpb) {
        const int64_t m = mb + rloc;
        __syncthreads();
        int sum = 0;
        if (m < M) {
            const float* row = a + m * K;
            uint32_t* dst = reinterpret_cast<uint32_t*>(packed + m * nblk * kBlockBytes);
            for (int64_t b0 = (int64_t)sub * 4; b0 < nblk; b0 += 4 * wpr) {
                float4 x[2][2];
                #pragma unroll
                for (int u = 0; u < 2; ++u) {
                    const int64_t k = (b0 + 2 * u) * kBlockCodes + 8 * lane;
                    const bool in = k < K;                                  // K is a multiple of 8: all eight or none
                    x[u][0] = in ? __ldg(reinterpret_cast<const float4*>(row + k)) : make_float4(0.f, 0.f, 0.f, 0.f);
                    x[u][1] = in ? __ldg(reinterpret_cast<const float4*>(row + k) + 1) : make_float4(0.f, 0.f, 0.f, 0.f);
                }
                uint32_t mine = 0;
                #pragma unroll
                for (int u = 0; u < 2; ++u) {
                    const int64_t k = (b0 + 2 * u) * kBlockCodes + 8 * lane;
                    const float v[8] = {x[u][0].x, x[u][0].y, x[u][0].z, x[u][0].w, x[u][1].x, x[u][1].y, x[u][1].z, x[u][1].w};
                    float lo[8], hi[8];
                    if (kPerK && k < K) {
                        const float4 l0 = __ldg(reinterpret_cast<const float4*>(t_lo + k)), l1 = __ldg(reinterpret_cast<const float4*>(t_lo + k) + 1);
                        const float4 h0 = __ldg(reinterpret_cast<const float4*>(t_hi + k)), h1 = __ldg(reinterpret_cast<const float4*>(t_hi + k) + 1);
                        lo[0] = l0.x; lo[1] = l0.y; lo[2] = l0.z; lo[3] = l0.w; lo[4] = l1.x; lo[5] = l1.y; lo[6] = l1.z; lo[7] = l1.w;
                        hi[0] = h0.x; hi[1] = h0.y; hi[2] = h0.z; hi[3] = h0.w; hi[4] = h1.x; hi[5] = h1.y; hi[6] = h1.z; hi[7] = h1.w;
                    } else {
                        #pragma unroll
                        for (int t = 0; t < 8; ++t) { lo[t] = lo0; hi[t] = hi0; }
                    }
                    uint32_t nzb = 0, posb = 0;
                    if (k < K) {
                        #pragma unroll
                        for (int t = 0; t < 8; ++t) {
                            bool nz, pos;
                            ternarize(v[t], lo[t], hi[t], nz, pos);
                            nzb |= nz ? (1u << t) : 0u;
                            posb |= pos ? (1u << t) : 0u;
                        }
                    }
                    sum += __popc(posb) - __popc(nzb & ~posb);
                    uint32_t xn = nzb << (8 * (lane & 3)), xp = posb << (8 * (lane & 3));
                    xn |= __shfl_xor_sync(0xffffffffu, xn, 1);
                    xp |= __shfl_xor_sync(0xffffffffu, xp, 1);
                    xn |= __shfl_xor_sync(0xffffffffu, xn, 2);
                    xp |= __shfl_xor_sync(0xffffffffu, xp, 2);
                    const uint32_t wn = __shfl_sync(0xffffffffu, xn, src), wp = __shfl_sync(0xffffffffu, xp, src);
                    if ((lane >> 4) == u) mine = (lane & 4) ? wp : wn;
                }
                const int64_t blk = b0 + (lane >> 3);
                if (blk < nblk) dst[blk * 8 + (lane & 7)] = mine;
            }
        }
        if (a_sum == nullptr) continue;
        sum = __reduce_add_sync(0xffffffffu, sum);
        if (wpr == 1) {
            if (lane == 0 && m < M) a_sum[m] = sum;
            continue;
        }
        if (lane == 0 && sum != 0) atomicAdd(&ssum[rloc], sum);
        __syncthreads();
        if (sub == 0 && lane == 0) {
            if (m < M) a_sum[m] = ssum[rloc];
            ssum[rloc] = 0;
        }
    }
}

// Short rows of 32, 64, 128 or 256 values (the channel counts of pixel rows): a row would leave most of a warp's
// lanes of the kernel above without work, so here the matrix is walked as one flat array, 256 values per warp and
// unit; 256 / K rows share a unit, lane l holds eight values of row (8 l) / K, a quad still holds one plane word,
// and the row's code sum is added up over its K / 8 lanes.  The quad's first lane stores the two words (and, for
// K < 128, the first quad of a row the block's unused words as zeros).  Two units per trip.
template <bool kPerK>
__global__ void __launch_bounds__(256, 4)
ternarize_pack_rows_kernel(const float* __restrict__ a, int64_t M, int K,
                           const float* __restrict__ t_lo, const float* __restrict__ t_hi,
                           uint8_t* __restrict__ packed, int32_t* __restrict__ a_sum)
{
    const int lane = threadIdx.x & 31;
    const int64_t warp = (blockIdx.x * (int64_t)blockDim.x + threadIdx.x) >> 5;
    const int64_t nwarps = ((int64_t)gridDim.x * blockDim.x) >> 5;
    const int64_t total = M * K, nunits = (total + 255) / 256;
    const int lanes_per_row = K / 8, words = K / 32, nblk = (K + kBlockCodes - 1) / kBlockCodes;
    const float lo0 = t_lo[0], hi0 = t_hi[0];

    for (int64_t u0 = warp * 2; u0 < nunits; u0 += nwarps * 2) {
        float4 x[2][2];
        #pragma unroll
        for (int u = 0; u < 2; ++u) {
            const int64_t flat = (u0 + u) * 256 + 8 * lane;
            const bool in = flat < total;                        // total is a multiple of 32
            x[u][0] = in ? __ldg(reinterpret_cast<const float4*>(a + flat)) : make_float4(0.f, 0.f, 0.f, 0.f);
            x[u][1] = in ? __ldg(reinterpret_cast<const float4*>(a + flat) + 1) : make_float4(0.f, 0.f, 0.f, 0.f);
        }
        #pragma unroll
        for (int u = 0; u < 2; ++u) {
            const int64_t flat = (u0 + u) * 256 + 8 * lane;
            const bool in = flat < total;
            const int64_t m = flat / K;
            const int col = (int)(flat - m * K);
            const float v[8] = {x[u][0].x, x[u][0].y, x[u][0].z, x[u][0].w, x[u][1].x, x[u][1].y, x[u][1].z, x[u][1].w};
            float lo[8], hi[8];
            if (kPerK && in) {
                const float4 l0 = __ldg(reinterpret_cast<const float4*>(t_lo + col)), l1 = __ldg(reinterpret_cast<const float4*>(t_lo + col) + 1);
                const float4 h0 = __ldg(reinterpret_cast<const float4*>(t_hi + col)), h1 = __ldg(reinterpret_cast<const float4*>(t_hi + col) + 1);
                lo[0] = l0.x; lo[1] = l0.y; lo[2] = l0.z; lo[3] = l0.w; lo[4] = l1.x; lo[5] = l1.y; lo[6] = l1.z; lo[7] = l1.w;
                hi[0] = h0.x; hi[1] = h0.y; hi[2] = h0.z; hi[3] = h0.w; hi[4] = h1.x; hi[5] = h1.y; hi[6] = h1.z; hi[7] = h1.w;
            } else {
                #pragma unroll
                for (int t = 0; t < 8; ++t) { lo[t] = lo0; hi[t] = hi0; }
            }
            uint32_t nzb = 0, posb = 0;
            if (in) {
                #pragma unroll
                for (int t = 0; t < 8; ++t) {
                    bool nz, pos;
                    ternarize(v[t], lo[t], hi[t], nz, pos);
                    nzb |= nz ? (1u << t) : 0u;
                    posb |= pos ? (1u << t) : 0u;
                }
            }
            int sum = __popc(posb) - __popc(nzb & ~posb);
            uint32_t xn = nzb << (8 * (lane & 3)), xp = posb << (8 * (lane & 3));
            xn |= __shfl_xor_sync(0xffffffffu, xn, 1);
            xp |= __shfl_xor_sync(0xffffffffu, xp, 1);
            xn |= __shfl_xor_sync(0xffffffffu, xn, 2);
            xp |= __shfl_xor_sync(0xffffffffu, xp, 2);
            for (int d = 1; d < lanes_per_row; d <<= 1) sum += __shfl_xor_sync(0xffffffffu, sum, d);
            if (in) {
                uint32_t* dst = reinterpret_cast<uint32_t*>(packed + m * nblk * kBlockBytes);
                const int wj = col >> 5;                            // the word of the row this quad holds
                if ((lane & 3) == 0) {
                    dst[(wj >> 2) * 8 + (wj & 3)] = xn;
                    dst[(wj >> 2) * 8 + 4 + (wj & 3)] = xp;
                    if (wj == 0)
                        for (int z = words; z < 4; ++z) { dst[z] = 0u; dst[4 + z] = 0u; }
                }
                if (a_sum != nullptr && col == 0) a_sum[m] = sum;
            }
        }
    }
}

cudaError_t launch_ternarize_pack(const float* a, int64_t M, int64_t K, const float* t_lo,
                                  const float* t_hi, int64_t n_thr, uint8_t* packed, int32_t* a_sum,
                                  cudaStream_t s)
{
    const int threads = 256;
    const int64_t ntrip = ((K + kBlockCodes - 1) / kBlockCodes + 3) / 4;      // four-block trips a row takes
    const int wpr = ntrip >= 8 ? 8 : ntrip >= 4 ? 4 : ntrip >= 2 ? 2 : 1;
    const int rpb = 8 / wpr;
    int64_t blocks = (M + rpb - 1) / rpb;
    if (blocks > device_sm_count() * 16) blocks = device_sm_count() * 16;
    const bool per_k = n_thr != 1;
    const bool vec = (K % 8) == 0 && (reinterpret_cast<uintptr_t>(a) & 15) == 0 &&
                     (!per_k || ((reinterpret_cast<uintptr_t>(t_lo) | reinterpret_cast<uintptr_t>(t_hi)) & 15) == 0);
    if (vec && (K == 32 || K == 64 || K == 128 || K == 256)) {
        const int64_t units = (M * K + 255) / 256, warps = (units + 1) / 2;
        int64_t blk = (warps + 7) / 8;
        if (blk > device_sm_count() * 16) blk = device_sm_count() * 16;
        if (!per_k)
            ternarize_pack_rows_kernel<false><<<(unsigned)blk, threads, 0, s>>>(a, M, (int)K, t_lo, t_hi, packed, a_sum);
        else
            ternarize_pack_rows_kernel<true><<<(unsigned)blk, threads, 0, s>>>(a, M, (int)K, t_lo, t_hi, packed, a_sum);
        return cudaGetLastError();
    }
    if (vec && !per_k)
        ternarize_pack_vec_kernel<false><<<(unsigned)blocks, threads, 0, s>>>(a, M, K, t_lo, t_hi, packed, a_sum, wpr);
    else if (vec)
        ternarize_pack_vec_kernel<true><<<(unsigned)blocks, threads, 0, s>>>(a, M, K, t_lo, t_hi, packed, a_sum, wpr);
    else if (!per_k)
        ternarize_pack_kernel<false><<<(unsigned)blocks, threads, 0, s>>>(a, M, K, t_lo, t_hi, packed, a_sum, wpr);
    else
        ternarize_pack_kernel<true><<<(unsigned)blocks, threads, 0, s>>>(a, M, K, t_lo, t_hi, packed, a_sum, wpr);
    return cudaGetLastError();
}

}  // namespace rtn
