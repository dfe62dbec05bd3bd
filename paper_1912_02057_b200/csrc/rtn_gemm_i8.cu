// Packed ternary GEMM, tensor-core variant: the bit planes are expanded to int8 {-1,0,+1} in
// shared memory and contracted with tcgen05.mma kind::i8 into int32 accumulators in tensor
// memory; the affine epilogue reads them back with tcgen05.ld.
//
// One CTA (256 threads) owns a 128 x BN output tile.  Per packed block (128 codes of K):
//   * thread t < 128 expands row t of the A tile, threads 128.. expand rows of the W tile
//     (two 128-bit loads of the row's planes, PRMT table expansion, 16-byte shared stores),
//   * after a CTA barrier one thread issues four K = 32 MMAs and commits them to the stage's
//     mbarrier, which frees the stage for re-use kStages blocks later.
// Operand tiles are K-major without swizzle: [k chunk of 16 bytes][row][16 bytes], so an
// 8-row x 16-byte core matrix is 128 contiguous bytes, and consecutive threads (rows) store
// consecutive 16-byte slots (no bank conflicts).
#include "rtn_internal.cuh"
#include "rtn_tcgen05.cuh"

namespace rtn {

namespace {

constexpr int kBM = 128;
constexpr int kStages = 3;
constexpr int kThreads = 256;

template <int BN>
struct GemmI8Smem {
    // [stage][chunk 0..7][row][16 B]
    uint4 a[kStages][8][kBM];
    uint4 b[kStages][8][BN];
    float p1[BN], p2[BN], p3[BN];       // per-column epilogue constants
    uint64_t bar_free[kStages];
    uint32_t tmem_base;
};

template <int BN>
__global__ void __launch_bounds__(kThreads)
gemm_i8_kernel(const GemmArgs g)
{
    extern __shared__ __align__(128) uint8_t smem_raw[];
    GemmI8Smem<BN>& sm = *reinterpret_cast<GemmI8Smem<BN>*>(smem_raw);

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int64_t m0 = (int64_t)blockIdx.x * kBM, n0 = (int64_t)blockIdx.y * BN;
    const int64_t nblk = (g.K + kBlockCodes - 1) / kBlockCodes;
    constexpr int kRowsPerPass = kThreads;                 // rows expanded per pass over the threads
    constexpr int kPasses = (kBM + BN) / kRowsPerPass;     // 1 (BN = 128) or ...
    static_assert((kBM + BN) % kRowsPerPass == 0, "tile rows must fill the threads");

    if (warp == 0) tc::tmem_alloc(&sm.tmem_base, BN);
    if (tid == 0) {
        for (int s = 0; s < kStages; ++s) tc::mbar_init(&sm.bar_free[s], 1);
        tc::mbar_init_fence();
    }
    // per-column constants, in double, rounded once:
    //   p1 = w_s, p2 = w_o, p3 = w_s*S_w + K*w_o
    for (int j = tid; j < BN; j += kThreads) {
        const int64_t n = n0 + j;
        float p1 = 0.f, p2 = 0.f, p3 = 0.f;
        if (n < g.N) {
            const double ws = g.ep.w_scale[g.ep.n_wparam == 1 ? 0 : n];
            const double wo = g.ep.w_offset[g.ep.n_wparam == 1 ? 0 : n];
            p1 = (float)ws; p2 = (float)wo;
            p3 = (float)(ws * (double)g.w_sum[n] + (double)g.K * wo);
        }
        sm.p1[j] = p1; sm.p2[j] = p2; sm.p3[j] = p3;
    }
    tc::tc_fence_before_sync();
    __syncthreads();
    tc::tc_fence_after_sync();
    const uint32_t tmem = sm.tmem_base;

    // rows this thread expands
    const uint4* src[kPasses];
    #pragma unroll
    for (int p = 0; p < kPasses; ++p) {
        const int r = tid + p * kRowsPerPass;              // 0..kBM-1: A rows, then W rows
        const bool isA = r < kBM;
        const int64_t grow = isA ? (m0 + r) : (n0 + r - kBM);
        const bool ok = grow < (isA ? g.M : g.N);
        src[p] = ok ? reinterpret_cast<const uint4*>((isA ? g.a_packed : g.w_packed) + grow * nblk * kBlockBytes)
                    : nullptr;
    }
    uint4 nzv[kPasses], sgv[kPasses];
    #pragma unroll
    for (int p = 0; p < kPasses; ++p) {
        nzv[p] = src[p] ? __ldg(src[p]) : make_uint4(0, 0, 0, 0);
        sgv[p] = src[p] ? __ldg(src[p] + 1) : make_uint4(0, 0, 0, 0);
    }

    constexpr uint32_t kIdesc = tc::idesc_i8(kBM, BN);
    bool alive = true;
    for (int64_t kb = 0; kb < nblk; ++kb) {
        const int s = (int)(kb % kStages);
        if (kb >= kStages)
            alive &= tc::mbar_wait(&sm.bar_free[s], (uint32_t)((kb / kStages - 1) & 1), g.status);
        #pragma unroll
        for (int p = 0; p < kPasses; ++p) {
            const uint4 nz = nzv[p], sg = sgv[p];
            if (kb + 1 < nblk && src[p]) {                 // prefetch the next block's planes
                nzv[p] = __ldg(src[p] + 2 * (kb + 1));
                sgv[p] = __ldg(src[p] + 2 * (kb + 1) + 1);
            }
            const int r = tid + p * kRowsPerPass;
            uint4* dst = (r < kBM) ? &sm.a[s][0][r] : &sm.b[s][0][r - kBM];
            const int stride = (r < kBM) ? kBM : BN;       // uint4 slots between k chunks
            uint32_t o[8];
            tc::unpack32(nz.x, sg.x, o);
            dst[0 * stride] = make_uint4(o[0], o[1], o[2], o[3]);
            dst[1 * stride] = make_uint4(o[4], o[5], o[6], o[7]);
            tc::unpack32(nz.y, sg.y, o);
            dst[2 * stride] = make_uint4(o[0], o[1], o[2], o[3]);
            dst[3 * stride] = make_uint4(o[4], o[5], o[6], o[7]);
            tc::unpack32(nz.z, sg.z, o);
            dst[4 * stride] = make_uint4(o[0], o[1], o[2], o[3]);
            dst[5 * stride] = make_uint4(o[4], o[5], o[6], o[7]);
            tc::unpack32(nz.w, sg.w, o);
            dst[6 * stride] = make_uint4(o[0], o[1], o[2], o[3]);
            dst[7 * stride] = make_uint4(o[4], o[5], o[6], o[7]);
        }
        tc::fence_smem_to_async_proxy();
        __syncthreads();
        if (tid == 0) {
            tc::tc_fence_after_sync();
            const uint32_t a_base = tc::smem_addr(&sm.a[s][0][0]);
            const uint32_t b_base = tc::smem_addr(&sm.b[s][0][0]);
            #pragma unroll
            for (int j = 0; j < 4; ++j) {                  // K = 32 per MMA = two 16-byte chunks
                const uint64_t ad = tc::smem_desc_kmajor(a_base + j * 2 * kBM * 16, kBM * 16, 128);
                const uint64_t bd = tc::smem_desc_kmajor(b_base + j * 2 * BN * 16, BN * 16, 128);
                tc::mma_i8_ss(tmem, ad, bd, kIdesc, kb > 0 || j > 0);
            }
            tc::mma_commit(&sm.bar_free[s]);
        }
    }
    // the last commit covers every MMA issued before it
    {
        const int64_t last = nblk - 1;
        alive &= tc::mbar_wait(&sm.bar_free[last % kStages], (uint32_t)((last / kStages) & 1), g.status);
    }
    tc::tc_fence_after_sync();

    // Epilogue.  Warp w reads TMEM lanes 32 (w mod 4) ..+31 (rows) and half of the columns.
    //   out = a_s * (p1*S_xw + p2*S_x) + a_o * p3
    {
        const int q = warp & 3, half = warp >> 2;
        const int64_t m = m0 + q * 32 + lane;
        const bool row_ok = m < g.M;
        float a_s = 0.f, a_o = 0.f, s_x = 0.f;
        if (row_ok) {
            a_s = g.ep.a_scale[g.ep.n_aparam == 1 ? 0 : m];
            a_o = g.ep.a_offset[g.ep.n_aparam == 1 ? 0 : m];
            s_x = (float)g.a_sum[m];
        }
        constexpr int kColsPerWarp = BN / 2;
        #pragma unroll 1
        for (int c0 = half * kColsPerWarp; c0 < (half + 1) * kColsPerWarp; c0 += 16) {
            uint32_t v[16];
            tc::tmem_ld16(tmem + ((uint32_t)(q * 32) << 16) + (uint32_t)c0, v);
            tc::tmem_ld_wait();
            if (row_ok && alive) {
                #pragma unroll
                for (int j = 0; j < 16; ++j) {
                    const int64_t n = n0 + c0 + j;
                    if (n < g.N) {
                        const int s_xw = (int)v[j];
                        const float u = fmaf(sm.p1[c0 + j], (float)s_xw, sm.p2[c0 + j] * s_x);
                        g.out[m * g.N + n] = fmaf(a_s, u, a_o * sm.p3[c0 + j]);
                        if (g.dbg_acc != nullptr) g.dbg_acc[m * g.N + n] = s_xw;
                    }
                }
            }
        }
    }
    tc::tc_fence_before_sync();
    __syncthreads();
    if (warp == 0) tc::tmem_dealloc(tmem, BN);
}

}  // namespace

bool gemm_i8_supported(int64_t M, int64_t N, int64_t K)
{
    return M >= 1 && N >= 1 && K >= 1 && (M + kBM - 1) / kBM <= 0x7fffffff && (N + 127) / 128 <= 65535;
}

cudaError_t launch_gemm_i8(const GemmArgs& g, cudaStream_t s)
{
    constexpr int BN = 128;
    const size_t smem = sizeof(GemmI8Smem<BN>) + 128;
    cudaError_t e = cudaFuncSetAttribute(gemm_i8_kernel<BN>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return e;
    dim3 grid((unsigned)((g.M + kBM - 1) / kBM), (unsigned)((g.N + BN - 1) / BN));
    gemm_i8_kernel<BN><<<grid, kThreads, smem, s>>>(g);
    return cudaGetLastError();
}

}  // namespace rtn
