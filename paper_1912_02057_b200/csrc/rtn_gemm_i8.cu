// Packed ternary GEMM, tensor-core variant: the bit planes of both operands (Table 1; A1, A2, W1,
// W2 of Eq. 9) are expanded to int8 {-1,0,+1} in shared memory and contracted with tcgen05.mma
// kind::i8 into int32 accumulators in tensor memory; the affine epilogue (Eq. 10 with a weight
// offset) reads them back with tcgen05.ld.
//
// Persistent CTA per SM walking 128*TM x BN output tiles, warp-specialised and decoupled through
// mbarriers (no CTA-wide barrier in the main loop):
//   warps 12..19  expanders: per packed block (128 codes of K) each thread expands whole rows of
//                 the A and W tiles (two 128-bit plane loads fetched two blocks ahead, PRMT table
//                 expansion, 16-byte shared stores) into a ring of stages, then fences and arrives
//   warp  0       one thread waits for a stage, issues its 4*TM MMAs (K = 32 each) and commits them
//                 to the stage's "empty" barrier; after the last block it commits the accumulators
//   warps 4..11   epilogue: tcgen05.ld, out = a_s (w_s S_xw + w_o S_x) + a_o (w_s S_w + K w_o), transposed
//                 through a small staging block so that a warp store covers whole sectors of 16 rows
//   warp  1       (operands expanded ahead of the kernel, see gemm_pre_mode) one thread fills the weight part of
//                 every stage, or both parts, with bulk asynchronous copies from the scratch buffer
//                 gemm_expand_operands_kernel wrote; with both parts copied the expander warps join the epilogue
// Operand stages are K-major without swizzle: [16-byte k chunk][row][16 B]; an 8-row core matrix is
// 128 contiguous bytes and consecutive threads (rows) store consecutive 16-byte slots.
#include "rtn_internal.cuh"
#include "rtn_tcgen05.cuh"
#include "rtn_timeline.cuh"
#include "rtn_tensormap.cuh"

// Timeline slots (instrumented build only): 0 kernel entry, 1 set-up done (expanded operands visible), 4 kernel end;
// per tile i < 8 of the CTA: 40+2i first stage of the tile ready for the tensor core, 41+2i accumulators committed,
// 56+2i / 57+2i epilogue (thread 0 of its first warp) begins / ends.
RTN_TL_DEFINE(gemm_i8)
#include "rtn_conv_i8_common.cuh"

namespace rtn {

namespace {

using conv_detail::wait_or_die;

constexpr int kEpiWarp0 = 4;
constexpr int kEpiWarps = 8;
constexpr int kEpiThreads = kEpiWarps * 32;
constexpr int kExpWarp0 = kEpiWarp0 + kEpiWarps;
constexpr int kExpWarps = 8;
constexpr int kExpThreads = kExpWarps * 32;
constexpr int kThreads = (kExpWarp0 + kExpWarps) * 32;
constexpr int kMaxStages = 6;
constexpr size_t kSmemLimit = 226 * 1024;
constexpr int kEpiBarrier = 3;
// Output staging of the epilogue: per warp 32 rows x 8 columns of fp32, rows 48 bytes apart (32 + 16: both the
// row-wise writes and the 8-rows-by-one-chunk reads of a quarter warp then fall on distinct banks).
constexpr int kStageRow = 48;
constexpr int kStageWarp = 32 * kStageRow;
constexpr int kMaxEpiWarps = kEpiWarps + kExpWarps;     // with both operands expanded ahead the expander warps join
// Output through TMA stores: a warp stages 32 rows x 16 columns of fp32 (64-byte rows, the 64-byte swizzle of the
// tensor map: 16-byte chunk c of row r sits at chunk c ^ ((r >> 1) & 3), which also makes a quarter warp's row-wise
// writes fall on distinct banks) and one thread hands the block to the copy engine, which writes whole row segments
// while the warp works on the next block.  No global store instruction and no address arithmetic in the warp.
constexpr int kTmaStageWarp = 32 * 64;
constexpr int kTmaCols = 16;
constexpr int kTmaWarpsPre = 12;                        // warps that write out when the expander warps are free to help

struct GemmI8Plan {
    int TM;                 // 128-row sub-tiles per tile
    int BN;                 // tile columns (multiple of 16, <= 256)
    int nAcc;               // accumulator sets
    int stages;
    int rows;               // rows per stage: TM*128 + BN
    int64_t tiles_m, tiles_n, tiles;
    int grid;
    uint32_t tmem_cols;
    uint32_t stage_bytes, off_stage, off_c, off_bar, off_misc, off_t;
    size_t smem_bytes;
    int tma_out;            // the epilogue writes the output with TMA stores (set by the launcher)
};

bool make_gemm_plan(int64_t M, int64_t N, int64_t K, GemmI8Plan& p, int sms)
{
    if (M < 1 || N < 1 || K < 1) return false;
    // Tile shape by a cost model: a K = 128 stage costs the slower of its MMAs (2 TM BN cycles) and of
    // expanding its rows from bit planes (about 4 cycles per row of A or W; this is what binds), and
    // a CTA runs ceil(tiles / SMs) tiles.  Larger tiles expand fewer rows per MAC, smaller ones
    // fill the machine more evenly.
    const int bn_full = (int)((N >= 256) ? 256 : (N + 15) / 16 * 16);
    double best = 0.0;
    p.TM = 2; p.BN = bn_full;
    for (int tm = 2; tm >= 1; --tm) {
        for (int bn = bn_full; bn >= 128 || bn == bn_full; bn = (bn > 128 ? 128 : 0)) {
            const int64_t nt = ((M + 128 * tm - 1) / (128 * tm)) * ((N + bn - 1) / bn);
            const int64_t rounds = (nt + sms - 1) / sms;
            const double mma = 2.0 * tm * bn, expand = 4.0 * (128 * tm + bn);
            const double cost = (double)rounds * (mma > expand ? mma : expand);
            if (best == 0.0 || cost < best) { best = cost; p.TM = tm; p.BN = bn; }
            if (bn <= 128) break;
        }
    }
    p.nAcc = (2 * p.TM * p.BN <= 512) ? 2 : 1;
    p.tiles_m = (M + 128 * p.TM - 1) / (128 * p.TM);
    p.tiles_n = (N + p.BN - 1) / p.BN;
    p.tiles = p.tiles_m * p.tiles_n;
    if (p.tiles > 0x7fffffff) return false;
    p.grid = (int)(p.tiles < sms ? p.tiles : sms);
    p.rows = p.TM * 128 + p.BN;
    p.stage_bytes = (uint32_t)p.rows * 128;
    uint32_t cols = 32;
    while (cols < (uint32_t)(p.nAcc * p.TM * p.BN)) cols *= 2;
    p.tmem_cols = cols;
    uint32_t o = 0;
    p.off_c = o;    o += (uint32_t)p.BN * 16;                  // float4 {p1, p2, p3, 0} per column
    p.off_bar = o;  o += (4 + 2 * kMaxStages) * 8;             // acc_full[2] acc_empty[2] full[] empty[]
    p.off_misc = o; o += 16;
    o = (o + 1023) / 1024 * 1024;                              // the swizzled staging blocks want 1 KB alignment
    p.off_t = o;                                               // staging of either way of writing out
    o += kMaxEpiWarps * kStageWarp > 1024 + kTmaWarpsPre * kTmaStageWarp ? kMaxEpiWarps * kStageWarp
                                                                           : 1024 + kTmaWarpsPre * kTmaStageWarp;
    p.tma_out = 0;
    o = (o + 127) / 128 * 128;
    p.off_stage = o;
    int ns = (int)((kSmemLimit - o) / p.stage_bytes);
    if (ns > kMaxStages) ns = kMaxStages;
    if (ns < 2) return false;
    p.stages = ns;
    p.smem_bytes = o + (uint32_t)ns * p.stage_bytes;
    return true;
}

// Operands expanded once: wexp[column tile][packed block of K][16-byte k chunk (8)][row of the tile (BN)][16 B]
// and, when aexp is not null, aexp[row tile][block][chunk][row of the tile (128 TM)][16 B]: the bytes the weight
// and the activation part of a ring stage hold.  Thread = (operand, tile, block, row).
__global__ void __launch_bounds__(256)
gemm_expand_operands_kernel(const GemmArgs g, const __grid_constant__ GemmI8Plan p, uint4* __restrict__ wexp,
                            uint4* __restrict__ aexp)
{
    tc::pdl_trigger();
    const int64_t nblk = (g.K + kBlockCodes - 1) / kBlockCodes;
    const int64_t items_w = p.tiles_n * nblk * p.BN;
    int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    const bool isA = i >= items_w;
    if (isA) i -= items_w;
    const int R = isA ? p.TM * 128 : p.BN;                  // rows of a tile of this operand
    if (isA && (aexp == nullptr || i >= p.tiles_m * nblk * R)) return;
    const int r = (int)(i % R);
    const int64_t tk = i / R, kb = tk % nblk, t = tk / nblk;
    const int64_t row = t * R + r;
    uint4 nz = make_uint4(0, 0, 0, 0), sg = nz;
    if (row < (isA ? g.M : g.N)) {
        const uint4* src = reinterpret_cast<const uint4*>((isA ? g.a_packed : g.w_packed) + (row * nblk + kb) * kBlockBytes);
        nz = __ldg(src);
        sg = __ldg(src + 1);
    }
    uint4* dst = (isA ? aexp : wexp) + tk * 8 * R + r;
    uint32_t o[8];
    tc::unpack32(nz.x, sg.x, o);
    dst[0 * R] = make_uint4(o[0], o[1], o[2], o[3]);
    dst[1 * R] = make_uint4(o[4], o[5], o[6], o[7]);
    tc::unpack32(nz.y, sg.y, o);
    dst[2 * R] = make_uint4(o[0], o[1], o[2], o[3]);
    dst[3 * R] = make_uint4(o[4], o[5], o[6], o[7]);
    tc::unpack32(nz.z, sg.z, o);
    dst[4 * R] = make_uint4(o[0], o[1], o[2], o[3]);
    dst[5 * R] = make_uint4(o[4], o[5], o[6], o[7]);
    tc::unpack32(nz.w, sg.w, o);
    dst[6 * R] = make_uint4(o[0], o[1], o[2], o[3]);
    dst[7 * R] = make_uint4(o[4], o[5], o[6], o[7]);
}

// kPreW: the weight part of every stage comes from the scratch buffer gemm_expand_operands_kernel wrote (one
// bulk asynchronous copy per stage, issued by a thread of warp 1), so the expander warps expand only the
// activation rows: half of the integer work that paces the kernel.  kPreA (only with kPreW): the activation
// part too; the expander warps then have nothing to do and the ring is paced by the copies and the MMAs.
template <bool kPreW, bool kPreA>
__global__ void __launch_bounds__(kThreads, 1)
gemm_i8_kernel(const GemmArgs g, const __grid_constant__ GemmI8Plan p, const uint4* __restrict__ wexp,
               const uint4* __restrict__ aexp, const __grid_constant__ CUtensorMap omap)
{
    extern __shared__ __align__(128) uint8_t smem[];
    float4* sC = reinterpret_cast<float4*>(smem + p.off_c);
    uint64_t* bars = reinterpret_cast<uint64_t*>(smem + p.off_bar);
    uint64_t* acc_full = bars;          // [2] MMA -> epilogue
    uint64_t* acc_empty = bars + 2;     // [2] epilogue -> MMA
    uint64_t* full = bars + 4;                      // [stages] expanders -> MMA
    uint64_t* empty = bars + 4 + kMaxStages;        // [stages] MMA -> expanders
    uint32_t* slot = reinterpret_cast<uint32_t*>(smem + p.off_misc);
    volatile int* dead = reinterpret_cast<volatile int*>(smem + p.off_misc + 8);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int64_t nblk = (g.K + kBlockCodes - 1) / kBlockCodes;
    const int rowsA = p.TM * 128;

    RTN_TL_INIT(gemm_i8)
    if (threadIdx.x == 0) RTN_TL(gemm_i8, 0);
    if (warp == 0) tc::tmem_alloc(slot, p.tmem_cols);
    if (threadIdx.x == 32) {
        for (int i = 0; i < 2; ++i) { tc::mbar_init(&acc_full[i], 1); tc::mbar_init(&acc_empty[i], kPreA ? kMaxEpiWarps * 32 : kEpiThreads); }
        for (int i = 0; i < kMaxStages; ++i) { tc::mbar_init(&full[i], kPreA ? 1 : kExpWarps + (kPreW ? 1 : 0)); tc::mbar_init(&empty[i], 1); }
        tc::mbar_init_fence();
        *dead = 0;
    }
    tc::tc_fence_before_sync();
    __syncthreads();
    tc::tc_fence_after_sync();
    const uint32_t tmem = *slot;
    if constexpr (kPreW) tc::pdl_wait();           // the expanded weights come from the kernel before
    if (threadIdx.x == 0) RTN_TL(gemm_i8, 1);

    if (!kPreA && warp >= kExpWarp0) {
        // ------------------------------------------------------------ expanders
        {
        const int tid = threadIdx.x - kExpWarp0 * 32;
        uint32_t count = 0;                                   // stages produced so far
        for (int64_t tile = blockIdx.x; tile < p.tiles; tile += gridDim.x) {
            const int64_t m0 = (tile / p.tiles_n) * rowsA, n0 = (tile % p.tiles_n) * p.BN;
            // up to two rows per thread and stage: row r of the stage is A row m0 + r or W row n0 + r - rowsA
            const uint4* src[2];
            uint4* dst_off[2];
            int stride[2];
            #pragma unroll
            for (int k = 0; k < 2; ++k) {
                const int r = tid + k * kExpThreads;
                src[k] = nullptr; dst_off[k] = nullptr; stride[k] = 0;
                if (r < (kPreW ? rowsA : p.rows)) {
                    const bool isA = r < rowsA;
                    const int64_t grow = isA ? m0 + r : n0 + (r - rowsA);
                    if (grow < (isA ? g.M : g.N))
                        src[k] = reinterpret_cast<const uint4*>((isA ? g.a_packed : g.w_packed) + grow * nblk * kBlockBytes);
                    // byte offset of this row's first chunk inside a stage
                    dst_off[k] = reinterpret_cast<uint4*>((size_t)(isA ? r : rowsA * 8 + (r - rowsA)) * 16);
                    stride[k] = isA ? rowsA : p.BN;
                }
            }
            // planes of the next two blocks, in registers
            uint4 nz[2][2], sg[2][2];
            #pragma unroll
            for (int d = 0; d < 2; ++d)
                #pragma unroll
                for (int k = 0; k < 2; ++k) {
                    const bool ok = src[k] != nullptr && d < nblk;
                    nz[d][k] = ok ? __ldg(src[k] + 2 * d) : make_uint4(0, 0, 0, 0);
                    sg[d][k] = ok ? __ldg(src[k] + 2 * d + 1) : make_uint4(0, 0, 0, 0);
                }
            for (int64_t kb = 0; kb < nblk; ++kb, ++count) {
                const uint32_t s = count % (uint32_t)p.stages;
                uint4 cnz[2], csg[2];
                #pragma unroll
                for (int k = 0; k < 2; ++k) {
                    cnz[k] = nz[0][k]; csg[k] = sg[0][k];
                    nz[0][k] = nz[1][k]; sg[0][k] = sg[1][k];
                    const bool ok = src[k] != nullptr && kb + 2 < nblk;
                    nz[1][k] = ok ? __ldg(src[k] + 2 * (kb + 2)) : make_uint4(0, 0, 0, 0);
                    sg[1][k] = ok ? __ldg(src[k] + 2 * (kb + 2) + 1) : make_uint4(0, 0, 0, 0);
                }
                wait_or_die(&empty[s], ((count / (uint32_t)p.stages) & 1) ^ 1, g.status, dead);
                uint8_t* stage = smem + p.off_stage + s * p.stage_bytes;
                #pragma unroll
                for (int k = 0; k < 2; ++k) {
                    if (stride[k] == 0) continue;
                    uint4* dst = reinterpret_cast<uint4*>(stage + reinterpret_cast<size_t>(dst_off[k]));
                    const int st = stride[k];
                    uint32_t o[8];
                    tc::unpack32(cnz[k].x, csg[k].x, o);
                    dst[0 * st] = make_uint4(o[0], o[1], o[2], o[3]);
                    dst[1 * st] = make_uint4(o[4], o[5], o[6], o[7]);
                    tc::unpack32(cnz[k].y, csg[k].y, o);
                    dst[2 * st] = make_uint4(o[0], o[1], o[2], o[3]);
                    dst[3 * st] = make_uint4(o[4], o[5], o[6], o[7]);
                    tc::unpack32(cnz[k].z, csg[k].z, o);
                    dst[4 * st] = make_uint4(o[0], o[1], o[2], o[3]);
                    dst[5 * st] = make_uint4(o[4], o[5], o[6], o[7]);
                    tc::unpack32(cnz[k].w, csg[k].w, o);
                    dst[6 * st] = make_uint4(o[0], o[1], o[2], o[3]);
                    dst[7 * st] = make_uint4(o[4], o[5], o[6], o[7]);
                }
                tc::fence_smem_to_async_proxy();
                __syncwarp();
                if (lane == 0) tc::mbar_arrive(&full[s]);
            }
        }
        }
    } else if (kPreW && warp == 1) {
        // ------------------------------------------------------------ weight stages from scratch (one thread)
        if (lane == 0) {
            const uint32_t w_bytes = (uint32_t)p.BN * 128u;
            const uint32_t w_off = (uint32_t)rowsA * 128u;            // the weight block follows the activation block
            const uint32_t a_bytes = kPreA ? w_off : 0u;
            uint32_t count = 0;
            bool alive = true;
            for (int64_t tile = blockIdx.x; tile < p.tiles && alive; tile += gridDim.x) {
                const int64_t tn = tile % p.tiles_n, tm = tile / p.tiles_n;
                for (int64_t kb = 0; kb < nblk; ++kb, ++count) {
                    const uint32_t s = count % (uint32_t)p.stages;
                    if (!wait_or_die(&empty[s], ((count / (uint32_t)p.stages) & 1) ^ 1, g.status, dead)) { alive = false; break; }
                    tc::mbar_arrive_expect_tx(&full[s], w_bytes + a_bytes);
                    if constexpr (kPreA)
                        tc::bulk_copy_g2s(tc::smem_addr(smem + p.off_stage + s * p.stage_bytes),
                                          aexp + (tm * nblk + kb) * (a_bytes / 16), a_bytes, &full[s]);
                    tc::bulk_copy_g2s(tc::smem_addr(smem + p.off_stage + s * p.stage_bytes + w_off),
                                      wexp + (tn * nblk + kb) * (w_bytes / 16), w_bytes, &full[s]);
                }
            }
        }
    } else if (warp == 0) {
        // ------------------------------------------------------------ MMA issue (one thread)
        if (lane == 0) {
            const uint32_t idesc = tc::idesc_i8(128, (uint32_t)p.BN);
            const uint64_t desc_hi = (uint64_t)((128u >> 4) | (1u << 14)) << 32;
            const uint32_t a_lbo = (((uint32_t)rowsA * 16) >> 4) << 16, b_lbo = (((uint32_t)p.BN * 16) >> 4) << 16;
            const uint32_t stage16 = tc::smem_addr(smem + p.off_stage) >> 4;
            uint32_t count = 0, tc_ = 0;
            bool alive = true;
            for (int64_t tile = blockIdx.x; tile < p.tiles && alive; tile += gridDim.x, ++tc_) {
                const int acc = p.nAcc == 2 ? (tc_ & 1) : 0;
                const uint32_t acc_ph = p.nAcc == 2 ? ((tc_ >> 1) & 1) : (tc_ & 1);
                alive = wait_or_die(&acc_empty[acc], acc_ph ^ 1, g.status, dead);
                for (int64_t kb = 0; kb < nblk && alive; ++kb, ++count) {
                    const uint32_t s = count % (uint32_t)p.stages;
                    if (!wait_or_die(&full[s], (count / (uint32_t)p.stages) & 1, g.status, dead)) { alive = false; break; }
                    tc::tc_fence_after_sync();
                    if (kb == 0 && tc_ < 8) RTN_TL(gemm_i8, 40 + 2 * (int)tc_);
                    const uint32_t a16 = stage16 + s * (p.stage_bytes >> 4) + a_lbo;
                    const uint32_t b16 = stage16 + s * (p.stage_bytes >> 4) + (uint32_t)(rowsA * 8) + b_lbo;
                    uint32_t la[8], lb[4];
                    #pragma unroll
                    for (int j = 0; j < 4; ++j) {                       // K = 32 per MMA = chunks 2j, 2j+1
                        lb[j] = b16 + (uint32_t)(2 * j * p.BN);
                        la[2 * j] = a16 + (uint32_t)(2 * j * rowsA);
                        la[2 * j + 1] = la[2 * j] + 128;                // second 128-row sub-tile
                    }
                    #pragma unroll
                    for (int j = 0; j < 4; ++j) {
                        tc::mma_i8_ss(tmem + (uint32_t)(acc * p.TM * p.BN), desc_hi | la[2 * j], desc_hi | lb[j], idesc,
                                      kb > 0 || j > 0);
                        if (p.TM == 2)
                            tc::mma_i8_ss(tmem + (uint32_t)((acc * p.TM + 1) * p.BN), desc_hi | la[2 * j + 1],
                                          desc_hi | lb[j], idesc, kb > 0 || j > 0);
                    }
                    tc::mma_commit(&empty[s]);
                }
                if (alive) tc::mma_commit(&acc_full[acc]);
                if (tc_ < 8) RTN_TL(gemm_i8, 41 + 2 * (int)tc_);
            }
        }
    } else if (warp >= kEpiWarp0) {
        // ------------------------------------------------------------ epilogue
        //   out = a_s * (p1*S_xw + p2*S_x) + a_o * p3,  p1 = w_s, p2 = w_o, p3 = w_s*S_w + K*w_o
        // (kPreA: all sixteen warps from kEpiWarp0 on; else the eight epilogue warps, the rest being expanders)
        constexpr int nEpiThreads = kPreA ? kMaxEpiWarps * 32 : kEpiThreads;
        constexpr int nParts = nEpiThreads / 128;              // column ranges; the four warps of a range take 32 rows each
        const int q = warp & 3, part = (warp - kEpiWarp0) >> 2;
        const int etid = threadIdx.x - kEpiWarp0 * 32;
        uint8_t* sT = smem + p.off_t + (warp - kEpiWarp0) * kStageWarp;
        // whole-row float4 stores need every row start on a 16-byte boundary (the same for all lanes)
        const bool vec_ok = g.dbg_acc == nullptr && (g.N & 3) == 0 && (((uintptr_t)g.out) & 15) == 0;
        // TMA-store staging block of this warp (the first 8 or, with the expander warps free, 12 warps write out;
        // 1 KB aligned shared address)
        const uint32_t tma_stage = ((tc::smem_addr(smem + p.off_t) + 1023u) & ~1023u) + (uint32_t)(warp - kEpiWarp0) * kTmaStageWarp;
        const int parts_used = p.tma_out ? (kPreA ? kTmaWarpsPre : kEpiWarps) / 4 : nParts;
        uint32_t tc_ = 0;
        for (int64_t tile = blockIdx.x; tile < p.tiles; tile += gridDim.x, ++tc_) {
            const int acc = p.nAcc == 2 ? (tc_ & 1) : 0;
            const uint32_t acc_ph = p.nAcc == 2 ? ((tc_ >> 1) & 1) : (tc_ & 1);
            const int64_t m0 = (tile / p.tiles_n) * rowsA, n0 = (tile % p.tiles_n) * p.BN;
            // per-column constants of this tile, in double, rounded once (the previous tile's readers
            // are past them: same warps, program order + barrier)
            asm volatile("bar.sync %0, %1;" ::"r"(kEpiBarrier), "r"(nEpiThreads) : "memory");
            for (int j = etid; j < p.BN; j += nEpiThreads) {
                const int64_t n = n0 + j;
                float p1 = 0.f, p2 = 0.f, p3 = 0.f;
                if (n < g.N) {
                    const double ws = g.ep.w_scale[g.ep.n_wparam == 1 ? 0 : n];
                    const double wo = g.ep.w_offset[g.ep.n_wparam == 1 ? 0 : n];
                    p1 = (float)ws; p2 = (float)wo;
                    p3 = (float)(ws * (double)g.w_sum[n] + (double)g.K * wo);
                }
                sC[j] = make_float4(p1, p2, p3, 0.f);
            }
            asm volatile("bar.sync %0, %1;" ::"r"(kEpiBarrier), "r"(nEpiThreads) : "memory");
            const bool alive = wait_or_die(&acc_full[acc], acc_ph, g.status, dead);
            tc::tc_fence_after_sync();
            if (etid == 0 && tc_ < 8) RTN_TL(gemm_i8, 56 + 2 * (int)tc_);
            const int per = ((p.BN + parts_used - 1) / parts_used + 15) / 16 * 16;     // columns per range, whole blocks of 16
            const int c_begin = part * per < p.BN ? part * per : p.BN;
            const int c_end = c_begin + per < p.BN ? c_begin + per : p.BN;
            for (int tm = 0; tm < p.TM; ++tm) {
                const int64_t m = m0 + tm * 128 + q * 32 + lane;
                const bool row_ok = alive && m < g.M;
                float a_s = 0.f, a_o = 0.f, s_x = 0.f;
                if (row_ok) {
                    a_s = g.ep.a_scale[g.ep.n_aparam == 1 ? 0 : m];
                    a_o = g.ep.a_offset[g.ep.n_aparam == 1 ? 0 : m];
                    s_x = (float)g.a_sum[m];
                }
                const uint32_t trow = tmem + ((uint32_t)(q * 32) << 16) + (uint32_t)((acc * p.TM + tm) * p.BN);
                const int64_t mbase = m0 + tm * 128 + q * 32;
                // write-out of a staged block: lane -> rows rr and rr + 16, 16-byte chunk ch
                const int rr = (lane & 7) + 8 * (lane >> 4), ch = (lane >> 3) & 1;
                for (int c0 = c_begin; c0 < c_end; c0 += 16) {
                    uint32_t v[16];
                    tc::tmem_ld16(trow + (uint32_t)c0, v);
                    tc::tmem_ld_wait();
                    if (p.tma_out) {
                        // (uniform over the kernel) columns past N and rows past M are clipped by the copy engine
                        float r[kTmaCols];
                        #pragma unroll
                        for (int j = 0; j < kTmaCols; ++j) {
                            const float4 c = sC[c0 + j];
                            r[j] = fmaf(a_s, fmaf(c.x, (float)(int)v[j], c.y * s_x), a_o * c.z);
                        }
                        // the copy of the block before has read the staging block
                        if (lane == 0) asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory");
                        __syncwarp();
                        #pragma unroll
                        for (int ch = 0; ch < 4; ++ch) {
                            const uint32_t dst = tma_stage + (uint32_t)lane * 64u + (uint32_t)((ch ^ ((lane >> 1) & 3)) << 4);
                            asm volatile("st.shared.v4.f32 [%0], {%1, %2, %3, %4};"
                                         ::"r"(dst), "f"(r[4 * ch]), "f"(r[4 * ch + 1]), "f"(r[4 * ch + 2]), "f"(r[4 * ch + 3]) : "memory");
                        }
                        tc::fence_smem_to_async_proxy();
                        __syncwarp();
                        if (lane == 0 && alive && mbase < g.M && n0 + c0 < g.N) {
                            asm volatile("cp.async.bulk.tensor.2d.global.shared::cta.bulk_group [%0, {%1, %2}], [%3];"
                                         ::"l"(reinterpret_cast<uint64_t>(&omap)), "r"((int)(n0 + c0)), "r"((int)mbase), "r"(tma_stage)
                                         : "memory");
                            asm volatile("cp.async.bulk.commit_group;" ::: "memory");
                        }
                    } else
                    if (vec_ok && n0 + c0 + 16 <= g.N) {
                        // A lane holds 16 columns of ONE row; stored as is, a warp store would touch 32 rows
                        // with 16 bytes each.  Through the staging block (8 columns at a time) a store covers
                        // 16 rows x 32 bytes: whole sectors.
                        #pragma unroll
                        for (int h = 0; h < 16; h += 8) {
                            #pragma unroll
                            for (int j = 0; j < 8; j += 4) {
                                float r[4];
                                #pragma unroll
                                for (int e = 0; e < 4; ++e) {
                                    const float4 c = sC[c0 + h + j + e];
                                    r[e] = fmaf(a_s, fmaf(c.x, (float)(int)v[h + j + e], c.y * s_x), a_o * c.z);
                                }
                                *reinterpret_cast<float4*>(sT + lane * kStageRow + j * 4) = make_float4(r[0], r[1], r[2], r[3]);
                            }
                            __syncwarp();
                            #pragma unroll
                            for (int i = 0; i < 32; i += 16) {
                                const float4 t = *reinterpret_cast<const float4*>(sT + (rr + i) * kStageRow + ch * 16);
                                const int64_t mt = mbase + rr + i;
                                if (alive && mt < g.M)
                                    *reinterpret_cast<float4*>(g.out + mt * g.N + n0 + c0 + h + ch * 4) = t;
                            }
                            __syncwarp();
                        }
                    } else if (row_ok) {
                        float* orow = g.out + m * g.N + n0 + c0;
                        #pragma unroll
                        for (int j = 0; j < 16; ++j) {
                            if (n0 + c0 + j >= g.N) continue;
                            const float4 c = sC[c0 + j];
                            const int s_xw = (int)v[j];
                            orow[j] = fmaf(a_s, fmaf(c.x, (float)s_xw, c.y * s_x), a_o * c.z);
                            if (g.dbg_acc != nullptr) g.dbg_acc[m * g.N + n0 + c0 + j] = s_xw;
                        }
                    }
                }
            }
            tc::tc_fence_before_sync();
            tc::mbar_arrive(&acc_empty[acc]);
            if (etid == 0 && tc_ < 8) RTN_TL(gemm_i8, 57 + 2 * (int)tc_);
        }
        // the copies this thread handed over have written their rows before the CTA ends
        if (p.tma_out && lane == 0) asm volatile("cp.async.bulk.wait_group 0;" ::: "memory");
    }
    tc::tc_fence_before_sync();
    __syncthreads();
    if (warp == 0) tc::tmem_dealloc(tmem, p.tmem_cols);
    if (threadIdx.x == 0) RTN_TL(gemm_i8, 4);
}

// Pre-expansion mode of a plan: 0 = both operands expanded inside the kernel (one row tile: every weight row
// is expanded once anyway), 1 = weights expanded ahead (several row tiles, one column tile), 2 = both ahead
// (several tiles each way: every row of either operand would be expanded once per tile it takes part in).
int gemm_pre_mode(const GemmI8Plan& p, int64_t K)
{
    const int64_t nblk = (K + kBlockCodes - 1) / kBlockCodes;
    const size_t wbytes = (size_t)p.tiles_n * nblk * p.BN * 128, abytes = (size_t)p.tiles_m * nblk * p.TM * 128 * 128;
    if (p.tiles_m < 2 || wbytes > (size_t(1) << 31)) return 0;
    if (p.tiles_n < 2 || wbytes + abytes > (size_t(1) << 31)) return 1;
    return 2;
}

}  // namespace

bool gemm_i8_supported(int64_t M, int64_t N, int64_t K)
{
    GemmI8Plan p;
    return make_gemm_plan(M, N, K, p, device_sm_count());
}

int gemm_i8_launches(int64_t M, int64_t N, int64_t K)
{
    GemmI8Plan p;
    if (!make_gemm_plan(M, N, K, p, device_sm_count())) return 0;
    return gemm_pre_mode(p, K) == 0 ? 1 : 2;
}

cudaError_t launch_gemm_i8(const GemmArgs& g, cudaStream_t s)
{
    GemmI8Plan p;
    if (!make_gemm_plan(g.M, g.N, g.K, p, device_sm_count())) return cudaErrorInvalidConfiguration;
    const int mode = gemm_pre_mode(p, g.K);
    // Output as a 2-D tensor for the epilogue's TMA stores: rows of N floats, boxes of 32 rows x 16 columns,
    // 64-byte swizzle.  Needs 16-byte aligned rows; the debug output keeps the store-instruction epilogue.
    CUtensorMap omap;
    memset(&omap, 0, sizeof(omap));
    if (g.dbg_acc == nullptr && (g.N & 3) == 0 && g.N >= kTmaCols && (reinterpret_cast<uintptr_t>(g.out) & 15) == 0) {
        EncodeTiledFn enc = encode_tiled_fn();
        const cuuint64_t dims[2] = {(cuuint64_t)g.N, (cuuint64_t)g.M};
        const cuuint64_t strides[1] = {(cuuint64_t)g.N * 4};
        const cuuint32_t box[2] = {(cuuint32_t)kTmaCols, 32};
        const cuuint32_t estr[2] = {1, 1};
        if (enc != nullptr &&
            enc(&omap, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 2, g.out, dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
                CU_TENSOR_MAP_SWIZZLE_64B, CU_TENSOR_MAP_L2_PROMOTION_NONE, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS)
            p.tma_out = 1;
    }
    if (mode == 0) {
        cudaError_t e = cudaFuncSetAttribute(gemm_i8_kernel<false, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)p.smem_bytes);
        if (e != cudaSuccess) return e;
        gemm_i8_kernel<false, false><<<(unsigned)p.grid, kThreads, p.smem_bytes, s>>>(g, p, nullptr, nullptr, omap);
        return cudaGetLastError();
    }
    // scratch from the stream-ordered allocator: N (and M) rounded up to tiles, times K rounded up to blocks, bytes
    const int64_t nblk = (g.K + kBlockCodes - 1) / kBlockCodes;
    const int64_t items_w = p.tiles_n * nblk * p.BN, items_a = mode == 2 ? p.tiles_m * nblk * p.TM * 128 : 0;
    void* scratch = nullptr;
    cudaError_t e = cudaMallocAsync(&scratch, (size_t)(items_w + items_a) * 128, s);
    if (e != cudaSuccess) return e;
    uint4* wexp = reinterpret_cast<uint4*>(scratch);
    uint4* aexp = mode == 2 ? wexp + items_w * 8 : nullptr;
    gemm_expand_operands_kernel<<<(unsigned)((items_w + items_a + 255) / 256), 256, 0, s>>>(g, p, wexp, aexp);
    e = cudaGetLastError();
    if (e == cudaSuccess && mode == 1) {
        e = cudaFuncSetAttribute(gemm_i8_kernel<true, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)p.smem_bytes);
        if (e == cudaSuccess)
            e = launch_pdl(gemm_i8_kernel<true, false>, dim3((unsigned)p.grid), dim3(kThreads), p.smem_bytes, s, g, p,
                           (const uint4*)wexp, (const uint4*)aexp, omap);
    } else if (e == cudaSuccess) {
        e = cudaFuncSetAttribute(gemm_i8_kernel<true, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)p.smem_bytes);
        if (e == cudaSuccess)
            e = launch_pdl(gemm_i8_kernel<true, true>, dim3((unsigned)p.grid), dim3(kThreads), p.smem_bytes, s, g, p,
                           (const uint4*)wexp, (const uint4*)aexp, omap);
    }
    const cudaError_t e2 = cudaFreeAsync(scratch, s);
    return e != cudaSuccess ? e : e2;
}

}  // namespace rtn
