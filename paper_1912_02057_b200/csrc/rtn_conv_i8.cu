// Ternary conv2d (stride 1), tensor-core variant: fp32 NCHW input ternarized in-kernel (Eq. 3)
// straight to int8 {-1,0,+1} in shared memory, filters expanded once per CTA from their bit
// planes to int8 in shared memory, tcgen05.mma kind::i8 into int32 accumulators in tensor memory,
// affine epilogue (Eq. 10 with a weight offset) fused.
//
// Implicit GEMM without im2col, by a shift.  Lay the zero-padded images of the batch out as one
// long sequence of padded rows G = b*PH + r (PH = H + 2 pad) of PW = W + 2 pad pixels each.  The
// output whose top-left tap sits at padded pixel Q = G*PW + c reads, for tap (i, j), padded pixel
// Q + i*PW + j.  For a run of consecutive Q the A operand of tap (i, j) is therefore the SAME
// shared-memory code array read from a start address shifted by (i*PW + j) pixels.  Outputs whose
// Q falls in the padding (c >= Wo or r >= Ho) are computed and dropped.
//
// Shared-memory code array: [channel chunk of 16][padded pixel][16 bytes] -- K-major, no swizzle:
// an 8-pixel x 16-channel core matrix is 128 contiguous bytes wherever the window starts.
// Filters: [tap][channel chunk][n][16 bytes].  Within a group of 32 channels both operands use
// the byte order of tc::unpack32.  One extra filter row of all +1 makes the tensor core produce
// the activation code sum S_x of every output pixel in accumulator column N.
//
// Work split: each CTA (one per SM, persistent) owns a contiguous strip of padded rows and walks
// it in tiles of RT rows (RT*PW <= TM*128 accumulator lanes).  A tile needs RT + kh - 1 rows of
// codes; the kh - 1 rows it shares with the previous tile are copied inside shared memory, so
// every input value is fetched and ternarized once per strip.
//
// Warp roles, pipelined through mbarriers (two code buffers, two accumulator buffers, a ring of
// input stages):
//   warp  0       one thread issues the MMAs of tile i and commits them
//   warp  1       producer: one thread streams the new fp32 rows of tile i+1.. into the stage ring
//                 with TMA (one box = 32 channels x one image row), ahead of the converters
//   warps 4..11   epilogue: tcgen05.ld the accumulators of tile i-1, affine form, store fp32
//   warps 2, 3, 12..17  converters: read a stage, ternarize, write the code array of tile i
// When the input cannot be described to TMA (W not a multiple of 4, unaligned base) the converters
// load the fp32 values themselves.  With packed pixel rows as input (hand-over from the layer before) there is
// no stage ring; in a layer that also adds a skip connection the producer warp then stages each tile's skip
// values in shared memory by TMA, a tile ahead of the epilogue that adds them (conv_i8_kernel<true, true>).
#include "rtn_internal.cuh"
#include "rtn_tcgen05.cuh"
#include "rtn_conv_i8_common.cuh"
#include "rtn_timeline.cuh"
#include "rtn_tensormap.cuh"

#include <cuda.h>
#include <string.h>

// Timeline slots (instrumented build only): 0 kernel entry, 1 set-up done, 2 filters expanded, 3 epilogue constants
// ready, 4 kernel end; per tile i < 8: 8+2i / 9+2i producer issues first / last batch, 24+2i / 25+2i converters begin /
// end, 40+2i / 41+2i first MMA can issue / commit, 56+2i / 57+2i epilogue begins / ends; per tile i < 6 and channel group
// j < 2: 72+4i+2j the group's staged rows have landed, 73+4i+2j converter thread 0 has converted its share.
RTN_TL_DEFINE(conv_i8)

namespace rtn {

namespace {

using namespace conv_detail;

constexpr int kMmaWarp = 0;
constexpr int kProdWarp = 1;
constexpr int kEpiWarp0 = 4;                           // first epilogue warp (multiple of 4)
constexpr int kEpiWarps = 8;                           // two per TMEM lane quarter
constexpr int kEpiThreads = kEpiWarps * 32;
constexpr int kConvWarps = 8;                          // warps 2, 3 and 12..17
constexpr int kConvThreads = kConvWarps * 32;
constexpr int kWarps = kEpiWarp0 + kEpiWarps + kConvWarps - 2;
constexpr int kThreads = kWarps * 32;
__device__ __forceinline__ bool is_conv_warp(int w) { return w == 2 || w == 3 || w >= kEpiWarp0 + kEpiWarps; }
__device__ __forceinline__ int conv_warp_index(int w) { return w < 4 ? w - 2 : w - (kEpiWarp0 + kEpiWarps) + 2; }
constexpr int kMaxStages = 8;                         // input batches (one tile's rows of 32 channels) in flight
constexpr int kMaxGroups = 16;                          // groups of 32 input channels (C <= 512)
constexpr int kMaxMma = 160;                           // MMAs per sub-tile the descriptor table holds
constexpr int kMaxSlots = 32;                          // row slots of a tile (rows + halo rows)
constexpr int kRowwiseMinPW = 24;                      // padded width from which a warp per staged image row pays
constexpr int kTileM = 128;                            // pixels per MMA (TMEM lanes)
constexpr size_t kSmemLimit = 220 * 1024;
constexpr int kConvBarrier = 1;                        // named barrier of the converter warps
constexpr int kEpiBarrier = 2;                         // named barrier of the epilogue warps

struct ConvI8Plan {
    int PW, PH;            // padded image extent
    int Cp;                // channels rounded up to 32
    int Np;                // accumulator columns: N outputs + the all-ones row, rounded up to 16
    int T;                 // taps
    int TM;                // 128-pixel sub-tiles per tile
    int RT;                // padded rows per tile
    int R0;                // padded rows of a strip's first tile (<= RT)
    int halo;              // kh - 1 rows shared with the next tile
    int ppix;              // pixels allocated per code buffer
    int strip;             // one code buffer holds the CTA's whole strip (no double buffering, no halo copies)
    int total_rows;        // B*PH
    int grid;              // CTAs = strips
    uint32_t tmem_cols;
    int const_tmem;        // epilogue constants replicated in tensor memory (columns cbase..), not read from smem
    uint32_t cbase, Nc;    // first constant column; columns per constant = N rounded up to 16
    FastDiv div_pw, div_ph;
    FastDiv div_np, div_cw;    // by Np and by Cp/32 (filter expansion)
    int n_mma;             // MMAs per sub-tile: taps * groups of 32 channels
    int use_tma;           // input rows staged by TMA (else loaded by the converters)
    int stages;            // depth of the staging ring
    uint32_t box_bytes;    // one TMA box: 32 channels x one image row of fp32
    int nslots;            // row slots of the TMA ring
    uint32_t off_stage;
    int sk_stage;          // the skip connection's values of a tile are staged in shared memory by TMA (set by the launcher)
    int sk_groups;         // 32-channel groups of the output (boxes per row)
    uint32_t off_skip, sk_box;     // two buffers of RT rows x sk_groups boxes of sk_box bytes (32 channels x one output row)
    uint32_t off_a[2], off_w, off_lo, off_hi, off_c, off_t, off_rows, off_bar, off_misc;
    size_t smem_bytes;
    // Per MMA of a sub-tile (tap t, channel group h), in 16-byte units: start of the A window
    // relative to the code buffer, start of the filter slice relative to the filter array.
    uint32_t tab_a[kMaxMma], tab_b[kMaxMma];
};

bool make_plan(const ConvArgs& c, ConvI8Plan& p, int sms, bool next = false)
{
    if (c.stride != 1) return false;
    if (c.Ho <= 0 || c.Wo <= 0) return false;
    p.PW = c.W + 2 * c.pad;
    p.PH = c.H + 2 * c.pad;
    if (p.PW > 256 || p.PH > 2048) return false;
    p.Cp = (c.C + 31) / 32 * 32;
    p.Np = (c.N + 1 + 15) / 16 * 16;
    p.T = c.kh * c.kw;
    p.halo = c.kh - 1;
    if (p.Np > 256) return false;
    if (p.Cp / 32 > kMaxGroups) return false;
    if ((int64_t)c.B * p.PH > (1 << 20)) return false;                // fast division ranges
    p.total_rows = c.B * p.PH;
    // two sub-tiles when the accumulators fit twice (double buffered) and there is enough work
    p.TM = (4 * p.Np <= 512 && (int64_t)p.total_rows * p.PW >= (int64_t)4 * sms * kTileM) ? 2 : 1;
    if (2 * p.TM * p.Np > 512) return false;
    p.RT = p.TM * kTileM / p.PW;
    if (p.RT > kMaxSlots - p.halo) p.RT = kMaxSlots - p.halo;
    if (p.RT < 1) return false;
    // A CTA's first tile is half as tall when its strip has several tiles: the tensor core and the
    // epilogue then start after half the input, and (the strip length permitting) the last tile,
    // whose epilogue nothing overlaps, is short as well.
    p.R0 = (p.RT >= 2 && (int64_t)p.total_rows >= (int64_t)2 * p.RT * sms) ? p.RT / 2 : p.RT;
#ifdef RTN_KNOB_R0
    if (p.R0 > RTN_KNOB_R0) p.R0 = RTN_KNOB_R0;
#endif
    p.ppix = (p.TM * kTileM + p.halo * p.PW + (c.kw - 1) + 7) / 8 * 8;
    const int tiles = (p.total_rows + p.RT - 1) / p.RT;
    p.grid = tiles < sms ? tiles : sms;
    // Short strips (small batches): the codes of a CTA's whole strip fit in shared memory at one byte per value.
    // The converters then run ahead of the tensor core as fast as the input arrives (nothing waits for a code
    // buffer to be free, no halo rows are copied), which takes the input stream off the critical path.
    const int strip_rows = (p.total_rows + p.grid - 1) / p.grid;
    const int strip_tiles = strip_rows <= p.R0 ? 1 : 1 + (strip_rows - p.R0 + p.RT - 1) / p.RT;
    const int strip_ppix = ((strip_rows - 1 + p.halo) * p.PW + p.TM * kTileM + (c.kw - 1) + 7) / 8 * 8;
    // (room must remain for the filters and for a staging ring of two tiles' rows)
    const int64_t strip_need = (int64_t)strip_ppix * p.Cp + (int64_t)p.T * p.Cp * p.Np +
                               (int64_t)2 * (p.RT + p.halo) * 32 * c.W * 4 + 8192;
    p.strip = (strip_tiles >= 2 && strip_tiles * (p.Cp / 32) <= 2 * kMaxGroups &&
               strip_need <= (int64_t)kSmemLimit) ? 1 : 0;
    if (p.strip) p.ppix = strip_ppix;
    p.Nc = (uint32_t)((c.N + 15) / 16 * 16);
    p.cbase = (uint32_t)(2 * p.TM * p.Np);
    p.const_tmem = (p.cbase + 3 * p.Nc <= 512) ? 1 : 0;
    uint32_t cols = 32;
    while (cols < p.cbase + (p.const_tmem ? 3 * p.Nc : 0)) cols *= 2;
    p.tmem_cols = cols;
    p.div_pw = make_fastdiv((uint32_t)p.PW);
    p.div_ph = make_fastdiv((uint32_t)p.PH);
    p.div_np = make_fastdiv((uint32_t)p.Np);
    p.div_cw = make_fastdiv((uint32_t)(p.Cp / 32));
    p.n_mma = p.T * (p.Cp / 32);
    if (p.n_mma > kMaxMma) return false;
    for (int i = 0; i < p.n_mma; ++i) {
        const int h = i / p.T, t = i % p.T;              // channel group outer, tap inner
        p.tab_a[i] = (uint32_t)(2 * h) * p.ppix + (uint32_t)((t / c.kw) * p.PW + (t % c.kw));
        p.tab_b[i] = (uint32_t)((t * (p.Cp / 16) + 2 * h) * p.Np);
    }
    uint32_t o = 0;
    const uint32_t a_bytes = (uint32_t)(p.Cp / 16) * p.ppix * 16;
    p.off_a[0] = o; o += a_bytes;
    p.off_a[1] = p.strip ? p.off_a[0] : o; o += p.strip ? 0 : a_bytes;
    p.off_w = o;    o += (uint32_t)p.T * (p.Cp / 16) * p.Np * 16;
    p.off_lo = o;   o += (uint32_t)p.Cp * 4;
    p.off_hi = o;   o += (uint32_t)p.Cp * 4;
    o = (o + 15) / 16 * 16;
    p.off_c = o;    o += (uint32_t)p.Np * 16;           // float4 {c1, c2, c3, 0} per column
    p.off_t = o;    o += next ? (uint32_t)p.Np * 8 : 0; // float2 {t_lo, t_hi} of the next layer per column
    p.off_rows = o; o += kMaxSlots * 4;                 // producer's row table
    p.off_bar = o;  o += (7 + 2 * kMaxStages + 2 * kMaxGroups) * 8;   // a_empty[2] acc_full[2] acc_empty[2] st_full[] st_empty[] a_full[2][groups]
    p.off_misc = o; o += 16;                            // tmem slot, dead flag
    if (o > kSmemLimit) return false;
    // staging ring for TMA
    p.use_tma = 0; p.stages = 0; p.nslots = 0; p.off_stage = o;
    p.sk_stage = 0; p.sk_groups = 0; p.off_skip = 0; p.sk_box = 0;
    p.box_bytes = 32u * (uint32_t)c.W * 4u;
    const bool tma_ok = (c.W % 4 == 0) && (reinterpret_cast<uintptr_t>(c.x) % 16 == 0);
    if (tma_ok) {
        const uint32_t base = (o + 127) / 128 * 128;
        // A ring of row slots (one TMA box each); a batch takes as many as the tile has new rows.  Two
        // steady-state batches in flight measured fastest (a deeper ring lost 3 %), so the ring is
        // capped at two tiles' worth of new rows.
        int ns = base < kSmemLimit ? (int)((kSmemLimit - base) / p.box_bytes) : 0;
        // (with the whole strip's codes resident the converters free a slot as soon as it lands: the ring is
        // then as deep as shared memory allows, which is what keeps enough bytes in flight from the start)
        const int cap = p.strip ? kMaxSlots * 2 : 2 * p.RT > p.RT + p.halo ? 2 * p.RT : p.RT + p.halo;
        if (ns > cap) ns = cap;
        if (ns >= p.RT + p.halo) {
            p.use_tma = 1; p.stages = kMaxStages; p.nslots = ns; p.off_stage = base;
            o = base + (uint32_t)ns * p.box_bytes;
        }
    }
    p.smem_bytes = o;
    return true;
}

// One warp of a role waits on the mbarrier; the role's other warps sleep on a hardware named
// barrier until it gets there (a polling warp costs issue slots, a warp parked on bar.sync none).
__device__ __forceinline__ void role_wait(bool leader, uint64_t* bar, uint32_t parity, unsigned* status,
                                          volatile int* dead, int barrier_id, int nthreads)
{
    if (leader) wait_or_die(bar, parity, status, dead);
    asm volatile("bar.sync %0, %1;" ::"r"(barrier_id), "r"(nthreads) : "memory");
}

// TMA: one box {W, 1, 32, 1} of the fp32 tensor viewed as (W, H, C, B) -> shared memory
// [32 channels][W]; completion is counted in bytes on `bar`.  Channels outside the tensor read as
// zero.  No multicast.
__device__ __forceinline__ void tma_load_row(uint32_t dst, const CUtensorMap* map, int r, int c0, int b,
                                             uint32_t bar)
{
    asm volatile(
        "cp.async.bulk.tensor.4d.shared::cluster.global.tile.mbarrier::complete_tx::bytes "
        "[%0], [%1, {%2, %3, %4, %5}], [%6];"
        ::"r"(dst), "l"(reinterpret_cast<uint64_t>(map)), "r"(0), "r"(r), "r"(c0), "r"(b), "r"(bar)
        : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint64_t* bar, uint32_t bytes)
{
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;"
                 ::"r"(tc::smem_addr(bar)), "r"(bytes) : "memory");
}

// Issues NB MMAs whose descriptor low words are first gathered into registers: nothing but the
// tcgen05.mma instructions then sits in the issue stream (loads left between MMAs would be
// ordered after them by the asm's memory clobber and stall the single issuing thread).
template <int NB>
__device__ __forceinline__ void issue_mmas(const ConvI8Plan& p, int i0, uint32_t d, uint32_t a_tm,
                                           uint32_t w16, uint64_t desc_hi, uint32_t idesc)
{
    uint32_t la[NB], lb[NB];
    #pragma unroll
    for (int j = 0; j < NB; ++j) { la[j] = a_tm + p.tab_a[i0 + j]; lb[j] = w16 + p.tab_b[i0 + j]; }
    tc::mma_i8_ss(d, desc_hi | la[0], desc_hi | lb[0], idesc, i0 > 0);
    #pragma unroll
    for (int j = 1; j < NB; ++j) tc::mma_i8_ss_acc(d, desc_hi | la[j], desc_hi | lb[j], idesc);
}

// Hand-over epilogue (NextLayerArgs) of one tile for one warp.  The warp reads TMEM lanes 32 q .. 32 q + 31
// (pixels) and is warp `part` of the `nparts` (2 or 4) that share this lane quarter.  Unit of work = (sub-tile,
// block of 128 output channels), dealt to those warps in turn: a thread then holds all 128 codes of its pixel and
// writes each bit plane of the packed row with one 16-byte store.  Constants and the next layer's thresholds come
// from shared memory.
template <bool kSk>
__device__ __forceinline__ void next_epilogue_tile(const ConvArgs& a, const ConvI8Plan& p, const NextLayerArgs& f,
                                                   const float4* sC, const float2* sT, uint32_t tmem, int buf, int g,
                                                   int nrows, bool alive, int q, int lane, int part, int nparts,
                                                   const float* sk_buf)
{
    const int ntm = (nrows * p.PW + kTileM - 1) / kTileM;
    const int64_t ostride = (int64_t)a.Ho * a.Wo;
    const int nblk16 = (a.N + 15) / 16;
    const int ncb = (a.N + kBlockCodes - 1) / kBlockCodes;
    const int nwords = a.N / 32;
    if (a.pad_mode == RTN_PAD_CODE_ZERO && (a.N == 64 || a.N == 128)) {
        // A 64- or 128-filter layer without border classes: the warps of a lane quarter split the output
        // channels, and a thread takes its pixel of BOTH sub-tiles (of the one, where the tile has one: the second
        // pixel then does not exist and nothing is read or written for it) through its channels, 16 at a time
        // (next_layer_block16_pair).  A warp writes its 32- or 16-bit pieces of each pixel's packed row; the words
        // past N of a 64-filter row (its zero fill) are shared out between the warps.
        bool ok2[2];
        uint32_t trow2[2];
        int64_t obase2[2];
        uint8_t* row2[2];
        uint32_t sx2[2];
        const float* sk2[2];                        // the pixel's staged skip values: channel n at sk2[t][skip_index(n)]
        #pragma unroll
        for (int t = 0; t < 2; ++t) {
            const uint32_t pl = (uint32_t)(t * kTileM + q * 32 + lane);
            const uint32_t row = fdiv(pl, p.div_pw);
            const int wo = (int)(pl - row * (uint32_t)p.PW);
            const uint32_t G = (uint32_t)g + row;
            const uint32_t b = fdiv(G, p.div_ph);
            const int ho = (int)(G - b * (uint32_t)p.PH);
            ok2[t] = alive && t < ntm && (int)row < nrows && b < (uint32_t)a.B && ho < a.Ho && wo < a.Wo;
            trow2[t] = tmem + ((uint32_t)(q * 32) << 16) + (uint32_t)((buf * p.TM + (t < ntm ? t : 0)) * p.Np);
            obase2[t] = (((int64_t)b * a.N) * a.Ho + ho) * a.Wo + wo;
            // staged as [row of the tile][32-channel group][channel][Wo]
            sk2[t] = kSk ? sk_buf + (size_t)row * p.sk_groups * (p.sk_box / 4) + wo : nullptr;
            row2[t] = (ok2[t] && f.out_packed != nullptr)
                          ? f.out_packed + (((int64_t)b * a.Ho + ho) * a.Wo + wo) * (int64_t)(ncb * kBlockBytes) : nullptr;
            asm volatile("tcgen05.ld.sync.aligned.32x32b.x1.b32 {%0}, [%1];"
                         : "=r"(sx2[t]) : "r"(trow2[t] + (uint32_t)a.N) : "memory");
        }
        tc::tmem_ld_wait();
        const float fsx0 = (float)(int)sx2[0], fsx1 = (float)(int)sx2[1];
        const bool want = f.out_packed != nullptr;
        const int nb = nblk16 / nparts;                              // 16-channel blocks of this warp: 1, 2 or 4
        uint32_t nz0 = 0, sg0 = 0, nz1 = 0, sg1 = 0;
        #pragma unroll 1
        for (int k = part * nb; k < (part + 1) * nb; ++k) {
            const int n0 = k * 16;
            uint32_t u0[16], u1[16];
            tc::tmem_ld16(trow2[0] + (uint32_t)n0, u0);
            tc::tmem_ld16(trow2[1] + (uint32_t)n0, u1);
            tc::tmem_ld_wait();
            uint32_t a0, b0, a1, b1;
            // (channel n0 + j of the staging buffer: group n0 / 32, channel n0 % 32 + j of the group, a.Wo floats apart)
            const int sk_off = ((n0 >> 5) * 32 + (n0 & 31)) * a.Wo;
            next_layer_block16_pair<kSk>(a, f, u0, u1, sC + n0, sT + n0, fsx0, fsx1, ok2[0], ok2[1],
                                         obase2[0] + (int64_t)n0 * ostride, obase2[1] + (int64_t)n0 * ostride, ostride, want,
                                         a0, b0, a1, b1, kSk ? sk2[0] + sk_off : nullptr, kSk ? sk2[1] + sk_off : nullptr,
                                         a.Wo);
            const int off = (k >> 3) * kBlockBytes + ((k >> 1) & 3) * 4;      // the block's word in the packed row
            if (nb == 1) {
                // a lone block is half a word: 16-bit stores
                if (row2[0] != nullptr) {
                    *reinterpret_cast<uint16_t*>(row2[0] + off + 2 * (k & 1)) = (uint16_t)a0;
                    *reinterpret_cast<uint16_t*>(row2[0] + off + 16 + 2 * (k & 1)) = (uint16_t)b0;
                }
                if (row2[1] != nullptr) {
                    *reinterpret_cast<uint16_t*>(row2[1] + off + 2 * (k & 1)) = (uint16_t)a1;
                    *reinterpret_cast<uint16_t*>(row2[1] + off + 16 + 2 * (k & 1)) = (uint16_t)b1;
                }
                continue;
            }
            // (nb is even and the warp's first block is even: blocks come in whole words)
            nz0 |= a0 << (16 * (k & 1)); sg0 |= b0 << (16 * (k & 1));
            nz1 |= a1 << (16 * (k & 1)); sg1 |= b1 << (16 * (k & 1));
            if (k & 1) {
                if (row2[0] != nullptr) {
                    *reinterpret_cast<uint32_t*>(row2[0] + off) = nz0;
                    *reinterpret_cast<uint32_t*>(row2[0] + off + 16) = sg0;
                }
                if (row2[1] != nullptr) {
                    *reinterpret_cast<uint32_t*>(row2[1] + off) = nz1;
                    *reinterpret_cast<uint32_t*>(row2[1] + off + 16) = sg1;
                }
                nz0 = sg0 = nz1 = sg1 = 0;
            }
        }
        for (int w = nwords + part; w < ncb * 4; w += nparts) {          // zero fill past N
            const int off = (w >> 2) * kBlockBytes + (w & 3) * 4;
            #pragma unroll
            for (int t = 0; t < 2; ++t)
                if (row2[t] != nullptr) {
                    *reinterpret_cast<uint32_t*>(row2[t] + off) = 0u;
                    *reinterpret_cast<uint32_t*>(row2[t] + off + 16) = 0u;
                }
        }
        return;
    }
    for (int tm = 0; tm < ntm; ++tm) {
        const uint32_t pl = (uint32_t)(tm * kTileM + q * 32 + lane);     // pixel within the tile
        const uint32_t row = fdiv(pl, p.div_pw);
        const int wo = (int)(pl - row * (uint32_t)p.PW);
        const uint32_t G = (uint32_t)g + row;
        const uint32_t b = fdiv(G, p.div_ph);
        const int ho = (int)(G - b * (uint32_t)p.PH);
        const bool ok = alive && (int)row < nrows && b < (uint32_t)a.B && ho < a.Ho && wo < a.Wo;
        int n_inside = p.T;
        if (ok && a.pad_mode == RTN_PAD_VALUE_ZERO) {
            n_inside = 0;
            for (int t = 0; t < p.T; ++t) {
                const int h = ho - a.pad + t / a.kw, v = wo - a.pad + t % a.kw;
                n_inside += (h >= 0 && h < a.H && v >= 0 && v < a.W);
            }
        }
        const bool border = n_inside < p.T;
        const uint32_t trow = tmem + ((uint32_t)(q * 32) << 16) + (uint32_t)((buf * p.TM + tm) * p.Np);
        const int64_t obase = (((int64_t)b * a.N) * a.Ho + ho) * a.Wo + wo;
        uint8_t* out_row = nullptr;
        if (ok && f.out_packed != nullptr)
            out_row = f.out_packed + (((int64_t)b * a.Ho + ho) * a.Wo + wo) * (int64_t)(ncb * kBlockBytes);
        // S_x of this pixel: accumulator column N (the all-ones filter row)
        uint32_t sx_raw;
        asm volatile("tcgen05.ld.sync.aligned.32x32b.x1.b32 {%0}, [%1];"
                     : "=r"(sx_raw) : "r"(trow + (uint32_t)a.N) : "memory");
        bool sx_ready = false;
        float fsx = 0.f;
        for (int cb = 0; cb < ncb; ++cb) {
            if ((tm * ncb + cb) % nparts != part) continue;
            uint32_t nzw[4] = {0u, 0u, 0u, 0u}, sgw[4] = {0u, 0u, 0u, 0u};
            #pragma unroll 1
            for (int k = 0; k < 8; ++k) {
                const int n0 = cb * kBlockCodes + k * 16;
                if (n0 >= nblk16 * 16) break;
                uint32_t u[16];
                tc::tmem_ld16(trow + (uint32_t)n0, u);
                tc::tmem_ld_wait();
                if (!sx_ready) { fsx = (float)(int)sx_raw; sx_ready = true; }
                if (!ok) continue;
                uint32_t nzb, sgb;
                next_layer_block16(a, f, u, sC + n0, sT + n0, fsx, border, p.T, ho, wo, n_inside, n0,
                                   obase + (int64_t)n0 * ostride, ostride, out_row != nullptr, nzb, sgb);
                nzb <<= 16 * (k & 1);
                sgb <<= 16 * (k & 1);
                #pragma unroll
                for (int w = 0; w < 4; ++w) {               // word k/2, without indexing the registers
                    nzw[w] |= (k >> 1) == w ? nzb : 0u;
                    sgw[w] |= (k >> 1) == w ? sgb : 0u;
                }
            }
            if (out_row != nullptr) {                       // codes past N are the row's zero fill
                uint4* dst = reinterpret_cast<uint4*>(out_row + cb * kBlockBytes);
                dst[0] = make_uint4(nzw[0], nzw[1], nzw[2], nzw[3]);
                dst[1] = make_uint4(sgw[0], sgw[1], sgw[2], sgw[3]);
            }
        }
        if (!sx_ready) tc::tmem_ld_wait();              // the S_x load still has to land
    }
}

// kNext: the layer hands its result to the next one (NextLayerArgs): the input may come as packed pixel
// rows (the converters then expand bit planes instead of ternarizing fp32), and the epilogue applies
// phi, adds the skip connection and writes fp32 and / or packed Eq. 3 codes.
// kSk (only with kNext, packed input and a skip connection): the producer warp stages each tile's skip values in
// shared memory by TMA (ConvI8Plan::sk_stage), and the epilogue reads them from there.
template <bool kNext, bool kSk = false>
__global__ void __launch_bounds__(kThreads, 1)
conv_i8_kernel(const ConvArgs a, const __grid_constant__ ConvI8Plan p, const __grid_constant__ CUtensorMap tmap,
               const NextLayerArgs f)
{
    extern __shared__ __align__(128) uint8_t smem[];
    uint4* sW = reinterpret_cast<uint4*>(smem + p.off_w);        // [T][Cp/16][Np]
    float* sLo = reinterpret_cast<float*>(smem + p.off_lo);
    float* sHi = reinterpret_cast<float*>(smem + p.off_hi);
    float4* sC = reinterpret_cast<float4*>(smem + p.off_c);     // {c1, c2, c3, 0} per column
    uint32_t* sRows = reinterpret_cast<uint32_t*>(smem + p.off_rows);
    uint64_t* bars = reinterpret_cast<uint64_t*>(smem + p.off_bar);
    uint64_t* a_empty = bars;           // [2] MMA -> converters: MMAs that read the buffer are done
    uint64_t* acc_full = bars + 2;      // [2] MMA -> epilogue: accumulators complete
    uint64_t* acc_empty = bars + 4;     // [2] epilogue -> MMA: accumulators read out
    uint64_t* st_full = bars + 6;                   // [stages] TMA -> converters: stage landed
    uint64_t* st_empty = bars + 6 + kMaxStages;     // [stages] converters -> producer: stage read
    uint64_t* a_full = bars + 6 + 2 * kMaxStages;   // [2][kMaxGroups] converters -> MMA: 32 channels of codes written
    uint64_t* w_ready = bars + 6 + 2 * kMaxStages + 2 * kMaxGroups;     // epilogue warps -> MMA: filters expanded
    uint32_t* slot = reinterpret_cast<uint32_t*>(smem + p.off_misc);
    volatile int* dead = reinterpret_cast<volatile int*>(smem + p.off_misc + 8);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int nchunk = p.Cp / 16;
    // this CTA's strip of padded rows
    const int s0 = (int)((int64_t)blockIdx.x * p.total_rows / p.grid);
    const int s1 = (int)((int64_t)(blockIdx.x + 1) * p.total_rows / p.grid);

    // ---------------------------------------------------------------- set-up (all threads)
    RTN_TL_INIT(conv_i8)
    if (threadIdx.x == 0) RTN_TL(conv_i8, 0);
    tc::pdl_trigger();
    if (warp == 0) tc::tmem_alloc(slot, p.tmem_cols);
    if (threadIdx.x == 32) {
        for (int i = 0; i < 2 * kMaxGroups; ++i) tc::mbar_init(&a_full[i], kConvThreads);
        tc::mbar_init(w_ready, kEpiThreads);
        tc::mbar_init(&a_empty[0], 1);
        tc::mbar_init(&a_empty[1], 1);
        tc::mbar_init(&acc_full[0], 1);
        tc::mbar_init(&acc_full[1], 1);
        tc::mbar_init(&acc_empty[0], kEpiThreads);
        tc::mbar_init(&acc_empty[1], kEpiThreads);
        for (int i = 0; i < kMaxStages; ++i) {
            tc::mbar_init(&st_full[i], 1);
            // (staged skip values: slots 0, 1 = the two tile buffers, released by the epilogue's threads)
            tc::mbar_init(&st_empty[i], kSk ? kEpiThreads : kConvThreads);
        }
        tc::mbar_init_fence();
        *dead = 0;
    }
    tc::tc_fence_before_sync();
    __syncthreads();
    tc::tc_fence_after_sync();
    const uint32_t tmem = *slot;
    if (threadIdx.x == 0) RTN_TL(conv_i8, 1);

    if (is_conv_warp(warp)) {
        // ------------------------------------------------------------ converters
        // consecutive lanes take consecutive padded pixels: conflict-free reads of a staged row,
        // coalesced global loads on the direct path, conflict-free 16-byte stores of the codes
        const int tid = conv_warp_index(warp) * 32 + lane;
        bool packed_in = false;
        if constexpr (kNext) packed_in = f.x_packed != nullptr;
        // thresholds (their global-load latency overlaps the first TMA loads, already in flight)
        for (int c = tid; c < p.Cp && !packed_in; c += kConvThreads) {
            // channel padding: thresholds that code everything to 0
            float lo = c < a.C ? a.t_lo[a.n_thr == 1 ? 0 : c] : -INFINITY;
            const float hi = c < a.C ? a.t_hi[a.n_thr == 1 ? 0 : c] : INFINITY;
            if (lo > hi) lo = nextafterf(hi, INFINITY);      // v < lo  <=>  v <= hi: -1 unless +1
            sLo[c] = lo;
            sHi[c] = hi;
        }
        asm volatile("bar.sync %0, %1;" ::"r"(kConvBarrier), "r"(kConvThreads) : "memory");
        if (!p.use_tma) tc::pdl_wait();             // the direct path reads x
        const int64_t cs = (int64_t)a.H * a.W;
        const bool per_layer = a.n_thr == 1 && a.C == p.Cp;     // padding channels need their own (infinite) thresholds
        const int ngroup = p.Cp / 32;
        const float lo0 = sLo[0], hi0 = sHi[0];
        uint32_t st_count = 0;                                 // batches consumed so far
        int row_base = 0;                                      // ring slot of the batch's first row
        int it = 0;
        for (int g = s0; g < s1; g += it == 0 ? p.R0 : p.RT, ++it) {
            const int buf = it & 1;
            // [Cp/16][ppix]; with the whole strip resident the tile's window starts at its first row
            uint4* sA = reinterpret_cast<uint4*>(smem + (buf ? p.off_a[1] : p.off_a[0])) + (p.strip ? (g - s0) * p.PW : 0);
            const int nrows = min(it == 0 ? p.R0 : p.RT, s1 - g);
            const int slot0 = it == 0 ? 0 : p.halo;            // first row slot that is new
            const int pp0 = slot0 * p.PW, pp1 = (nrows + p.halo) * p.PW;
            // (the barrier inside also orders this tile after every converter's writes to the previous buffer)
            if (!p.strip) role_wait(tid < 32, &a_empty[buf], ((it >> 1) & 1) ^ 1, a.status, dead, kConvBarrier, kConvThreads);
            if (tid == 0 && it < 8) RTN_TL(conv_i8, 24 + 2 * it);
            if (it > 0 && !p.strip) {
                // the kh-1 rows shared with the previous tile: copy their codes
                const uint4* prev = reinterpret_cast<const uint4*>(smem + (buf ? p.off_a[0] : p.off_a[1]));
                const int ncopy = p.halo * p.PW;
                const int prev_rows = it == 1 ? p.R0 : p.RT;      // rows of the previous tile
                for (int i = tid; i < nchunk * ncopy; i += kConvThreads) {
                    const int ch = i / ncopy, x = i - ch * ncopy;
                    sA[ch * p.ppix + x] = prev[ch * p.ppix + prev_rows * p.PW + x];
                }
            }
            if (packed_in) {
                // packed pixel rows: item = (padded pixel, 32-channel group) = one word of each bit plane
                // -> 32 int8 codes (two 16-byte chunks)
                if constexpr (kNext) {
                    const int npix = pp1 - pp0;
                    const int64_t row_bytes = (int64_t)((a.C + kBlockCodes - 1) / kBlockCodes) * kBlockBytes;
                    for (int i = tid; i < ngroup * npix; i += kConvThreads) {
                        const int grp = i / npix, pp = pp0 + (i - grp * npix);
                        const uint32_t sl = fdiv((uint32_t)pp, p.div_pw);
                        const int c = (int)((uint32_t)pp - sl * (uint32_t)p.PW) - a.pad;
                        const uint32_t G = (uint32_t)g + sl;
                        const uint32_t b = fdiv(G, p.div_ph);
                        const int r = (int)(G - b * (uint32_t)p.PH) - a.pad;
                        uint32_t nz = 0, sg = 0;
                        if (b < (uint32_t)a.B && r >= 0 && r < a.H && c >= 0 && c < a.W) {
                            const uint32_t* blk = reinterpret_cast<const uint32_t*>(
                                f.x_packed + (((int64_t)b * a.H + r) * a.W + c) * row_bytes) + (grp >> 2) * 8 + (grp & 3);
                            nz = __ldg(blk);
                            sg = __ldg(blk + 4);
                            if (grp * 32 + 32 > a.C) nz &= (1u << (a.C - grp * 32)) - 1u;      // positions past C code to 0
                        }
                        uint32_t o[8];
                        tc::unpack32(nz, sg, o);
                        sA[(2 * grp) * p.ppix + pp] = make_uint4(o[0], o[1], o[2], o[3]);
                        sA[(2 * grp + 1) * p.ppix + pp] = make_uint4(o[4], o[5], o[6], o[7]);
                    }
                }
            } else if (p.use_tma) {
                const int npix = pp1 - pp0;
                for (int grp = 0; grp < ngroup; ++grp, ++st_count) {
                    const uint32_t s = st_count % (uint32_t)kMaxStages;
                    role_wait(tid < 32, &st_full[s], (st_count / (uint32_t)kMaxStages) & 1, a.status, dead,
                              kConvBarrier, kConvThreads);
                    const float* ring = reinterpret_cast<const float*>(smem + p.off_stage);
                    if (tid == 0 && it < 6 && grp < 2) RTN_TL(conv_i8, 72 + 4 * it + 2 * grp);
                    if (p.PW >= kRowwiseMinPW) {
                        // Wide rows: a warp takes a whole (row slot, 16-channel half) and its lanes walk the
                        // row's padded columns, so the row's image, ring slot and validity are worked out once
                        // per warp and row instead of once per value group (index arithmetic was the larger
                        // part of this loop's instructions).
                        const int nnew = nrows + p.halo - slot0;
                        const int W = a.W, PW = p.PW, pad = a.pad;
                        for (int u = tid >> 5; u < 2 * nnew; u += kConvWarps) {
                            const int rowi = u >> 1, hf = u & 1;
                            const int sl = slot0 + rowi;
                            const uint32_t G = (uint32_t)(g + sl);
                            const uint32_t b = fdiv(G, p.div_ph);
                            const int r = (int)(G - b * (uint32_t)p.PH) - pad;
                            const bool row_ok = b < (uint32_t)a.B && r >= 0 && r < a.H;
                            int rs = row_base + rowi;
                            if (rs >= p.nslots) rs -= p.nslots;
                            const int ch = 2 * grp + hf;
                            const float* src_row = ring + ((uint32_t)rs * 32u + 16u * hf) * (uint32_t)W;
                            uint4* dst = sA + ch * p.ppix + sl * PW;
                            // two columns per lane at a time: 32 shared-memory loads in flight per thread
                            for (int cp0 = lane; cp0 < PW; cp0 += 64) {
                                const int cp1 = cp0 + 32;
                                uint4 w0 = make_uint4(0, 0, 0, 0), w1 = w0;
                                if (row_ok) {
                                    const bool ok0 = cp0 >= pad && cp0 < pad + W, ok1 = cp1 >= pad && cp1 < pad + W;
                                    const float* q0 = src_row + (ok0 ? cp0 - pad : 0);      // always inside the slot
                                    const float* q1 = src_row + (ok1 ? cp1 - pad : 0);
                                    float v0[16], v1[16];
                                    #pragma unroll
                                    for (int e = 0; e < 16; ++e) v0[e] = q0[perm16(e) * W];
                                    #pragma unroll
                                    for (int e = 0; e < 16; ++e) v1[e] = q1[perm16(e) * W];
                                    const uint4 t0 = per_layer ? codes16<true>(v0, sLo, sHi, ch * 16, lo0, hi0)
                                                               : codes16<false>(v0, sLo, sHi, ch * 16, lo0, hi0);
                                    const uint4 t1 = per_layer ? codes16<true>(v1, sLo, sHi, ch * 16, lo0, hi0)
                                                               : codes16<false>(v1, sLo, sHi, ch * 16, lo0, hi0);
                                    w0 = make_uint4(ok0 ? t0.x : 0u, ok0 ? t0.y : 0u, ok0 ? t0.z : 0u, ok0 ? t0.w : 0u);
                                    w1 = make_uint4(ok1 ? t1.x : 0u, ok1 ? t1.y : 0u, ok1 ? t1.z : 0u, ok1 ? t1.w : 0u);
                                }
                                dst[cp0] = w0;
                                if (cp1 < PW) dst[cp1] = w1;
                            }
                        }
                    } else
                    // item = (padded pixel, half of the group's 32 channels)
                    for (int i = tid; i < 2 * npix; i += kConvThreads) {
                        const int hf = i >= npix ? 1 : 0;
                        const int pp = pp0 + i - hf * npix;
                        const int ch = 2 * grp + hf;
                        // padded pixel -> (row slot, column) -> (image, row)
                        const uint32_t sl = fdiv((uint32_t)pp, p.div_pw);
                        const int c = (int)((uint32_t)pp - sl * (uint32_t)p.PW) - a.pad;
                        const uint32_t G = (uint32_t)g + sl;
                        const uint32_t b = fdiv(G, p.div_ph);
                        const int r = (int)(G - b * (uint32_t)p.PH) - a.pad;
                        uint4 w = make_uint4(0, 0, 0, 0);
                        if (b < (uint32_t)a.B && r >= 0 && r < a.H && c >= 0 && c < a.W) {
                            int rs = row_base + (int)sl - slot0;
                            if (rs >= p.nslots) rs -= p.nslots;
                            const float* src = ring + ((uint32_t)rs * 32u + 16u * hf) * (uint32_t)a.W + (uint32_t)c;
                            float v[16];
                            #pragma unroll
                            for (int e = 0; e < 16; ++e) v[e] = src[perm16(e) * a.W];
                            w = per_layer ? codes16<true>(v, sLo, sHi, ch * 16, lo0, hi0)
                                          : codes16<false>(v, sLo, sHi, ch * 16, lo0, hi0);
                        }
                        sA[ch * p.ppix + pp] = w;
                    }
                    if (tid == 0 && it < 6 && grp < 2) RTN_TL(conv_i8, 73 + 4 * it + 2 * grp);
                    tc::mbar_arrive(&st_empty[s]);
                    tc::fence_smem_to_async_proxy();
                    tc::mbar_arrive(&a_full[p.strip ? it * ngroup + grp : buf * kMaxGroups + grp]);
                    row_base += nrows + p.halo - slot0;
                    if (row_base >= p.nslots) row_base -= p.nslots;
                }
            } else {
                // direct path: item = (padded pixel, chunk of 16 channels), 16 loads in flight
                const int npix = pp1 - pp0;
                for (int i = tid; i < nchunk * npix; i += kConvThreads) {
                    const int ch = i / npix, pp = pp0 + (i - ch * npix);
                    const uint32_t sl = fdiv((uint32_t)pp, p.div_pw);
                    const int c = (int)((uint32_t)pp - sl * (uint32_t)p.PW) - a.pad;
                    const uint32_t G = (uint32_t)g + sl;
                    const uint32_t b = fdiv(G, p.div_ph);
                    const int r = (int)(G - b * (uint32_t)p.PH) - a.pad;
                    uint4 w = make_uint4(0, 0, 0, 0);
                    if (b < (uint32_t)a.B && r >= 0 && r < a.H && c >= 0 && c < a.W) {
                        const float* src = a.x + (((int64_t)b * a.C + ch * 16) * a.H + r) * a.W + c;
                        float v[16];
                        #pragma unroll
                        for (int e = 0; e < 16; ++e)
                            v[e] = (ch * 16 + perm16(e) < a.C) ? __ldg(src + perm16(e) * cs) : 0.0f;
                        w = codes16<false>(v, sLo, sHi, ch * 16, lo0, hi0);
                    }
                    sA[ch * p.ppix + pp] = w;
                }
            }
            if (!p.use_tma) {
                tc::fence_smem_to_async_proxy();
                for (int grp = 0; grp < ngroup; ++grp)
                    tc::mbar_arrive(&a_full[p.strip ? it * ngroup + grp : buf * kMaxGroups + grp]);
            }
            if (tid == 0 && it < 8) RTN_TL(conv_i8, 25 + 2 * it);
        }
    } else if (warp == kProdWarp) {
        // ------------------------------------------------------------ producer
        if (p.use_tma) {
            const int ngroup = p.Cp / 32;
            // the tensor map sits in the kernel's parameters: fetch it while the previous kernel drains
            asm volatile("prefetch.tensormap [%0];" ::"l"(reinterpret_cast<uint64_t>(&tmap)) : "memory");
            tc::pdl_wait();                         // x may be the previous kernel's output
            uint32_t st_count = 0;              // batches issued
            uint32_t rel = 0;                   // batches known to be released by the converters
            int rel_it = 0, rel_grp = 0;        // (tile, channel group) of batch `rel`
            int head = 0, used = 0;             // ring: next free row slot, row slots held by batches rel..
            bool alive = true;
            int it = 0;
            for (int g = s0; g < s1 && alive; g += it == 0 ? p.R0 : p.RT, ++it) {
                const int nrows = min(it == 0 ? p.R0 : p.RT, s1 - g);
                const int slot0 = it == 0 ? 0 : p.halo;
                const int nnew = nrows + p.halo - slot0;           // new row slots (<= 32)
                // lane j looks at new slot j: which image row is it, if any
                uint32_t info = 0xFFFFFFFFu;
                if (lane < nnew) {
                    const uint32_t G = (uint32_t)(g + slot0 + lane);
                    const uint32_t b = fdiv(G, p.div_ph);
                    const int r = (int)(G - b * (uint32_t)p.PH) - a.pad;
                    if (b < (uint32_t)a.B && r >= 0 && r < a.H) info = (b << 11) | (uint32_t)r;
                }
                const uint32_t mask = __ballot_sync(0xffffffffu, info != 0xFFFFFFFFu);
                __syncwarp();
                sRows[lane] = info;
                __syncwarp();
                if (lane == 0 && it < 8) RTN_TL(conv_i8, 8 + 2 * it);
                for (int grp = 0; grp < ngroup && alive; ++grp, ++st_count) {
                    // room in the ring and a free pair of barriers: retire the oldest batches
                    while (used + nnew > p.nslots || st_count - rel >= (uint32_t)kMaxStages) {
                        const bool ok = wait_or_die(&st_empty[rel % (uint32_t)kMaxStages],
                                                    (rel / (uint32_t)kMaxStages) & 1, a.status, dead);
                        if (!__all_sync(0xffffffffu, ok)) { alive = false; break; }
                        const int rg = s0 + (rel_it == 0 ? 0 : p.R0 + (rel_it - 1) * p.RT);
                        const int rrows = min(rel_it == 0 ? p.R0 : p.RT, s1 - rg);
                        used -= rel_it == 0 ? rrows + p.halo : rrows;
                        ++rel;
                        if (++rel_grp == ngroup) { rel_grp = 0; ++rel_it; }
                    }
                    if (!alive) break;
                    const uint32_t s = st_count % (uint32_t)kMaxStages;
                    if (lane == 0) {
                        if (mask == 0) {
                            tc::mbar_arrive(&st_full[s]);
                        } else {
                            mbar_expect_tx(&st_full[s], (uint32_t)__popc(mask) * p.box_bytes);
                            const uint32_t ring = tc::smem_addr(smem + p.off_stage);
                            const uint32_t bar = tc::smem_addr(&st_full[s]);
                            uint32_t m = mask;
                            while (m) {
                                const int j = __ffs(m) - 1;
                                m &= m - 1;
                                const uint32_t inf = sRows[j];
                                int rs = head + j;
                                if (rs >= p.nslots) rs -= p.nslots;
                                tma_load_row(ring + (uint32_t)rs * p.box_bytes, &tmap, (int)(inf & 0x7FFu), grp * 32,
                                             (int)(inf >> 11), bar);
                            }
                        }
                    }
                    head += nnew;
                    if (head >= p.nslots) head -= p.nslots;
                    used += nnew;
                    __syncwarp();
                }
                if (lane == 0 && it < 8) RTN_TL(conv_i8, 9 + 2 * it);
            }
        }
        if constexpr (kNext && kSk) {
            {
                // The skip connection's values of tile it go to buffer it & 1, one box (32 channels x one output row)
                // per row and channel group, a tile ahead of the epilogue that reads them.
                tc::pdl_wait();                         // the skip tensor may be the previous kernel's output
                const uint32_t stage0 = tc::smem_addr(smem + p.off_skip);
                bool alive = true;
                int it = 0;
                for (int g = s0; g < s1 && alive; g += it == 0 ? p.R0 : p.RT, ++it) {
                    const int nrows = min(it == 0 ? p.R0 : p.RT, s1 - g);
                    const int buf = it & 1;
                    uint32_t info = 0xFFFFFFFFu;        // lane j: output row of the tile's row j, if it is one
                    if (lane < nrows) {
                        const uint32_t G = (uint32_t)(g + lane);
                        const uint32_t b = fdiv(G, p.div_ph);
                        const int ho = (int)(G - b * (uint32_t)p.PH);
                        if (b < (uint32_t)a.B && ho < a.Ho) info = (b << 11) | (uint32_t)ho;
                    }
                    const uint32_t mask = __ballot_sync(0xffffffffu, info != 0xFFFFFFFFu);
                    bool ok = true;
                    if (lane == 0) ok = wait_or_die(&st_empty[buf], ((it >> 1) & 1) ^ 1, a.status, dead);
                    if (!__shfl_sync(0xffffffffu, ok ? 1 : 0, 0)) { alive = false; break; }
                    if (lane == 0) {
                        if (mask == 0) tc::mbar_arrive(&st_full[buf]);
                        else mbar_expect_tx(&st_full[buf], (uint32_t)__popc(mask) * (uint32_t)p.sk_groups * p.sk_box);
                    }
                    __syncwarp();
                    // lane j issues the boxes of row j
                    if (info != 0xFFFFFFFFu) {
                        const uint32_t bar = tc::smem_addr(&st_full[buf]);
                        for (int gq = 0; gq < p.sk_groups; ++gq)
                            tma_load_row(stage0 + (uint32_t)(((buf * p.RT + lane) * p.sk_groups + gq)) * p.sk_box, &tmap,
                                         (int)(info & 0x7FFu), gq * 32, (int)(info >> 11), bar);
                    }
                    __syncwarp();
                }
            }
        }
    } else if (warp == kMmaWarp) {
        // ------------------------------------------------------------ MMA issue (one thread)
        if (lane == 0) {
            const uint32_t idesc = tc::idesc_i8(kTileM, (uint32_t)p.Np);
            // descriptor high word: 8-row group stride 128 bytes, sm_100 descriptor version, no swizzle
            const uint64_t desc_hi = (uint64_t)((128u >> 4) | (1u << 14)) << 32;
            const uint32_t a_lbo_field = (((uint32_t)p.ppix * 16) >> 4) << 16;
            const uint32_t w16 = (tc::smem_addr(sW) >> 4) + ((((uint32_t)p.Np * 16) >> 4) << 16);
            // Filters of up to nine taps: the taps' operand offsets stay in registers, so that nothing
            // but arithmetic sits between two batches of MMAs (the tensor core's queue is short: while
            // the issuing thread waits for a table load, the tensor core idles).
            const bool taps_in_regs = p.T <= 9;
            uint32_t ta[9], tb[9];
            #pragma unroll
            for (int t = 0; t < 9; ++t) {
                ta[t] = taps_in_regs && t < p.T ? p.tab_a[t] : 0u;
                tb[t] = taps_in_regs && t < p.T ? p.tab_b[t] : 0u;
            }
            int it = 0;
            bool filters_ok = wait_or_die(w_ready, 0, a.status, dead);
            for (int g = s0; g < s1 && filters_ok; g += it == 0 ? p.R0 : p.RT, ++it) {
                const int buf = it & 1;
                const uint32_t ph = (it >> 1) & 1;
                const int nrows = min(it == 0 ? p.R0 : p.RT, s1 - g);
                const int ntm = (nrows * p.PW + kTileM - 1) / kTileM;          // sub-tiles with any row
                if (!wait_or_die(&acc_empty[buf], ph ^ 1, a.status, dead)) break;
                const uint32_t a16 = (tc::smem_addr(smem + (buf ? p.off_a[1] : p.off_a[0])) >> 4) +
                                     (p.strip ? (uint32_t)((g - s0) * p.PW) : 0u);
                bool alive = true;
                // channel group by channel group, as the converters finish them
                for (int grp = 0; grp < p.Cp / 32 && alive; ++grp) {
                    alive = wait_or_die(&a_full[p.strip ? it * (p.Cp / 32) + grp : buf * kMaxGroups + grp], p.strip ? 0u : ph,
                                        a.status, dead);
                    if (!alive) break;
                    tc::tc_fence_after_sync();
                    if (grp == 0 && it < 8) RTN_TL(conv_i8, 40 + 2 * it);
                    for (int tm = 0; tm < ntm; ++tm) {
                        const uint32_t d = tmem + (uint32_t)((buf * p.TM + tm) * p.Np);
                        const uint32_t a_tm = a16 + (uint32_t)(tm * kTileM) + a_lbo_field;
                        if (taps_in_regs) {
                            const uint32_t ag = a_tm + (uint32_t)(2 * grp) * (uint32_t)p.ppix;
                            const uint32_t bg = w16 + (uint32_t)(2 * grp) * (uint32_t)p.Np;
                            if (p.T == 9) {
                                tc::mma_i8_ss(d, desc_hi | (ag + ta[0]), desc_hi | (bg + tb[0]), idesc, grp > 0);
                                #pragma unroll
                                for (int t = 1; t < 9; ++t)
                                    tc::mma_i8_ss_acc(d, desc_hi | (ag + ta[t]), desc_hi | (bg + tb[t]), idesc);
                            } else {
                                #pragma unroll
                                for (int t = 0; t < 9; ++t)
                                    if (t < p.T)
                                        tc::mma_i8_ss(d, desc_hi | (ag + ta[t]), desc_hi | (bg + tb[t]), idesc,
                                                      grp > 0 || t > 0);
                            }
                            continue;
                        }
                        int i = grp * p.T;
                        const int i_end = i + p.T;
                        for (; i + 9 <= i_end; i += 9) issue_mmas<9>(p, i, d, a_tm, w16, desc_hi, idesc);
                        if (i + 8 <= i_end) { issue_mmas<8>(p, i, d, a_tm, w16, desc_hi, idesc); i += 8; }
                        if (i + 4 <= i_end) { issue_mmas<4>(p, i, d, a_tm, w16, desc_hi, idesc); i += 4; }
                        if (i + 2 <= i_end) { issue_mmas<2>(p, i, d, a_tm, w16, desc_hi, idesc); i += 2; }
                        if (i + 1 <= i_end) { issue_mmas<1>(p, i, d, a_tm, w16, desc_hi, idesc); i += 1; }
                    }
                }
                if (!alive) break;
                tc::mma_commit(&a_empty[buf]);
                tc::mma_commit(&acc_full[buf]);
                if (it < 8) RTN_TL(conv_i8, 41 + 2 * it);
            }
        }
    } else if (warp >= kEpiWarp0 && warp < kEpiWarp0 + kEpiWarps) {
        // ------------------------------------------------------------ epilogue (8 warps)
        //   out = c1*S_xw + c2*S_x + c3.  Warp w reads TMEM lanes 32 (w mod 4)..+31 (pixels); the two
        //   warps of a lane quarter split the 16-column blocks of the accumulator between them.
        // While the first input rows are in flight these warps, idle until the first accumulators are
        // complete, expand the filters and work out the epilogue constants.
        const int etid = threadIdx.x - kEpiWarp0 * 32;
        // The operands of the epilogue constants are fetched first, so that their trip to memory overlaps the filters'.
        const bool has_col = etid < p.Np && etid < a.N;
        float ws_f = 0.f, wo_f = 0.f;
        int wsum_i = 0;
        if (has_col) {
            ws_f = a.ep.w_scale[a.ep.n_wparam == 1 ? 0 : etid];
            wo_f = a.ep.w_offset[a.ep.n_wparam == 1 ? 0 : etid];
            wsum_i = a.w_sum[etid];
        }
        float2 next_t = make_float2(-INFINITY, INFINITY);
        if constexpr (kNext) {
            if (has_col && f.out_packed != nullptr)
                next_t = make_float2(f.next_lo[f.n_next == 1 ? 0 : etid], f.next_hi[f.n_next == 1 ? 0 : etid]);
        }
        // filters: bit planes -> int8, [tap][chunk][n]; row N is all +1, rows above it are 0
        expand_filter_rows<2>(a.w_packed, sW, p.T, p.Cp / 32, p.Np, p.div_np, p.div_cw, 0, a.N, a.N, etid, kEpiThreads);
        tc::fence_smem_to_async_proxy();
        tc::mbar_arrive(w_ready);
        if (etid == 0) RTN_TL(conv_i8, 2);
        {   // per-output-channel constants in double, rounded once (first needed by the first epilogue):
            //   c1 = a_s*w_s, c2 = a_s*w_o, c3 = a_o*(w_s*S_w + K*w_o)     (K = C*kh*kw)
            const double a_s = a.ep.a_scale_val, a_o = a.ep.a_offset_val;
            if (etid < p.Np) {                          // Np <= 256 = the epilogue's threads: one column each
                float c1 = 0.f, c2 = 0.f, c3 = 0.f;
                if (has_col) {
                    const double ws = ws_f, wo = wo_f;
                    c1 = (float)(a_s * ws);
                    c2 = (float)(a_s * wo);
                    c3 = (float)(a_o * (ws * (double)wsum_i + (double)a.C * p.T * wo));
                }
                sC[etid] = make_float4(c1, c2, c3, 0.f);
            }
            if constexpr (kNext) {
                // the next layer's threshold pair per column; columns past N code to 0
                float2* sT = reinterpret_cast<float2*>(smem + p.off_t);
                if (etid < p.Np) sT[etid] = next_t;
            }
        }
        asm volatile("bar.sync %0, %1;" ::"r"(kEpiBarrier), "r"(kEpiThreads) : "memory");     // constants visible
        tc::pdl_wait();                             // out may still be read by the previous kernel
        if (etid == 0) RTN_TL(conv_i8, 3);
        const int q = warp & 3, half = (warp - kEpiWarp0) >> 2;      // kEpiWarp0 is a multiple of 4
        const int64_t ostride = (int64_t)a.Ho * a.Wo;
        const int nblk16 = (a.N + 15) / 16;
        const int blk_begin = half == 0 ? 0 : (nblk16 + 1) / 2;
        const int blk_end = half == 0 ? (nblk16 + 1) / 2 : nblk16;
        // The constants of this warp's columns go to tensor memory, replicated in each of its 32 lanes:
        // the epilogue then fetches them with tcgen05.ld, which does not compete with the tensor core,
        // the converters and TMA for shared-memory bandwidth as a broadcast shared load per output did.
        const uint32_t cq = tmem + ((uint32_t)(q * 32) << 16) + p.cbase;
        if (p.const_tmem && !kNext) {
            for (int blk = blk_begin; blk < blk_end; ++blk) {
                uint32_t k1[16], k2[16], k3[16];
                #pragma unroll
                for (int j = 0; j < 16; ++j) {
                    const float4 c = sC[blk * 16 + j];
                    k1[j] = __float_as_uint(c.x); k2[j] = __float_as_uint(c.y); k3[j] = __float_as_uint(c.z);
                }
                tc::tmem_st16(cq + (uint32_t)(blk * 16), k1);
                tc::tmem_st16(cq + p.Nc + (uint32_t)(blk * 16), k2);
                tc::tmem_st16(cq + 2 * p.Nc + (uint32_t)(blk * 16), k3);
            }
            tc::tmem_st_wait();
        }
        int it = 0;
        for (int g = s0; g < s1; g += it == 0 ? p.R0 : p.RT, ++it) {
            const int buf = it & 1;
            const int nrows = min(it == 0 ? p.R0 : p.RT, s1 - g);
            const int ntm = (nrows * p.PW + kTileM - 1) / kTileM;
            if (warp == kEpiWarp0) {
                wait_or_die(&acc_full[buf], (it >> 1) & 1, a.status, dead);
                if constexpr (kSk) wait_or_die(&st_full[buf], (it >> 1) & 1, a.status, dead);     // the tile's skip values
            }
            asm volatile("bar.sync %0, %1;" ::"r"(kEpiBarrier), "r"(kEpiThreads) : "memory");
            const bool alive = !*dead;
            tc::tc_fence_after_sync();
            if (etid == 0 && it < 8) RTN_TL(conv_i8, 56 + 2 * it);
            if constexpr (kNext) {
                const float* sk_buf = kSk ? reinterpret_cast<const float*>(smem + p.off_skip) +
                                                (size_t)buf * p.RT * p.sk_groups * (p.sk_box / 4) : nullptr;
                next_epilogue_tile<kSk>(a, p, f, sC, reinterpret_cast<const float2*>(smem + p.off_t), tmem, buf, g, nrows,
                                        alive, q, lane, half, 2, sk_buf);
                if constexpr (kSk) tc::mbar_arrive(&st_empty[buf]);    // this thread has read its skip values
            } else if (p.const_tmem && a.dbg_acc == nullptr && a.pad_mode == RTN_PAD_CODE_ZERO) {
                // Constants in tensor memory, no border classes: the thread's pixels of both sub-tiles (where the
                // tile has one sub-tile, the second pixel does not exist and nothing is stored for it) go
                // through the channel blocks together, so that one fetch of a block's
                // constants serves two pixels and the epilogue waits for tensor memory half as often
                // (the wait for a tcgen05.ld, several hundred cycles while the tensor core works on the next
                // tile, is what this epilogue's time is made of).
                float* optr2[2];
                bool ok2[2];
                uint32_t trow2[2], sx2[2];
                #pragma unroll
                for (int t = 0; t < 2; ++t) {
                    const uint32_t pl = (uint32_t)(t * kTileM + q * 32 + lane);
                    const uint32_t row = fdiv(pl, p.div_pw);
                    const int wo = (int)(pl - row * (uint32_t)p.PW);
                    const uint32_t G = (uint32_t)g + row;
                    const uint32_t b = fdiv(G, p.div_ph);
                    const int ho = (int)(G - b * (uint32_t)p.PH);
                    ok2[t] = alive && t < ntm && (int)row < nrows && b < (uint32_t)a.B && ho < a.Ho && wo < a.Wo;
                    trow2[t] = tmem + ((uint32_t)(q * 32) << 16) + (uint32_t)((buf * p.TM + (t < ntm ? t : 0)) * p.Np);
                    optr2[t] = a.out + (((int64_t)b * a.N) * a.Ho + ho) * a.Wo + wo;
                    asm volatile("tcgen05.ld.sync.aligned.32x32b.x1.b32 {%0}, [%1];"
                                 : "=r"(sx2[t]) : "r"(trow2[t] + (uint32_t)a.N) : "memory");
                }
                tc::tmem_ld_wait();
                const float fsx0 = (float)(int)sx2[0], fsx1 = (float)(int)sx2[1];
                for (int blk = blk_begin; blk < blk_end; ++blk) {
                    const int n0 = blk * 16;
                    if (n0 + 16 <= a.N) {
                        // running pointers: one 64-bit add per store instead of a 64-bit product and a shift
                        float* q0 = optr2[0] + (int64_t)n0 * ostride;
                        float* q1 = optr2[1] + (int64_t)n0 * ostride;
                        #pragma unroll
                        for (int h8 = 0; h8 < 16; h8 += 8) {
                            uint32_t u0[8], u1[8], k1[8], k2[8], k3[8];
                            tc::tmem_ld8(trow2[0] + (uint32_t)(n0 + h8), u0);
                            tc::tmem_ld8(trow2[1] + (uint32_t)(n0 + h8), u1);
                            tc::tmem_ld8(cq + (uint32_t)(n0 + h8), k1);
                            tc::tmem_ld8(cq + p.Nc + (uint32_t)(n0 + h8), k2);
                            tc::tmem_ld8(cq + 2 * p.Nc + (uint32_t)(n0 + h8), k3);
                            tc::tmem_ld_wait();
                            if (ok2[0]) {
                                #pragma unroll
                                for (int j = 0; j < 8; ++j, q0 += ostride)
                                    *q0 = fmaf(__uint_as_float(k1[j]), (float)(int)u0[j],
                                               fmaf(__uint_as_float(k2[j]), fsx0, __uint_as_float(k3[j])));
                            }
                            if (ok2[1]) {
                                #pragma unroll
                                for (int j = 0; j < 8; ++j, q1 += ostride)
                                    *q1 = fmaf(__uint_as_float(k1[j]), (float)(int)u1[j],
                                               fmaf(__uint_as_float(k2[j]), fsx1, __uint_as_float(k3[j])));
                            }
                        }
                    } else {
                        // the last, ragged block: constants from shared memory
                        uint32_t u0[16], u1[16];
                        tc::tmem_ld16(trow2[0] + (uint32_t)n0, u0);
                        tc::tmem_ld16(trow2[1] + (uint32_t)n0, u1);
                        tc::tmem_ld_wait();
                        #pragma unroll
                        for (int j = 0; j < 16; ++j) {
                            if (n0 + j >= a.N) continue;
                            const float4 c = sC[n0 + j];
                            if (ok2[0]) optr2[0][(int64_t)(n0 + j) * ostride] = fmaf(c.x, (float)(int)u0[j], fmaf(c.y, fsx0, c.z));
                            if (ok2[1]) optr2[1][(int64_t)(n0 + j) * ostride] = fmaf(c.x, (float)(int)u1[j], fmaf(c.y, fsx1, c.z));
                        }
                    }
                }
            } else
            for (int tm = 0; tm < ntm; ++tm) {
                const uint32_t pl = (uint32_t)(tm * kTileM + q * 32 + lane);     // pixel within the tile
                const uint32_t row = fdiv(pl, p.div_pw);
                const int wo = (int)(pl - row * (uint32_t)p.PW);
                const uint32_t G = (uint32_t)g + row;
                const uint32_t b = fdiv(G, p.div_ph);
                const int ho = (int)(G - b * (uint32_t)p.PH);
                const bool ok = alive && (int)row < nrows && b < (uint32_t)a.B && ho < a.Ho && wo < a.Wo;
                int n_inside = p.T;
                if (ok && a.pad_mode == RTN_PAD_VALUE_ZERO) {
                    n_inside = 0;
                    for (int t = 0; t < p.T; ++t) {
                        const int h = ho - a.pad + t / a.kw, v = wo - a.pad + t % a.kw;
                        n_inside += (h >= 0 && h < a.H && v >= 0 && v < a.W);
                    }
                }
                const bool border = n_inside < p.T;
                const uint32_t trow = tmem + ((uint32_t)(q * 32) << 16) + (uint32_t)((buf * p.TM + tm) * p.Np);
                float* optr = a.out + (((int64_t)b * a.N) * a.Ho + ho) * a.Wo + wo;
                int32_t* dptr = a.dbg_acc ? a.dbg_acc + (((int64_t)b * a.N) * a.Ho + ho) * a.Wo + wo : nullptr;
                // S_x of this pixel: accumulator column N (the all-ones filter row)
                uint32_t sx_raw;
                asm volatile("tcgen05.ld.sync.aligned.32x32b.x1.b32 {%0}, [%1];"
                             : "=r"(sx_raw) : "r"(trow + (uint32_t)a.N) : "memory");
                bool sx_ready = false;
                float fsx = 0.f;
                // uniform over the warp: whole blocks with constants in tensor memory and no debug output
                const bool tm_path = p.const_tmem && a.dbg_acc == nullptr;
                for (int blk = blk_begin; blk < blk_end; ++blk) {
                    const int n0 = blk * 16;
                    if (tm_path && n0 + 16 <= a.N) {
                        // eight columns at a time: accumulators and the three constants from tensor memory
                        #pragma unroll
                        for (int h8 = 0; h8 < 16; h8 += 8) {
                            uint32_t u8[8], k1[8], k2[8], k3[8];
                            tc::tmem_ld8(trow + (uint32_t)(n0 + h8), u8);
                            tc::tmem_ld8(cq + (uint32_t)(n0 + h8), k1);
                            tc::tmem_ld8(cq + p.Nc + (uint32_t)(n0 + h8), k2);
                            tc::tmem_ld8(cq + 2 * p.Nc + (uint32_t)(n0 + h8), k3);
                            tc::tmem_ld_wait();
                            if (!sx_ready) { fsx = (float)(int)sx_raw; sx_ready = true; }
                            if (ok && !border) {
                                #pragma unroll
                                for (int j = 0; j < 8; ++j)
                                    optr[(int64_t)(n0 + h8 + j) * ostride] =
                                        fmaf(__uint_as_float(k1[j]), (float)(int)u8[j],
                                             fmaf(__uint_as_float(k2[j]), fsx, __uint_as_float(k3[j])));
                            } else if (ok) {
                                // value-zero padding at an image border: S_w and K over inside taps only
                                #pragma unroll
                                for (int j = 0; j < 8; ++j) {
                                    const int n = n0 + h8 + j;
                                    int s_w = 0;
                                    for (int t = 0; t < p.T; ++t) {
                                        const int h = ho - a.pad + t / a.kw, vv = wo - a.pad + t % a.kw;
                                        if (h >= 0 && h < a.H && vv >= 0 && vv < a.W) s_w += a.w_sum[(1 + t) * a.N + n];
                                    }
                                    const double ws = a.ep.w_scale[a.ep.n_wparam == 1 ? 0 : n];
                                    const double wo_ = a.ep.w_offset[a.ep.n_wparam == 1 ? 0 : n];
                                    const float c3 = (float)((double)a.ep.a_offset_val *
                                                             (ws * (double)s_w + (double)a.C * n_inside * wo_));
                                    optr[(int64_t)n * ostride] = fmaf(__uint_as_float(k1[j]), (float)(int)u8[j],
                                                                      fmaf(__uint_as_float(k2[j]), fsx, c3));
                                }
                            }
                        }
                        continue;
                    }
                    uint32_t u[16];
                    tc::tmem_ld16(trow + (uint32_t)n0, u);
                    tc::tmem_ld_wait();
                    if (!sx_ready) { fsx = (float)(int)sx_raw; sx_ready = true; }
                    if (ok) {
                        if (!border && dptr == nullptr && n0 + 16 <= a.N) {
                            // results first, stores after (a load of the next constants may not pass a global store)
                            float r[16];
                            #pragma unroll
                            for (int j = 0; j < 16; ++j) {
                                const float4 c = sC[n0 + j];
                                r[j] = fmaf(c.x, (float)(int)u[j], fmaf(c.y, fsx, c.z));
                            }
                            float* o = optr + (int64_t)n0 * ostride;
                            #pragma unroll
                            for (int j = 0; j < 16; ++j, o += ostride) *o = r[j];
                        } else {
                            #pragma unroll
                            for (int j = 0; j < 16; ++j) {
                                const int n = n0 + j;
                                if (n >= a.N) continue;
                                const int s_xw = (int)u[j];
                                const float4 c = sC[n];
                                float c3 = c.z;
                                if (border) {
                                    // value-zero padding at an image border: S_w and K over inside taps only
                                    int s_w = 0;
                                    for (int t = 0; t < p.T; ++t) {
                                        const int h = ho - a.pad + t / a.kw, vv = wo - a.pad + t % a.kw;
                                        if (h >= 0 && h < a.H && vv >= 0 && vv < a.W) s_w += a.w_sum[(1 + t) * a.N + n];
                                    }
                                    const double ws = a.ep.w_scale[a.ep.n_wparam == 1 ? 0 : n];
                                    const double wo_ = a.ep.w_offset[a.ep.n_wparam == 1 ? 0 : n];
                                    c3 = (float)((double)a.ep.a_offset_val *
                                                 (ws * (double)s_w + (double)a.C * n_inside * wo_));
                                }
                                optr[(int64_t)n * ostride] = fmaf(c.x, (float)s_xw, fmaf(c.y, fsx, c3));
                                if (dptr != nullptr) dptr[(int64_t)n * ostride] = s_xw;
                            }
                        }
                    }
                }
                if (blk_begin >= blk_end) tc::tmem_ld_wait();      // the S_x load still has to land
            }
            tc::tc_fence_before_sync();
            tc::mbar_arrive(&acc_empty[buf]);
            if (etid == 0 && it < 8) RTN_TL(conv_i8, 57 + 2 * it);
        }
    }
    tc::tc_fence_before_sync();
    __syncthreads();
    if (warp == 0) tc::tmem_dealloc(tmem, p.tmem_cols);
    if (threadIdx.x == 0) RTN_TL(conv_i8, 4);
}

}  // namespace

bool conv_i8_supported(const ConvArgs& c)
{
    ConvI8Plan p;
    return make_plan(c, p, device_sm_count());
}

bool conv_i8_next_supported(const ConvArgs& c)
{
    ConvI8Plan p;
    return make_plan(c, p, device_sm_count(), true);
}

static cudaError_t launch_conv_i8_any_mode(const ConvArgs& c, const NextLayerArgs* f, cudaStream_t s)
{
    ConvI8Plan p;
    if (!make_plan(c, p, device_sm_count(), f != nullptr)) return cudaErrorInvalidConfiguration;
    CUtensorMap tmap;
    memset(&tmap, 0, sizeof(tmap));
    if (f != nullptr && f->x_packed != nullptr) {
        // packed pixel rows are read with plain loads by the converters: no staging ring
        p.use_tma = 0;
        p.smem_bytes = p.off_stage;
        // The skip connection of a block's second layer: with no input ring to fill, the producer warp stages each
        // tile's skip values in shared memory by TMA a tile ahead (boxes of 32 channels x one output row), and the
        // epilogue reads them from there: as global loads they were a dependent trip to memory per half block, half of
        // such a layer's time.  Two tile buffers must fit; the channel-split epilogue is the one that reads them.
        const uint32_t base = (p.off_stage + 127) / 128 * 128;
        const uint32_t sk_box = 32u * (uint32_t)c.Wo * 4u;
        const int groups = (int)(c.N / 32);
        if (f->skip != nullptr && (c.N == 64 || c.N == 128) && c.pad_mode == RTN_PAD_CODE_ZERO && c.Wo % 4 == 0 &&
            reinterpret_cast<uintptr_t>(f->skip) % 16 == 0 &&
            base + (uint64_t)2 * p.RT * groups * sk_box <= kSmemLimit) {
            EncodeTiledFn enc = encode_tiled_fn();
            const cuuint64_t dims[4] = {(cuuint64_t)c.Wo, (cuuint64_t)c.Ho, (cuuint64_t)c.N, (cuuint64_t)c.B};
            const cuuint64_t strides[3] = {(cuuint64_t)c.Wo * 4, (cuuint64_t)c.Wo * c.Ho * 4,
                                           (cuuint64_t)c.Wo * c.Ho * c.N * 4};
            const cuuint32_t box[4] = {(cuuint32_t)c.Wo, 1, 32, 1};
            const cuuint32_t estr[4] = {1, 1, 1, 1};
            if (enc != nullptr &&
                enc(&tmap, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 4, const_cast<float*>(f->skip), dims, strides, box, estr,
                    CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_NONE, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
                    CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS) {
                p.sk_stage = 1; p.sk_groups = groups; p.off_skip = base; p.sk_box = sk_box;
                p.smem_bytes = base + (size_t)2 * p.RT * groups * sk_box;
            }
        }
    }
    if (p.use_tma) {
        EncodeTiledFn enc = encode_tiled_fn();
        const cuuint64_t dims[4] = {(cuuint64_t)c.W, (cuuint64_t)c.H, (cuuint64_t)c.C, (cuuint64_t)c.B};
        const cuuint64_t strides[3] = {(cuuint64_t)c.W * 4, (cuuint64_t)c.W * c.H * 4,
                                       (cuuint64_t)c.W * c.H * c.C * 4};
        const cuuint32_t box[4] = {(cuuint32_t)c.W, 1, 32, 1};
        const cuuint32_t estr[4] = {1, 1, 1, 1};
        if (enc == nullptr ||
            enc(&tmap, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 4, const_cast<float*>(c.x), dims, strides, box, estr,
                CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_NONE, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
                CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS) {
            // describing the input to TMA failed: let the converters load it themselves
            p.use_tma = 0;
            p.smem_bytes = p.off_stage;
        }
    }
    if (f != nullptr) {
        if (p.sk_stage) {
            cudaError_t e = cudaFuncSetAttribute(conv_i8_kernel<true, true>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                                 (int)p.smem_bytes);
            if (e != cudaSuccess) return e;
            return launch_pdl(conv_i8_kernel<true, true>, dim3((unsigned)p.grid), dim3(kThreads), p.smem_bytes, s, c, p, tmap, *f);
        }
        cudaError_t e = cudaFuncSetAttribute(conv_i8_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                             (int)p.smem_bytes);
        if (e != cudaSuccess) return e;
        return launch_pdl(conv_i8_kernel<true>, dim3((unsigned)p.grid), dim3(kThreads), p.smem_bytes, s, c, p, tmap, *f);
    }
    cudaError_t e = cudaFuncSetAttribute(conv_i8_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                         (int)p.smem_bytes);
    if (e != cudaSuccess) return e;
    return launch_pdl(conv_i8_kernel<false>, dim3((unsigned)p.grid), dim3(kThreads), p.smem_bytes, s, c, p, tmap,
                      NextLayerArgs{});
}

cudaError_t launch_conv_i8(const ConvArgs& c, cudaStream_t s) { return launch_conv_i8_any_mode(c, nullptr, s); }

// The same kernel with the hand-over to the next layer (and, optionally, packed input).
cudaError_t launch_conv_i8_next(const ConvArgs& c, const NextLayerArgs& f, cudaStream_t s)
{
    return launch_conv_i8_any_mode(c, &f, s);
}

}  // namespace rtn
