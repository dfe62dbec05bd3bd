// Ternary conv2d, tensor-core variant with STREAMED filters: for layers whose int8 filter bank does
// not fit shared memory (e.g. 256 -> 256 channels, 3x3) and for 1x1 convolutions of any stride.
//
// Same arithmetic as the resident-filter kernel: fp32 NCHW input ternarized in-kernel (Eq. 3) to
// int8 codes in shared memory laid out [16-channel chunk][pixel][16 B] (K-major, no swizzle), the
// implicit GEMM of a stride-1 conv done by shifting the A window by (i*PW + j) pixels per filter
// tap, tcgen05.mma kind::i8 into int32 accumulators in tensor memory, affine epilogue fused.
// Differences:
//   * the filters are expanded from their bit planes (Table 1) to int8 one packed block (four
//     K = 32 slices) at a time into a ring of shared-memory stages by warps of their own, while the
//     tensor core consumes earlier stages; expanding costs a quarter of the SM's issue slots per
//     256-pixel tile, so a CTA's tile is made 256 pixels whenever its strip has that many;
//   * when C is a multiple of 128 the K loop runs 128-channel block by block (all taps of a block,
//     then the next block), and the ternarizer hands the code buffer over in 32-channel groups, so
//     the tensor core starts on a tile before all of its input has arrived;
//   * S_x comes from per-pixel code sums the ternarizer leaves in shared memory (summed over the
//     taps in the epilogue), so all 256 accumulator columns are free for output channels;
//   * a 1x1 convolution (any stride, no padding) uses the same code with "rows" = output rows and a
//     strided pixel gather in the ternarizer (no halo, one tap);
//   * for a long filter stream (four stages or more) every CTA expanding the whole bank again is the
//     kernel's largest cost (cfg3a: 18 stages of about 1 us each per tile against 9 us of MMAs), so
//     the bank is expanded ONCE, by a small kernel of its own, into a scratch buffer laid out stage by
//     stage as the ring wants it; one thread of the contraction kernel then fills the ring with bulk
//     asynchronous copies (one 32 KB run per stage, served by L2) and the expander warps have
//     nothing to do.
//
// Warp roles: warp 0 issues MMAs (one thread); warps 12..19 expand filters; warps 4..11 ternarize
// tile i+1 and then run the epilogue of tile i; warps 1..3 only ternarize.  One or two code buffers
// and accumulator sets (as fit), mbarrier hand-offs with bounded waits.  Every CTA takes an equal
// strip of the padded rows and cuts it into equal tiles, so that all SMs are busy whatever the
// batch size.
#include "rtn_internal.cuh"
#include "rtn_tcgen05.cuh"
#include "rtn_conv_i8_common.cuh"
#include "rtn_timeline.cuh"

// Timeline slots (instrumented build only; same plan as conv_i8_kernel): 0 kernel entry, 1 set-up done, 4 kernel end;
// per tile i < 8: 24+2i / 25+2i ternarizer thread 0 begins / ends, 40+2i / 41+2i first MMA issued / accumulators
// committed, 56+2i / 57+2i epilogue begins / ends.
RTN_TL_DEFINE(conv_i8s)

namespace rtn {

namespace {

using namespace conv_detail;

constexpr int kEpiWarp0 = 4;
constexpr int kEpiWarps = 8;
constexpr int kEpiThreads = kEpiWarps * 32;
constexpr int kExpWarp0 = 12;
constexpr int kExpWarps = 8;
constexpr int kExpThreads = kExpWarps * 32;
constexpr int kTernWarps = 11;                         // warps 1..11
constexpr int kTernThreads = kTernWarps * 32;
constexpr int kThreads = 20 * 32;
constexpr int kTileM = 128;
constexpr int kMaxK = 304;                             // K = 32 slices per tile the table holds
constexpr int kMaxWStages = 8;
constexpr int kSlices = 4;                             // K = 32 slices per filter stage (one packed block)
constexpr int kMaxGroups = 16;                         // 32-channel groups (C <= 512)
constexpr int kPsumRing = 4;
constexpr size_t kSmemLimit = 220 * 1024;
constexpr int kEpiBarrier = 1, kTernBarrier = 2, kExpBarrier = 3;

struct ConvI8SPlan {
    int PW, PH;            // row length / rows per image of the pixel sequence (padded for k > 1)
    int istride, ipad;     // input pixel of sequence pixel (r, c): (r*istride - ipad, c*istride - ipad)
    int Cp, Np, T, TM, RT, halo, ppix, total_rows, grid;
    int nK;                // K = 32 slices per tile in stage order, padded to whole packed blocks
    int nW;                // filter ring depth
    int nAcc;              // accumulator sets (1 or 2)
    int npass, NpP;        // passes over the output channels (groups of NpP filters) and columns per pass
    int split;             // the passes are dealt to CTAs (CTA = strip x filter group) instead of run one after the other
    int nstrips;           // strips of rows; grid = nstrips * (split ? npass : 1)
    int nA;                // code buffers (1 or 2)
    uint32_t tmem_cols;
    FastDiv div_pw, div_ph, div_T;   // div_T: stage -> (128-channel block, tap)
    uint32_t off_a[2], off_w, off_psum, off_lo, off_hi, off_c, off_t, off_bar, off_misc, off_tab;
    size_t smem_bytes;
    int blocks_major;      // stage order: 128-channel block outer, tap inner (else the packed order)
    int pre;               // filters expanded beforehand into scratch, slices in (32-channel group, tap) order
    uint32_t tab_a[kMaxK]; // per slice of the stage order: start of the A window in 16-byte units of
                           // the code buffer (bits 0..23) and its 32-channel group (bits 24..27);
                           // 0xFFFFFFFF for the padding slices of the last packed block
};

// split: the filter bank is cut into groups of 128 filters and a CTA takes one group for its strip (it streams a
// group's share of the bank only; its tensor-core instructions are 128 columns wide).
bool make_plan_mode(const ConvArgs& c, ConvI8SPlan& p, int sms, bool next, bool split)
{
    if (c.Ho <= 0 || c.Wo <= 0) return false;
    p.T = c.kh * c.kw;
    if (c.stride == 1) {
        p.PW = c.W + 2 * c.pad; p.PH = c.H + 2 * c.pad; p.istride = 1; p.ipad = c.pad; p.halo = c.kh - 1;
    } else if (p.T == 1 && c.pad == 0) {
        p.PW = c.Wo; p.PH = c.Ho; p.istride = c.stride; p.ipad = 0; p.halo = 0;
    } else {
        return false;
    }
    if (p.PW > 256 || p.PH > 2048) return false;
    if ((int64_t)c.B * p.PH > (1 << 20)) return false;
    p.Cp = (c.C + 31) / 32 * 32;
    p.Np = (c.N + 15) / 16 * 16;
    // More than 256 filters: two passes over the tile's codes, 256 output channels each; a pass is to the
    // accumulator sets and their barriers what a tile is, so with two sets the first pass's epilogue runs
    // under the second pass's MMAs.  Only with the filters expanded beforehand (checked below).
    if (p.Np > 512) return false;
    p.split = split ? 1 : 0;
    if (split) {
        if (p.Np <= 128) return false;
        p.NpP = 128;
        p.npass = (p.Np + 127) / 128;
    } else {
        p.npass = p.Np > 256 ? 2 : 1;
        p.NpP = p.npass == 2 ? 256 : p.Np;
    }
    if (p.Cp / 32 > kMaxGroups) return false;
    p.total_rows = c.B * p.PH;
    if (split) {
        // one wave of CTAs: a strip per whole 256-pixel tile when that many CTAs fit, else as many strips as fit
        const int rt2 = 2 * kTileM / p.PW;
        if (rt2 < 1 || sms / p.npass < 1) return false;
        const int tiles2 = (p.total_rows + rt2 - 1) / rt2;
        p.nstrips = tiles2 * p.npass <= sms ? tiles2 : sms / p.npass;
        if (p.nstrips > p.total_rows) p.nstrips = p.total_rows;
        p.grid = p.nstrips * p.npass;
    } else {
        p.nstrips = p.total_rows < sms ? p.total_rows : sms;
        p.grid = p.nstrips;
    }
    // 256-pixel tiles whenever a CTA's strip has more than 128 pixels: a tile's filter stream costs
    // the same whatever its size
    const int strip_rows = (p.total_rows + p.nstrips - 1) / p.nstrips;
    p.TM = (2 * p.NpP <= 512 && strip_rows * p.PW > kTileM) ? 2 : 1;
    p.nAcc = (2 * p.TM * p.NpP <= 512) ? 2 : 1;
    p.RT = p.TM * kTileM / p.PW;
    if (p.RT < 1) return false;
    p.ppix = (p.TM * kTileM + p.halo * p.PW + (c.kw - 1) + 7) / 8 * 8;
    uint32_t cols = 32;
    while (cols < (uint32_t)(p.nAcc * p.TM * p.NpP)) cols *= 2;
    p.tmem_cols = cols;
    p.div_pw = make_fastdiv((uint32_t)p.PW);
    p.div_ph = make_fastdiv((uint32_t)p.PH);
    p.div_T = make_fastdiv((uint32_t)p.T);
    const int cwords = p.Cp / 32;
    const int nwords = p.T * cwords;
    const int nblocks = (nwords + kSlices - 1) / kSlices;
    p.nK = nblocks * kSlices;
    if (p.nK > kMaxK) return false;
    p.blocks_major = (cwords % kSlices == 0) ? 1 : 0;
    // A long filter stream is expanded beforehand into scratch, and the order of its K = 32 slices is then
    // free: 32-channel group outer, tap inner, so that the tensor core starts on a tile as soon as the
    // first 32 channels are ternarized and follows the ternarizers group by group.
    p.pre = nblocks >= 4 ? 1 : 0;
    if (p.npass > 1 && !p.pre) return false;
    if (split && !p.pre) return false;
    for (int i = 0; p.pre && i < p.nK; ++i) {
        uint32_t e = 0xFFFFFFFFu;
        if (i < nwords) {
            const int h = i / p.T, t = i % p.T;
            e = ((uint32_t)(2 * h) * p.ppix + (uint32_t)((t / c.kw) * p.PW + (t % c.kw))) | ((uint32_t)h << 24);
        }
        p.tab_a[i] = e;
    }
    for (int st = 0; !p.pre && st < nblocks; ++st) {
        // packed block of stage st
        const int blk = p.blocks_major ? (st % p.T) * (cwords / kSlices) + st / p.T : st;
        for (int j = 0; j < kSlices; ++j) {
            const int word = blk * kSlices + j;
            uint32_t e = 0xFFFFFFFFu;
            if (word < nwords) {
                const int t = word / cwords, h = word % cwords;
                e = ((uint32_t)(2 * h) * p.ppix + (uint32_t)((t / c.kw) * p.PW + (t % c.kw))) | ((uint32_t)h << 24);
            }
            p.tab_a[st * kSlices + j] = e;
        }
    }
    const uint32_t a_bytes = (uint32_t)(p.Cp / 16) * p.ppix * 16;
    const uint32_t stage = (uint32_t)p.NpP * 32 * kSlices;
    const int nstages = p.nK / kSlices;
    // two code buffers when they leave room for a filter ring of four stages (or all of them); a CTA with a single
    // tile has no use for the second one, and the ring, whose depth is what hides a stage's trip from L2, gets the room
    const int strip_tiles = (strip_rows + p.RT - 1) / p.RT;
    for (p.nA = strip_tiles == 1 ? 1 : 2; p.nA >= 1; --p.nA) {
        uint32_t o = 0;
        p.off_a[0] = o; o += a_bytes;
        p.off_a[1] = o; if (p.nA == 2) o += a_bytes;
        p.off_psum = o; o += (uint32_t)kPsumRing * (uint32_t)p.ppix * 4;
        p.off_lo = o;   o += (uint32_t)p.Cp * 4;
        p.off_hi = o;   o += (uint32_t)p.Cp * 4;
        o = (o + 15) / 16 * 16;
        p.off_c = o;    o += (uint32_t)p.Np * 16;
        p.off_t = o;    o += next ? (uint32_t)p.Np * 8 : 0;     // float2 {t_lo, t_hi} of the next layer per column
        p.off_bar = o;  o += (6 + 2 * kMaxWStages + 2 * kMaxGroups) * 8;   // a_empty[2] acc_full[2] acc_empty[2] w_full[] w_empty[] a_full[2][]
        p.off_misc = o; o += 16;
        p.off_tab = o;  o += p.pre ? (uint32_t)(nstages + 1) * 16 : 0;     // per stage: the A windows of its four slices
        o = (o + 127) / 128 * 128;
        p.off_w = o;
        if (o > kSmemLimit) continue;
        int nw = (int)((kSmemLimit - o) / stage);
        if (nw > kMaxWStages) nw = kMaxWStages;
        if (nw > nstages) nw = nstages;
        const int want = nstages < 4 ? nstages : 4;
        if (nw < want && p.nA == 2) continue;
        if (nw < 2 && nstages > 1) return false;
        if (nw < 1) return false;
        p.nW = nw;
        p.smem_bytes = o + (uint32_t)nw * stage;
        return true;
    }
    return false;
}

// Rough time of a plan, in microseconds, from measurements on B200 (packed input; fp32 input adds to every plan
// alike).  With the filters streamed from scratch a tensor-core instruction of N columns costs about N/2 + 60
// cycles in this kernel's issue loop and the stream keeps up; expanded in the kernel a 32 KB stage takes 1 us.  A
// tile's codes take 2 ns per pixel and 32-channel group; the last tile's epilogue, which nothing overlaps, 1.5 us
// plus a microsecond per 7500 outputs of a CTA; launch, set-up and the first stage's trip about 3 us.
static double plan_estimate_us(const ConvI8SPlan& p)
{
    const int strip_rows = (p.total_rows + p.nstrips - 1) / p.nstrips;
    const int tiles = (strip_rows + p.RT - 1) / p.RT;
    const int nstages = p.nK / kSlices;
    const int passes = p.split ? 1 : p.npass;
    double stage_us = kSlices * p.TM * (p.NpP / 2.0 + 60.0) / 1900.0;
    if (!p.pre && stage_us < (double)p.NpP / 256.0) stage_us = (double)p.NpP / 256.0;
    const double px = (double)(strip_rows < p.RT ? strip_rows : p.RT) * p.PW;
    const double tern_us = px * (p.Cp / 32) * 0.002;
    const double mma_us = (double)passes * nstages * stage_us;
    const double tile_us = mma_us > tern_us ? mma_us : tern_us;
    return 3.0 + tile_us * tiles + tern_us / (p.Cp / 32) + 1.5 + px * p.NpP / 7500.0;
}

// The plan of the faster of the two ways to share out the filters.  (Groups of 128 as passes of ONE CTA, so that a
// pass's epilogue runs under the next pass's MMAs, measured slower than either on every ResNet-18 layer: 128-column
// instructions cost this kernel's issue loop 124 cycles against 188 for 256 columns.)
bool make_plan_s(const ConvArgs& c, ConvI8SPlan& p, int sms, bool next = false)
{
    ConvI8SPlan q;
    const bool whole = make_plan_mode(c, p, sms, next, false);
    const bool split = make_plan_mode(c, q, sms, next, true);
    if (split && (!whole || plan_estimate_us(q) < plan_estimate_us(p))) p = q;
    return whole || split;
}

// One warp of a role waits on the mbarrier; the role's other warps sleep on a hardware named
// barrier until it gets there.
__device__ __forceinline__ void role_wait(bool leader, uint64_t* bar, uint32_t parity, unsigned* status,
                                          volatile int* dead, int barrier_id, int nthreads)
{
    if (leader) wait_or_die(bar, parity, status, dead);
    asm volatile("bar.sync %0, %1;" ::"r"(barrier_id), "r"(nthreads) : "memory");
}

// The filter bank expanded once: wexp[pass][stage][16-byte k chunk (8)][filter row of the pass][16 B], the bytes a ring
// stage holds, in the slice order of the plan (32-channel group outer, tap inner).  Thread = (stage, slice of the
// stage, filter row): one word of each bit plane in, 32 bytes out (the kernel is a launch and one round trip to
// memory long, so the work is spread thin).
__global__ void __launch_bounds__(256)
conv_expand_filters_kernel(const ConvArgs a, const __grid_constant__ ConvI8SPlan p, uint4* __restrict__ wexp)
{
    tc::pdl_trigger();          // the contraction kernel may start its set-up (it reads no expanded filters there)
    const int nstages = p.nK / kSlices;
    const int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= (int64_t)p.npass * nstages * kSlices * p.NpP) return;
    const int r = (int)(i % p.NpP);
    const int sj = (int)(i / p.NpP);                         // (pass * nstages + stage of the pass) * kSlices + slice
    const int j = sj % kSlices, st = sj / kSlices;
    const int row = r + (st / nstages) * p.NpP;             // filter
    const int stage_of_pass = st % nstages;
    const int cwords = p.Cp / 32, nwords = p.T * cwords;
    const int64_t row_blocks = ((int64_t)p.T * cwords + 3) / 4;
    // slice stage*4 + j of the stream = (32-channel group h, tap t) = word t*cwords + h of the packed row
    const int sl = stage_of_pass * kSlices + j;
    uint32_t nz = 0, sg = 0;
    if (sl < nwords && row < a.N) {
        const uint32_t* Wrow = reinterpret_cast<const uint32_t*>(a.w_packed) + (int64_t)row * row_blocks * 8;
        const int h = sl / p.T, t = sl - h * p.T;
        const int word = t * cwords + h;
        nz = __ldg(Wrow + (word >> 2) * 8 + (word & 3));
        sg = __ldg(Wrow + (word >> 2) * 8 + 4 + (word & 3));
    }
    uint32_t o[8];
    tc::unpack32(nz, sg, o);
    uint4* dst = wexp + ((int64_t)st * kSlices + j) * 2 * p.NpP + r;
    dst[0] = make_uint4(o[0], o[1], o[2], o[3]);
    dst[p.NpP] = make_uint4(o[4], o[5], o[6], o[7]);
}

// kPre: the filter stages come from the scratch buffer conv_expand_filters_kernel wrote (bulk copies by
// one thread) instead of being expanded by warps 12..19.
// kNext: the layer hands its result to the next one (NextLayerArgs): the input may come as packed pixel
// rows (the ternarizers then expand bit planes), and the epilogue applies phi, adds the skip connection and
// writes fp32 and / or packed Eq. 3 codes against the next layer's thresholds.
template <bool kPre, bool kNext>
__global__ void __launch_bounds__(kThreads, 1)
conv_i8s_kernel(const ConvArgs a, const __grid_constant__ ConvI8SPlan p, const uint4* __restrict__ wexp,
                const NextLayerArgs f)
{
    extern __shared__ __align__(128) uint8_t smem[];
    uint4* sWr = reinterpret_cast<uint4*>(smem + p.off_w);       // [nW][kSlices][2][Np]
    int* sPsum = reinterpret_cast<int*>(smem + p.off_psum);      // [kPsumRing][ppix]
    float* sLo = reinterpret_cast<float*>(smem + p.off_lo);
    float* sHi = reinterpret_cast<float*>(smem + p.off_hi);
    float4* sC = reinterpret_cast<float4*>(smem + p.off_c);
    uint64_t* bars = reinterpret_cast<uint64_t*>(smem + p.off_bar);
    uint64_t* a_empty = bars;           // [2] MMA -> ternarizers: the MMAs that read the code buffer are done
    uint64_t* acc_full = bars + 2;      // [2] MMA -> epilogue
    uint64_t* acc_empty = bars + 4;     // [2] epilogue -> MMA
    uint64_t* w_full = bars + 6;                    // [nW] expanders -> MMA: filter stage expanded
    uint64_t* w_empty = bars + 6 + kMaxWStages;     // [nW] MMA -> expanders: stage consumed
    uint64_t* a_full = bars + 6 + 2 * kMaxWStages;  // [2][kMaxGroups] ternarizers -> MMA: 32 channels of codes written
    uint32_t* slot = reinterpret_cast<uint32_t*>(smem + p.off_misc);
    volatile int* dead = reinterpret_cast<volatile int*>(smem + p.off_misc + 8);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int ngroup = p.Cp / 32;
    const int nstages = p.nK / kSlices;
    // this CTA's strip of rows, cut into equal tiles of at most RT rows, and its passes over the filter groups (all
    // of them, or the one group dealt to it)
    const int strip = p.split ? (int)blockIdx.x / p.npass : (int)blockIdx.x;
    const int pass0 = p.split ? (int)blockIdx.x % p.npass : 0;
    const int npass_cta = p.split ? 1 : p.npass;
    const int s0 = (int)((int64_t)strip * p.total_rows / p.nstrips);
    const int s1 = (int)((int64_t)(strip + 1) * p.total_rows / p.nstrips);
    const int ntile = (s1 - s0 + p.RT - 1) / p.RT;
    const int rt = ntile > 0 ? (s1 - s0 + ntile - 1) / ntile : 1;

    RTN_TL_INIT(conv_i8s)
    if (threadIdx.x == 0) RTN_TL(conv_i8s, 0);
    tc::pdl_trigger();
    if (warp == 0) tc::tmem_alloc(slot, p.tmem_cols);
    if (threadIdx.x == 32) {
        for (int i = 0; i < 2; ++i) {
            tc::mbar_init(&a_empty[i], 1);
            tc::mbar_init(&acc_full[i], 1);
            tc::mbar_init(&acc_empty[i], kEpiThreads);
        }
        for (int i = 0; i < kMaxWStages; ++i) { tc::mbar_init(&w_full[i], kPre ? 1 : kExpWarps); tc::mbar_init(&w_empty[i], 1); }
        for (int i = 0; i < 2 * kMaxGroups; ++i) tc::mbar_init(&a_full[i], kTernThreads);
        tc::mbar_init_fence();
        *dead = 0;
    }
    if constexpr (kPre) {
        // Per stage of the filter stream, the A windows of its four K = 32 slices (one 16-byte load for the issuing
        // thread).  A padding slice of the last packed block gets window 0 of the last group: its filter slice is
        // all zeros, so the instruction adds nothing and the issue loop needs no branch for it.
        uint4* sTab = reinterpret_cast<uint4*>(smem + p.off_tab);
        for (int i = threadIdx.x; i <= nstages; i += kThreads) {
            const int st = i < nstages ? i : nstages - 1;
            uint32_t e[kSlices];
            #pragma unroll
            for (int j = 0; j < kSlices; ++j) {
                const uint32_t v = p.tab_a[st * kSlices + j];
                e[j] = v == 0xFFFFFFFFu ? (uint32_t)(ngroup - 1) << 24 : v;
            }
            sTab[i] = make_uint4(e[0], e[1], e[2], e[3]);
        }
    }
    bool packed_in = false;
    if constexpr (kNext) packed_in = f.x_packed != nullptr;
    if constexpr (kNext) {
        // the next layer's threshold pair per column; columns past N code to 0
        float2* sT = reinterpret_cast<float2*>(smem + p.off_t);
        for (int n = threadIdx.x; n < p.Np; n += kThreads) {
            float2 t = make_float2(-INFINITY, INFINITY);
            if (f.out_packed != nullptr && n < a.N)
                t = make_float2(f.next_lo[f.n_next == 1 ? 0 : n], f.next_hi[f.n_next == 1 ? 0 : n]);
            sT[n] = t;
        }
    }
    for (int c = threadIdx.x; c < p.Cp && !packed_in; c += kThreads) {
        float lo = c < a.C ? a.t_lo[a.n_thr == 1 ? 0 : c] : -INFINITY;
        const float hi = c < a.C ? a.t_hi[a.n_thr == 1 ? 0 : c] : INFINITY;
        if (lo > hi) lo = nextafterf(hi, INFINITY);      // v < lo  <=>  v <= hi: -1 unless +1
        sLo[c] = lo;
        sHi[c] = hi;
    }
    {   // per-output-channel constants in double, rounded once:
        //   c1 = a_s*w_s, c2 = a_s*w_o, c3 = a_o*(w_s*S_w + K*w_o)     (K = C*kh*kw)
        const double a_s = a.ep.a_scale_val, a_o = a.ep.a_offset_val;
        for (int n = threadIdx.x; n < p.Np; n += kThreads) {
            float c1 = 0.f, c2 = 0.f, c3 = 0.f;
            if (n < a.N) {
                const double ws = a.ep.w_scale[a.ep.n_wparam == 1 ? 0 : n];
                const double wo = a.ep.w_offset[a.ep.n_wparam == 1 ? 0 : n];
                c1 = (float)(a_s * ws);
                c2 = (float)(a_s * wo);
                c3 = (float)(a_o * (ws * (double)a.w_sum[n] + (double)a.C * p.T * wo));
            }
            sC[n] = make_float4(c1, c2, c3, 0.f);
        }
    }
    tc::tc_fence_before_sync();
    __syncthreads();
    tc::tc_fence_after_sync();
    const uint32_t tmem = *slot;
    tc::pdl_wait();         // from here on: x, out (the set-up above read only the layer's parameters)
    if (threadIdx.x == 0) RTN_TL(conv_i8s, 1);

    if (warp >= 1 && warp < 1 + kTernWarps) {
        // ------------------------------------------------------------ ternarizers / epilogue
        // Ternarizing: item = (32-channel group, pixel of the tile's sequence), groups outer; a thread
        // arrives on a group's barrier when its next item lies beyond the group, so nobody idles at
        // a group's end.  Warps 4..11 then run the epilogue of the tile before: the tensor core works
        // on tile i while they ternarize tile i+1 (second code buffer) or write out tile i-1.
        const int tid = (warp - 1) * 32 + lane;
        const bool epi_warp = warp >= kEpiWarp0;
        const int64_t cs = (int64_t)a.H * a.W;
        const bool per_layer = a.n_thr == 1 && a.C == p.Cp;     // padding channels need their own (infinite) thresholds
        const float lo0 = packed_in ? 0.f : sLo[0], hi0 = packed_in ? 0.f : sHi[0];
        const int q = warp & 3, half = (warp - kEpiWarp0) >> 2;
        const int64_t ostride = (int64_t)a.Ho * a.Wo;
        const int nblk16 = (a.N + 15) / 16;
        for (int step = 0; step <= ntile; ++step) {
            if (step < ntile) {
                const int it = step, g = s0 + it * rt;
                const int nrows = min(rt, s1 - g);
            const int buf = p.nA == 2 ? (it & 1) : 0;
            const uint32_t use_ph = p.nA == 2 ? ((it >> 1) & 1) : (it & 1);
            uint4* sA = reinterpret_cast<uint4*>(smem + (buf ? p.off_a[1] : p.off_a[0]));      // [Cp/16][ppix]
            const int npix = (nrows + p.halo) * p.PW;
            int* psum = sPsum + (it & (kPsumRing - 1)) * p.ppix;
            role_wait(tid < 32, &a_empty[buf], use_ph ^ 1, a.status, dead, kTernBarrier, kTernThreads);
            if (tid == 0 && it < 8) RTN_TL(conv_i8s, 24 + 2 * it);
            for (int i = tid; i < p.ppix; i += kTernThreads) psum[i] = 0;
            asm volatile("bar.sync %0, %1;" ::"r"(kTernBarrier), "r"(kTernThreads) : "memory");
            uint64_t* full = &a_full[buf * kMaxGroups];
            int h = 0, pp = tid, arrived = 0;
            while (pp >= npix && h < ngroup) { pp -= npix; ++h; }
            for (; arrived < h && arrived < ngroup; ++arrived) tc::mbar_arrive(&full[arrived]);
            while (h < ngroup) {
                const uint32_t sl = fdiv((uint32_t)pp, p.div_pw);
                const int c = (int)((uint32_t)pp - sl * (uint32_t)p.PW) * p.istride - p.ipad;
                const uint32_t G = (uint32_t)g + sl;
                const uint32_t b = fdiv(G, p.div_ph);
                const int r = (int)(G - b * (uint32_t)p.PH) * p.istride - p.ipad;
                uint4 w0 = make_uint4(0, 0, 0, 0), w1 = make_uint4(0, 0, 0, 0);
                if (packed_in) {
                    // packed pixel rows: one word of each bit plane = the 32 codes of this (pixel, group)
                    if constexpr (kNext) {
                        if (b < (uint32_t)a.B && r >= 0 && r < a.H && c >= 0 && c < a.W) {
                            const int64_t row_bytes = (int64_t)((a.C + kBlockCodes - 1) / kBlockCodes) * kBlockBytes;
                            const uint32_t* blk = reinterpret_cast<const uint32_t*>(
                                f.x_packed + (((int64_t)b * a.H + r) * a.W + c) * row_bytes) + (h >> 2) * 8 + (h & 3);
                            uint32_t nz = __ldg(blk);
                            const uint32_t sg = __ldg(blk + 4);
                            if (h * 32 + 32 > a.C) nz &= (1u << (a.C - h * 32)) - 1u;      // positions past C code to 0
                            uint32_t o[8];
                            tc::unpack32(nz, sg, o);
                            w0 = make_uint4(o[0], o[1], o[2], o[3]);
                            w1 = make_uint4(o[4], o[5], o[6], o[7]);
                            const int sm = __popc(nz & sg) - __popc(nz & ~sg);
                            if (sm != 0) atomicAdd(&psum[pp], sm);
                        }
                    }
                } else
                if (b < (uint32_t)a.B && r >= 0 && r < a.H && c >= 0 && c < a.W) {
                    const float* src = a.x + (((int64_t)b * a.C + h * 32) * a.H + r) * a.W + c;
                    float v0[16], v1[16];
                    #pragma unroll
                    for (int e = 0; e < 16; ++e) {
                        v0[e] = (h * 32 + perm16(e) < a.C) ? __ldg(src + perm16(e) * cs) : 0.0f;
                        v1[e] = (h * 32 + 16 + perm16(e) < a.C) ? __ldg(src + (16 + perm16(e)) * cs) : 0.0f;
                    }
                    w0 = per_layer ? codes16<true>(v0, sLo, sHi, h * 32, lo0, hi0)
                                   : codes16<false>(v0, sLo, sHi, h * 32, lo0, hi0);
                    w1 = per_layer ? codes16<true>(v1, sLo, sHi, h * 32 + 16, lo0, hi0)
                                   : codes16<false>(v1, sLo, sHi, h * 32 + 16, lo0, hi0);
                    int s = __dp4a((int)w0.x, 0x01010101, __dp4a((int)w0.y, 0x01010101,
                            __dp4a((int)w0.z, 0x01010101, __dp4a((int)w0.w, 0x01010101, 0))));
                    s = __dp4a((int)w1.x, 0x01010101, __dp4a((int)w1.y, 0x01010101,
                        __dp4a((int)w1.z, 0x01010101, __dp4a((int)w1.w, 0x01010101, s))));
                    if (s != 0) atomicAdd(&psum[pp], s);
                }
                sA[(2 * h) * p.ppix + pp] = w0;
                sA[(2 * h + 1) * p.ppix + pp] = w1;
                pp += kTernThreads;
                while (pp >= npix && h < ngroup) { pp -= npix; ++h; }
                if (arrived < h) {
                    tc::fence_smem_to_async_proxy();
                    for (; arrived < h && arrived < ngroup; ++arrived) tc::mbar_arrive(&full[arrived]);
                }
            }
            if (tid == 0 && it < 8) RTN_TL(conv_i8s, 25 + 2 * it);
            }
            if (step >= 1 && epi_warp) {
                const int it = step - 1, g = s0 + it * rt;
                const int nrows = min(rt, s1 - g);
            const int ntm = (nrows * p.PW + kTileM - 1) / kTileM;
            const int* psum = sPsum + (it & (kPsumRing - 1)) * p.ppix;
          for (int pass = pass0; pass < pass0 + npass_cta; ++pass) {
            const int vt = it * npass_cta + (pass - pass0);             // the accumulators go round per (tile, pass)
            const int acc = p.nAcc == 2 ? (vt & 1) : 0;
            const uint32_t acc_ph = p.nAcc == 2 ? ((vt >> 1) & 1) : (vt & 1);
            const int slot_acc = acc;
            role_wait(warp == kEpiWarp0, &acc_full[slot_acc], acc_ph, a.status, dead, kEpiBarrier, kEpiThreads);
            const bool alive = !*dead;
            tc::tc_fence_after_sync();
            if (warp == kEpiWarp0 && lane == 0 && pass == pass0 && it < 8) RTN_TL(conv_i8s, 56 + 2 * it);
            const int pass_blocks = p.npass > 1 ? min(p.NpP / 16, nblk16 - pass * (p.NpP / 16)) : nblk16;
            const int pb_begin = half == 0 ? 0 : (pass_blocks + 1) / 2;
            const int pb_end = half == 0 ? (pass_blocks + 1) / 2 : pass_blocks;
            for (int tm = 0; tm < ntm; ++tm) {
                const uint32_t pl = (uint32_t)(tm * kTileM + q * 32 + lane);
                const uint32_t row = fdiv(pl, p.div_pw);
                const int wo = (int)(pl - row * (uint32_t)p.PW);
                const uint32_t G = (uint32_t)g + row;
                const uint32_t b = fdiv(G, p.div_ph);
                const int ho = (int)(G - b * (uint32_t)p.PH);
                const bool ok = alive && (int)row < nrows && b < (uint32_t)a.B && ho < a.Ho && wo < a.Wo;
                int n_inside = p.T, s_x = 0;
                if (ok) {
                    for (int t = 0; t < p.T; ++t) s_x += psum[pl + (t / a.kw) * p.PW + (t % a.kw)];
                    if (a.pad_mode == RTN_PAD_VALUE_ZERO) {
                        n_inside = 0;
                        for (int t = 0; t < p.T; ++t) {
                            const int h = ho * a.stride - a.pad + t / a.kw, v = wo * a.stride - a.pad + t % a.kw;
                            n_inside += (h >= 0 && h < a.H && v >= 0 && v < a.W);
                        }
                    }
                }
                const bool border = n_inside < p.T;
                const float fsx = (float)s_x;
                const uint32_t trow = tmem + ((uint32_t)(q * 32) << 16) + (uint32_t)((slot_acc * p.TM + tm) * p.NpP);
                float* optr = a.out + (((int64_t)b * a.N) * a.Ho + ho) * a.Wo + wo;
                int32_t* dptr = a.dbg_acc ? a.dbg_acc + (((int64_t)b * a.N) * a.Ho + ho) * a.Wo + wo : nullptr;
                // packed output: this pixel's row of N codes; the positions from the last computed block to the
                // end of the last 128-code block are zero-filled (first warp set, last pass)
                const int packed_cols = (a.N + kBlockCodes - 1) / kBlockCodes * kBlockCodes;
                uint8_t* out_row = nullptr;
                if constexpr (kNext) {
                    if (ok && f.out_packed != nullptr) {
                        out_row = f.out_packed + (((int64_t)b * a.Ho + ho) * a.Wo + wo) * (int64_t)(packed_cols / 4);
                        if (half == 0 && pass == p.npass - 1) zero_fill_packed_row(out_row, nblk16 * 16, packed_cols);
                    }
                }
                for (int blk = pb_begin; blk < pb_end; ++blk) {
                    uint32_t v[16];
                    tc::tmem_ld16(trow + (uint32_t)(blk * 16), v);
                    tc::tmem_ld_wait();
                    if (!ok) continue;
                    const int n0 = pass * p.NpP + blk * 16;
                    if constexpr (kNext) {
                        uint32_t nzb, sgb;
                        const bool codes = out_row != nullptr && n0 < packed_cols;
                        next_layer_block16(a, f, v, sC + n0, reinterpret_cast<const float2*>(smem + p.off_t) + n0, fsx,
                                           border, p.T, ho, wo, n_inside, n0,
                                           (((int64_t)b * a.N) * a.Ho + ho) * a.Wo + wo + (int64_t)n0 * ostride, ostride,
                                           codes, nzb, sgb);
                        if (codes) {
                            uint8_t* dst = out_row + (n0 >> 7) * kBlockBytes + ((n0 & 127) >> 3);
                            *reinterpret_cast<uint16_t*>(dst) = (uint16_t)nzb;
                            *reinterpret_cast<uint16_t*>(dst + 16) = (uint16_t)sgb;
                        }
                        continue;
                    }
                    if (!border && dptr == nullptr && n0 + 16 <= a.N) {
                        // all sixteen results first, then the stores: a shared-memory load of the next column's
                        // constants may not be moved above a global store the compiler cannot tell apart from it, so
                        // with load and store alternating every column waited for the one before
                        float r[16];
                        #pragma unroll
                        for (int j = 0; j < 16; ++j) {
                            const float4 c = sC[n0 + j];
                            r[j] = fmaf(c.x, (float)(int)v[j], fmaf(c.y, fsx, c.z));
                        }
                        float* o = optr + (int64_t)n0 * ostride;
                        #pragma unroll
                        for (int j = 0; j < 16; ++j, o += ostride) *o = r[j];
                    } else {
                        #pragma unroll
                        for (int j = 0; j < 16; ++j) {
                            const int n = n0 + j;
                            if (n >= a.N) continue;
                            const int s_xw = (int)v[j];
                            const float4 c = sC[n];
                            float c3 = c.z;
                            if (border) {
                                // value-zero padding at an image border: S_w and K over inside taps only
                                int s_w = 0;
                                for (int t = 0; t < p.T; ++t) {
                                    const int h = ho * a.stride - a.pad + t / a.kw, vv = wo * a.stride - a.pad + t % a.kw;
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
            tc::tc_fence_before_sync();
            tc::mbar_arrive(&acc_empty[acc]);
            if (warp == kEpiWarp0 && lane == 0 && pass == pass0 + npass_cta - 1 && it < 8) RTN_TL(conv_i8s, 57 + 2 * it);
          }
            }
        }
    } else if (warp >= kExpWarp0 && warp < kExpWarp0 + kExpWarps) {
        // ------------------------------------------------------------ filter expanders
        // thread = filter row; a stage = one packed block of the row (four K = 32 slices).  The
        // planes of the next two stages are in flight while this one expands.
        if constexpr (kPre) {
            // one thread streams the expanded stages into the ring
            if (warp == kExpWarp0 && lane == 0) {
                const uint32_t stage_bytes = (uint32_t)p.NpP * 32u * kSlices;
                const uint32_t ring = tc::smem_addr(sWr);
                uint32_t wcount = 0;
                bool alive = true;
                for (int it = 0; it < ntile && alive; ++it)
                    for (int s = pass0 * nstages; s < (pass0 + npass_cta) * nstages; ++s, ++wcount) {      // pass after pass
                        const uint32_t st = wcount % (uint32_t)p.nW;
                        if (!wait_or_die(&w_empty[st], ((wcount / (uint32_t)p.nW) & 1) ^ 1, a.status, dead)) { alive = false; break; }
                        tc::mbar_arrive_expect_tx(&w_full[st], stage_bytes);
                        tc::bulk_copy_g2s(ring + st * stage_bytes, wexp + (size_t)s * (stage_bytes / 16), stage_bytes, &w_full[st]);
                    }
            }
        } else {
        const int tid = threadIdx.x - kExpWarp0 * 32;
        const int cwords = p.Cp / 32;
        const int64_t row_blocks = ((int64_t)p.T * cwords + 3) / 4;
        const uint4* Wrow = tid < a.N ? reinterpret_cast<const uint4*>(a.w_packed) + (int64_t)tid * row_blocks * 2
                                      : nullptr;
        const int cblocks = cwords / kSlices;
        auto block_of = [&](int st) {
            if (!p.blocks_major) return st;
            const int cb = (int)fdiv((uint32_t)st, p.div_T), t = st - cb * p.T;
            return t * cblocks + cb;
        };
        uint32_t wcount = 0;
        for (int it = 0; it < ntile; ++it) {
            uint4 nz1 = make_uint4(0, 0, 0, 0), sg1 = nz1, nz2 = nz1, sg2 = nz1;
            if (Wrow != nullptr) {
                const int b0 = block_of(0);
                nz1 = __ldg(Wrow + 2 * b0); sg1 = __ldg(Wrow + 2 * b0 + 1);
                if (nstages > 1) { const int b1 = block_of(1); nz2 = __ldg(Wrow + 2 * b1); sg2 = __ldg(Wrow + 2 * b1 + 1); }
            }
            for (int s = 0; s < nstages; ++s, ++wcount) {
                const uint4 nzv = nz1, sgv = sg1;
                nz1 = nz2; sg1 = sg2;
                if (Wrow != nullptr && s + 2 < nstages) {
                    const int b2 = block_of(s + 2);
                    nz2 = __ldg(Wrow + 2 * b2); sg2 = __ldg(Wrow + 2 * b2 + 1);
                }
                const uint32_t st = wcount % (uint32_t)p.nW;
                role_wait(tid < 32, &w_empty[st], ((wcount / (uint32_t)p.nW) & 1) ^ 1, a.status, dead, kExpBarrier,
                          kExpThreads);
                if (tid < p.Np) {
                    uint4* dst = sWr + (size_t)st * kSlices * 2 * p.Np + tid;
                    uint32_t o[8];
                    tc::unpack32(nzv.x, sgv.x, o);
                    dst[0 * p.Np] = make_uint4(o[0], o[1], o[2], o[3]);
                    dst[1 * p.Np] = make_uint4(o[4], o[5], o[6], o[7]);
                    tc::unpack32(nzv.y, sgv.y, o);
                    dst[2 * p.Np] = make_uint4(o[0], o[1], o[2], o[3]);
                    dst[3 * p.Np] = make_uint4(o[4], o[5], o[6], o[7]);
                    tc::unpack32(nzv.z, sgv.z, o);
                    dst[4 * p.Np] = make_uint4(o[0], o[1], o[2], o[3]);
                    dst[5 * p.Np] = make_uint4(o[4], o[5], o[6], o[7]);
                    tc::unpack32(nzv.w, sgv.w, o);
                    dst[6 * p.Np] = make_uint4(o[0], o[1], o[2], o[3]);
                    dst[7 * p.Np] = make_uint4(o[4], o[5], o[6], o[7]);
                }
                tc::fence_smem_to_async_proxy();
                __syncwarp();
                if (lane == 0) tc::mbar_arrive(&w_full[st]);
            }
        }
        }
    } else if (warp == 0) {
        // ------------------------------------------------------------ MMA issue (one thread)
        // The tensor core's queue is short, so whatever the issuing thread does between two MMAs is
        // tensor-core idle time: the A offsets of a stage are fetched one stage ahead.
        if (lane == 0) {
            const uint32_t idesc = tc::idesc_i8(kTileM, (uint32_t)p.NpP);
            const uint64_t desc_hi = (uint64_t)((128u >> 4) | (1u << 14)) << 32;
            const uint32_t a_lbo_field = (((uint32_t)p.ppix * 16) >> 4) << 16;
            const uint32_t w16 = (tc::smem_addr(sWr) >> 4) + ((((uint32_t)p.NpP * 16) >> 4) << 16);
            const uint32_t wslice16 = ((uint32_t)p.NpP * 32) >> 4;
            const uint32_t wstage16 = wslice16 * kSlices;
            uint32_t wcount = 0;
            int it = 0;
            bool alive = true;
            if constexpr (kPre) {
                // Filters streamed from scratch: slices come 32-channel group by group, so the groups a stage needs
                // are a count; the stage's four A windows arrive with one shared-memory load, fetched a stage ahead;
                // ring slot, phase and accumulator set advance by increments; the next stage's barrier is tested
                // before this stage's MMAs go out.  What is left between two tensor-core instructions of a stage is
                // one or two additions (a division, a chain of table look-ups and a branch per slice were 0.85 us
                // per stage of eight instructions that the tensor core runs in 0.3 us).
                const uint4* sTab = reinterpret_cast<const uint4*>(smem + p.off_tab);
                uint32_t st = 0, wph = 0;           // filter ring slot and its phase
                bool have = false;                  // slot st is known to be full
                uint32_t acc = 0, acc_ph = 0;       // accumulator set and its phase
                for (int g = s0; g < s1 && alive; g += rt, ++it) {
                    const int buf = p.nA == 2 ? (it & 1) : 0;
                    const uint32_t use_ph = p.nA == 2 ? ((it >> 1) & 1) : (it & 1);
                    const bool two = min(rt, s1 - g) * p.PW > kTileM;      // the tile has a second 128-pixel sub-tile
                    const uint32_t a16 = (tc::smem_addr(smem + (buf ? p.off_a[1] : p.off_a[0])) >> 4) + a_lbo_field;
                    uint64_t* full = &a_full[buf * kMaxGroups];
                    uint32_t nready = 0;            // 32-channel groups whose codes are known to be written
                    for (int pass = 0; pass < npass_cta && alive; ++pass) {
                        alive = wait_or_die(&acc_empty[acc], acc_ph ^ 1, a.status, dead);
                        if (!alive) break;
                        const uint32_t d0 = tmem + acc * (uint32_t)(p.TM * p.NpP), d1 = d0 + (uint32_t)p.NpP;
                        uint4 cur = sTab[0];
                        for (int sg = 0; sg < nstages; ++sg) {
                            const uint4 nxt = sTab[sg + 1];
                            if (!have && !wait_or_die(&w_full[st], wph, a.status, dead)) { alive = false; break; }
                            const uint32_t hmax = cur.w >> 24;
                            while (nready <= hmax && alive) {
                                alive = wait_or_die(&full[nready], use_ph, a.status, dead);
                                ++nready;
                            }
                            if (!alive) break;
                            tc::tc_fence_after_sync();
                            const uint32_t st_cur = st;
                            if (++st == (uint32_t)p.nW) { st = 0; wph ^= 1u; }
                            have = tc::mbar_test(&w_full[st], wph);
                            const uint32_t b0 = w16 + st_cur * wstage16, b1 = b0 + wslice16, b2 = b1 + wslice16, b3 = b2 + wslice16;
                            const uint32_t a0 = a16 + (cur.x & 0xFFFFFFu), a1 = a16 + (cur.y & 0xFFFFFFu);
                            const uint32_t a2 = a16 + (cur.z & 0xFFFFFFu), a3 = a16 + (cur.w & 0xFFFFFFu);
                            if (sg == 0 && pass == 0 && it < 8) RTN_TL(conv_i8s, 40 + 2 * it);
                            if (two) {
                                tc::mma_i8_ss(d0, desc_hi | a0, desc_hi | b0, idesc, sg > 0);
                                tc::mma_i8_ss(d1, desc_hi | (a0 + (uint32_t)kTileM), desc_hi | b0, idesc, sg > 0);
                                tc::mma_i8_ss_acc(d0, desc_hi | a1, desc_hi | b1, idesc);
                                tc::mma_i8_ss_acc(d1, desc_hi | (a1 + (uint32_t)kTileM), desc_hi | b1, idesc);
                                tc::mma_i8_ss_acc(d0, desc_hi | a2, desc_hi | b2, idesc);
                                tc::mma_i8_ss_acc(d1, desc_hi | (a2 + (uint32_t)kTileM), desc_hi | b2, idesc);
                                tc::mma_i8_ss_acc(d0, desc_hi | a3, desc_hi | b3, idesc);
                                tc::mma_i8_ss_acc(d1, desc_hi | (a3 + (uint32_t)kTileM), desc_hi | b3, idesc);
                            } else {
                                tc::mma_i8_ss(d0, desc_hi | a0, desc_hi | b0, idesc, sg > 0);
                                tc::mma_i8_ss_acc(d0, desc_hi | a1, desc_hi | b1, idesc);
                                tc::mma_i8_ss_acc(d0, desc_hi | a2, desc_hi | b2, idesc);
                                tc::mma_i8_ss_acc(d0, desc_hi | a3, desc_hi | b3, idesc);
                            }
                            tc::mma_commit(&w_empty[st_cur]);
                            cur = nxt;
                        }
                        if (!alive) break;
                        tc::mma_commit(&acc_full[acc]);      // this pass's accumulators are complete
                        if (pass == npass_cta - 1 && it < 8) RTN_TL(conv_i8s, 41 + 2 * it);
                        if (p.nAcc == 2) { acc ^= 1u; if (acc == 0) acc_ph ^= 1u; } else acc_ph ^= 1u;
                    }
                    if (!alive) break;
                    tc::mma_commit(&a_empty[buf]);
                }
            } else
            for (int g = s0; g < s1 && alive; g += rt, ++it) {
                const int buf = p.nA == 2 ? (it & 1) : 0;
                const uint32_t use_ph = p.nA == 2 ? ((it >> 1) & 1) : (it & 1);
                const int nrows = min(rt, s1 - g);
                const int ntm = (nrows * p.PW + kTileM - 1) / kTileM;
                const uint32_t a16 = (tc::smem_addr(smem + (buf ? p.off_a[1] : p.off_a[0])) >> 4) + a_lbo_field;
                uint64_t* full = &a_full[buf * kMaxGroups];
                uint32_t ready = 0;             // 32-channel groups whose codes are known to be written
              for (int pass = 0; pass < npass_cta && alive; ++pass) {
                const int vt = it * npass_cta + pass;
                const int slot_acc = p.nAcc == 2 ? (vt & 1) : 0;
                const uint32_t acc_ph = p.nAcc == 2 ? ((vt >> 1) & 1) : (vt & 1);
                alive = wait_or_die(&acc_empty[slot_acc], acc_ph ^ 1, a.status, dead);
                if (!alive) break;
                uint32_t ta[kSlices], tn[kSlices];
                #pragma unroll
                for (int j = 0; j < kSlices; ++j) tn[j] = p.tab_a[j];
                bool accum = false;
                for (int s = 0; s < nstages && alive; ++s, ++wcount) {
                    #pragma unroll
                    for (int j = 0; j < kSlices; ++j) {
                        ta[j] = tn[j];
                        tn[j] = p.tab_a[min((s + 1) * kSlices + j, p.nK - 1)];
                    }
                    const uint32_t st = wcount % (uint32_t)p.nW;
                    if (!wait_or_die(&w_full[st], (wcount / (uint32_t)p.nW) & 1, a.status, dead)) { alive = false; break; }
                    tc::tc_fence_after_sync();
                    #pragma unroll
                    for (int j = 0; j < kSlices; ++j) {
                        if (ta[j] != 0xFFFFFFFFu && alive) {
                            const uint32_t h = ta[j] >> 24;
                            if (!((ready >> h) & 1u)) {
                                alive = wait_or_die(&full[h], use_ph, a.status, dead);
                                tc::tc_fence_after_sync();
                                ready |= 1u << h;
                            }
                            if (alive) {
                                const uint64_t bd = desc_hi | (uint64_t)(w16 + st * wstage16 + (uint32_t)j * wslice16);
                                const uint32_t aw = a16 + (ta[j] & 0xFFFFFFu);
                                if (!accum && pass == 0 && it < 8) RTN_TL(conv_i8s, 40 + 2 * it);
                                tc::mma_i8_ss(tmem + (uint32_t)((slot_acc * p.TM) * p.NpP), desc_hi | (uint64_t)aw, bd, idesc, accum);
                                if (ntm == 2)
                                    tc::mma_i8_ss(tmem + (uint32_t)((slot_acc * p.TM + 1) * p.NpP),
                                                  desc_hi | (uint64_t)(aw + (uint32_t)kTileM), bd, idesc, accum);
                                accum = true;
                            }
                        }
                    }
                    if (alive) tc::mma_commit(&w_empty[st]);
                }
                if (alive) tc::mma_commit(&acc_full[slot_acc]);      // this pass's accumulators are complete
                if (pass == npass_cta - 1 && it < 8) RTN_TL(conv_i8s, 41 + 2 * it);
              }
                if (!alive) break;
                tc::mma_commit(&a_empty[buf]);
            }
        }
    }
    tc::tc_fence_before_sync();
    __syncthreads();
    if (warp == 0) tc::tmem_dealloc(tmem, p.tmem_cols);
    if (threadIdx.x == 0) RTN_TL(conv_i8s, 4);
}

}  // namespace

bool conv_i8s_supported(const ConvArgs& c)
{
    ConvI8SPlan p;
    return make_plan_s(c, p, device_sm_count());
}

// A filter stream of four stages or more is expanded once into scratch (an extra small kernel).
static bool pre_expand(const ConvI8SPlan& p) { return p.pre != 0; }

int conv_i8s_launches(const ConvArgs& c)
{
    ConvI8SPlan p;
    if (!make_plan_s(c, p, device_sm_count())) return 0;
    return pre_expand(p) ? 2 : 1;
}

template <bool kNext>
static cudaError_t launch_i8s_mode(const ConvArgs& c, const NextLayerArgs& f, cudaStream_t s)
{
    ConvI8SPlan p;
    if (!make_plan_s(c, p, device_sm_count(), kNext)) return cudaErrorInvalidConfiguration;
    if (!pre_expand(p)) {
        cudaError_t e = cudaFuncSetAttribute(conv_i8s_kernel<false, kNext>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                             (int)p.smem_bytes);
        if (e != cudaSuccess) return e;
        return launch_pdl(conv_i8s_kernel<false, kNext>, dim3((unsigned)p.grid), dim3(kThreads), p.smem_bytes, s, c, p,
                          (const uint4*)nullptr, f);
    }
    // scratch from the stream-ordered allocator, given back right after the two launches, in stream order
    const int nstages = p.nK / kSlices;
    const size_t bytes = (size_t)p.npass * nstages * p.NpP * 32 * kSlices;
    void* scratch = nullptr;
    cudaError_t e = cudaMallocAsync(&scratch, bytes, s);
    if (e != cudaSuccess) return e;
    const int64_t items = (int64_t)p.npass * nstages * kSlices * p.NpP;
    conv_expand_filters_kernel<<<(unsigned)((items + 255) / 256), 256, 0, s>>>(c, p, reinterpret_cast<uint4*>(scratch));
    e = cudaGetLastError();
    if (e == cudaSuccess)
        e = cudaFuncSetAttribute(conv_i8s_kernel<true, kNext>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                 (int)p.smem_bytes);
    if (e == cudaSuccess)
        e = launch_pdl(conv_i8s_kernel<true, kNext>, dim3((unsigned)p.grid), dim3(kThreads), p.smem_bytes, s, c, p,
                       (const uint4*)scratch, f);
    const cudaError_t e2 = cudaFreeAsync(scratch, s);
    return e != cudaSuccess ? e : e2;
}

cudaError_t launch_conv_i8s(const ConvArgs& c, cudaStream_t s) { return launch_i8s_mode<false>(c, NextLayerArgs{}, s); }

// Rough time of this variant for a shape, in microseconds (negative: not taken), for the choice between it
// and the variant that keeps a share of the filter bank resident per CTA.
double conv_i8s_estimate_us(const ConvArgs& c)
{
    ConvI8SPlan p;
    if (!make_plan_s(c, p, device_sm_count())) return -1.0;
    return plan_estimate_us(p);
}

// The same kernels with the hand-over to the next layer (and, optionally, packed input).
bool conv_i8s_next_supported(const ConvArgs& c)
{
    ConvI8SPlan p;
    return make_plan_s(c, p, device_sm_count(), true);
}
int conv_i8s_next_launches(const ConvArgs& c)
{
    ConvI8SPlan p;
    if (!make_plan_s(c, p, device_sm_count(), true)) return 0;
    return pre_expand(p) ? 2 : 1;
}
cudaError_t launch_conv_i8s_next(const ConvArgs& c, const NextLayerArgs& f, cudaStream_t s)
{
    return launch_i8s_mode<true>(c, f, s);
}

}  // namespace rtn
