// Ternary conv2d, tensor-core variant for the layers the other two cannot take: more than 256 filters
// (e.g. 512 -> 512, 3x3) and strided filters larger than 1x1 (e.g. 3x3 stride 2).  Two kernels and a
// scratch buffer of int8 codes.  (On 256 -> 256, 3x3 it runs at 44 us against 38 us of the streamed-filter kernel, which
// therefore keeps that shape.)
//
//   conv_codes_kernel   ternarizes the fp32 NCHW input once (Eq. 3) into int8 codes {-1,0,+1} laid out
//                       [16-channel chunk][padded pixel][16 B] over the whole batch, zero padding
//                       included, plus the per-pixel code sum over all channels.  4 B read and
//                       about 1 B written per value: a stream through HBM.
//   conv_i8r_kernel     implicit GEMM on the codes.  The filter bank is SPLIT over CTAs: a CTA keeps
//                       the int8 expansion of N/S filters (all taps, all channels) resident in shared
//                       memory for its whole life and walks pixel tiles; the S CTAs of a tile each
//                       produce their share of the output channels.  Nothing is expanded in the main
//                       loop (a streamed filter bank costs a quarter of the SM's integer pipe per
//                       tile and paces the tensor core) and the fp32 input is ternarized once, not
//                       once per filter group.
//
// The code layout in the scratch buffer is the shared-memory operand layout, so a tile's window of
// one 16-channel chunk is one contiguous run of bytes: the producer moves it with one bulk
// asynchronous copy (cp.async.bulk, completion counted on an mbarrier; no tensor map, no multicast).
// Shifted-window implicit GEMM as in the other conv kernels: tap (i, j) reads the same rows of
// shared memory from a start shifted by i*PW + j pixels.  For stride 2 the code kernel writes the
// four phase images of the padded input (even/odd rows x even/odd columns) one after the other: tap
// (i, j) reads phase (i mod 2, j mod 2) shifted by (i div 2, j div 2), a stride-1 window again.  K loop: 32-channel group outer, tap inner;
// unit of the pipeline = (tile, group) = two chunk windows in one ring slot, 9 MMAs for a 3x3 filter.
// S_x of a pixel = sum over the taps of the per-pixel code sums (read from the scratch buffer in
// the epilogue), so all accumulator columns are output channels.
//
// Roles of conv_i8r_kernel (384 threads): warp 0 issues MMAs (one thread), warp 1 issues the bulk
// copies (one thread), warps 4..11 epilogue; all threads expand the CTA's filters at set-up, which
// overlaps the code kernel through programmatic dependent launch.
#include "rtn_internal.cuh"
#include "rtn_tcgen05.cuh"
#include "rtn_conv_i8_common.cuh"
#include "rtn_timeline.cuh"

// Timeline slots of conv_i8r_kernel (instrumented build only): 0 kernel entry, 1 set-up done (filters expanded, the code
// kernel finished), 4 kernel end; per tile i < 8 of the CTA: 8+2i / 9+2i producer issues the first / last slot, 40+2i / 41+2i
// first slot ready for the tensor core / accumulators committed, 56+2i / 57+2i epilogue begins / ends.
RTN_TL_DEFINE(conv_i8r)

namespace rtn {

namespace {

using namespace conv_detail;

constexpr int kTileM = 128;
constexpr int kEpiWarp0 = 4;
constexpr int kEpiWarps = 8;
constexpr int kEpiThreads = kEpiWarps * 32;
constexpr int kThreads = (kEpiWarp0 + kEpiWarps) * 32;
constexpr int kMaxSlots = 16;
constexpr int kMaxAcc = 4;
constexpr int kMaxTaps = 25;
constexpr int kMaxSplit = 32;                          // filter groups at most
constexpr size_t kSmemLimit = 220 * 1024;
constexpr int kEpiBarrier = 1;
constexpr int kCodePixels = 64;                        // pixels per block of the code kernel
constexpr int kCodeGroups = 8;                         // 32-channel groups it works on at a time

struct ConvI8RPlan {
    int PW, PH;            // row length / rows per image of a phase image (the padded image for stride 1)
    int Cp, T, halo, RT;   // channels rounded to 32, taps, (kh-1)/stride, rows per tile
    int ppix;              // pixels of a window: 128 + halo*PW + (kw-1)/stride, rounded up to 8
    int nph;               // phase images some tap reads (1 for stride 1; up to 4 for stride 2)
    int ph_r[4], ph_c[4];  // their row / column phases
    int total_rows, ntiles;
    int S, Nq;             // filter groups; filters per group (multiple of 16)
    int cpg, grid;         // CTAs per filter group; grid = S * cpg
    int ngroup;            // 32-channel groups
    int gps;               // groups per ring slot (2 when their number is even: fewer hand-offs)
    int nslots, nAcc;
    uint32_t tmem_cols;
    int64_t Ptot, Pstride; // padded pixels of the batch; pixels per chunk row of the scratch (with slack)
    FastDiv div_pw, div_ph, div_nq, div_cw;
    uint32_t off_w, off_c, off_t, off_bar, off_misc, off_slot, slot_bytes;
    size_t smem_bytes;
    size_t codes_bytes, scratch_bytes;     // scratch = codes, then the per-pixel sums
    uint32_t tap_shift[kMaxTaps];          // start of the tap's A window inside a slot, 16-byte units
    uint32_t tap_psum[kMaxTaps];           // the tap's offset into the per-pixel sums
};

bool make_plan_r(const ConvArgs& c, ConvI8RPlan& p, int sms, bool fused = false)
{
    if (c.stride < 1 || c.Ho <= 0 || c.Wo <= 0) return false;
    p.T = c.kh * c.kw;
    if (p.T > kMaxTaps) return false;
    // Stride s: the padded image splits into s*s phase images (rows = a mod s, columns = b mod s);
    // tap (i, j) reads phase (i mod s, j mod s) at the output pixel shifted by (i div s, j div s), so
    // inside a phase image the convolution has stride 1 and the shifted-window scheme applies.
    const int st = c.stride;
    p.nph = 0;
    int ph_of_tap[kMaxTaps];
    for (int t = 0; t < p.T; ++t) {
        const int a = (t / c.kw) % st, b = (t % c.kw) % st;
        int w = -1;
        for (int k = 0; k < p.nph; ++k) if (p.ph_r[k] == a && p.ph_c[k] == b) w = k;
        if (w < 0) {
            if (p.nph == 4) return false;
            w = p.nph++;
            p.ph_r[w] = a; p.ph_c[w] = b;
        }
        ph_of_tap[t] = w;
    }
    p.PW = (c.W + 2 * c.pad + st - 1) / st;
    p.PH = (c.H + 2 * c.pad + st - 1) / st;
    if (p.PW > kTileM || p.PH > 2048) return false;
    if ((int64_t)c.B * p.PH > (1 << 20)) return false;
    p.Cp = (c.C + 31) / 32 * 32;
    p.ngroup = p.Cp / 32;
    if (p.ngroup > 16) return false;
    p.halo = (c.kh - 1) / st;
    p.RT = kTileM / p.PW;
    p.ppix = (kTileM + p.halo * p.PW + (c.kw - 1) / st + 7) / 8 * 8;
    p.total_rows = c.B * p.PH;
    p.ntiles = (p.total_rows + p.RT - 1) / p.RT;
    p.Ptot = (int64_t)p.total_rows * p.PW;
    p.Pstride = p.Ptot + p.ppix;
    if ((int64_t)p.nph * p.Pstride >= (int64_t(1) << 31)) return false;
    p.gps = (p.ngroup % 2 == 0 && p.nph == 1) ? 2 : 1;
    p.slot_bytes = (uint32_t)p.nph * (uint32_t)p.gps * 2u * (uint32_t)p.ppix * 16u;
    p.div_pw = make_fastdiv((uint32_t)p.PW);
    p.div_ph = make_fastdiv((uint32_t)p.PH);
    p.div_cw = make_fastdiv((uint32_t)p.ngroup);
    for (int t = 0; t < p.T; ++t) {
        const uint32_t shift = (uint32_t)(((t / c.kw) / st) * p.PW + (t % c.kw) / st);
        p.tap_shift[t] = (uint32_t)ph_of_tap[t] * (uint32_t)(2 * p.gps * p.ppix) + shift;
        p.tap_psum[t] = (uint32_t)((int64_t)ph_of_tap[t] * p.Pstride) + shift;
    }
    // fewest filter groups whose share of the bank leaves room for a ring of at least three slots
    for (p.S = 1; p.S <= kMaxSplit; p.S *= 2) {
        if (p.S > sms) return false;
        p.Nq = ((c.N + p.S - 1) / p.S + 15) / 16 * 16;
        if (p.Nq > 256) continue;
        uint32_t o = 0;
        p.off_w = o;    o += (uint32_t)p.T * (uint32_t)(p.Cp / 16) * (uint32_t)p.Nq * 16u;
        p.off_c = o;    o += (uint32_t)p.Nq * 16u;
        p.off_t = o;    o += fused ? (uint32_t)p.Nq * 8u : 0u;     // next layer's {t_lo, t_hi} per column
        p.off_bar = o;  o += (2 * kMaxSlots + 2 * kMaxAcc + 1) * 8;
        p.off_misc = o; o += 16;
        o = (o + 127) / 128 * 128;
        p.off_slot = o;
        if (o >= kSmemLimit) continue;
        int ns = (int)((kSmemLimit - o) / p.slot_bytes);
        if (ns > kMaxSlots) ns = kMaxSlots;
        if (ns < 3) continue;
        p.nslots = ns;
        p.smem_bytes = o + (size_t)ns * p.slot_bytes;
        break;
    }
    if (p.S > kMaxSplit) return false;
    p.div_nq = make_fastdiv((uint32_t)p.Nq);
    p.cpg = sms / p.S;
    if (p.cpg > p.ntiles) p.cpg = p.ntiles;
    if (p.cpg < 1) return false;
    p.grid = p.S * p.cpg;
    p.nAcc = 512 / p.Nq < kMaxAcc ? 512 / p.Nq : kMaxAcc;
    uint32_t cols = 32;
    while (cols < (uint32_t)(p.nAcc * p.Nq)) cols *= 2;
    p.tmem_cols = cols;
    p.codes_bytes = (size_t)p.nph * (size_t)(p.Cp / 16) * (size_t)p.Pstride * 16;
    p.scratch_bytes = p.codes_bytes + ((size_t)p.nph * (size_t)p.Pstride * 4 + 255) / 256 * 256;
    return true;
}

// ------------------------------------------------------------------------------------------------
// Kernel 1: fp32 NCHW -> int8 codes [chunk][padded pixel][16 B] + per-pixel code sums.
// Block = 64 consecutive padded pixels x up to 8 channel groups; lanes run along pixels, so the
// loads of one channel are coalesced along an image row and the 16-byte code stores are contiguous.
// ------------------------------------------------------------------------------------------------
__global__ void __launch_bounds__(kCodePixels * kCodeGroups)
conv_codes_kernel(const ConvArgs a, const __grid_constant__ ConvI8RPlan p, uint4* __restrict__ codes,
                  int* __restrict__ psum)
{
    extern __shared__ __align__(16) uint8_t smem_c[];
    float* sLo = reinterpret_cast<float*>(smem_c);
    float* sHi = sLo + p.Cp;
    int* sSum = reinterpret_cast<int*>(sHi + p.Cp);            // [kCodeGroups][kCodePixels]
    tc::pdl_trigger();          // the contraction kernel may start its set-up (it reads no codes there)
    for (int c = threadIdx.x; c < p.Cp; c += blockDim.x) {
        float lo = c < a.C ? a.t_lo[a.n_thr == 1 ? 0 : c] : -INFINITY;
        const float hi = c < a.C ? a.t_hi[a.n_thr == 1 ? 0 : c] : INFINITY;
        if (lo > hi) lo = nextafterf(hi, INFINITY);      // v < lo  <=>  v <= hi: -1 unless +1
        sLo[c] = lo;
        sHi[c] = hi;
    }
    __syncthreads();
    const int px = threadIdx.x % kCodePixels, gi = threadIdx.x / kCodePixels;
    const int64_t P = (int64_t)blockIdx.x * kCodePixels + px;
    const int w = blockIdx.y;                               // phase image
    codes += (int64_t)w * (p.Cp / 16) * p.Pstride;
    psum += (int64_t)w * p.Pstride;
    const bool per_layer = a.n_thr == 1 && a.C == p.Cp;     // padding channels need their own (infinite) thresholds
    const float lo0 = sLo[0], hi0 = sHi[0];
    const int64_t cs = (int64_t)a.H * a.W;
    // padded pixel -> (image, row, column) of the input, if any
    bool inside = false;
    const float* src0 = nullptr;
    if (P < p.Ptot) {
        const uint32_t G = fdiv((uint32_t)P, p.div_pw);
        const int col = (int)((uint32_t)P - G * (uint32_t)p.PW) * a.stride + p.ph_c[w] - a.pad;
        const uint32_t b = fdiv(G, p.div_ph);
        const int r = (int)(G - b * (uint32_t)p.PH) * a.stride + p.ph_r[w] - a.pad;
        inside = r >= 0 && r < a.H && col >= 0 && col < a.W;
        if (inside) src0 = a.x + (((int64_t)b * a.C) * a.H + r) * a.W + col;
    }
    int sum = 0;
    for (int h = gi; h < p.ngroup; h += kCodeGroups) {
        uint4 w0 = make_uint4(0, 0, 0, 0), w1 = make_uint4(0, 0, 0, 0);
        if (inside) {
            const float* src = src0 + (int64_t)(h * 32) * cs;
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
            sum = __dp4a((int)w0.x, 0x01010101, __dp4a((int)w0.y, 0x01010101,
                  __dp4a((int)w0.z, 0x01010101, __dp4a((int)w0.w, 0x01010101, sum))));
            sum = __dp4a((int)w1.x, 0x01010101, __dp4a((int)w1.y, 0x01010101,
                  __dp4a((int)w1.z, 0x01010101, __dp4a((int)w1.w, 0x01010101, sum))));
        }
        if (P < p.Pstride) {
            codes[(int64_t)(2 * h) * p.Pstride + P] = w0;
            codes[(int64_t)(2 * h + 1) * p.Pstride + P] = w1;
        }
    }
    sSum[gi * kCodePixels + px] = sum;
    __syncthreads();
    if (gi == 0 && P < p.Pstride) {
        int s = 0;
        for (int k = 0; k < kCodeGroups; ++k) s += sSum[k * kCodePixels + px];
        psum[P] = s;
    }
}

// Kernel 1 for an input that arrives as packed pixel rows (the layer before wrote them from its
// epilogue, or rtn_ternarize_pack_act did): bit planes -> the same int8 code layout and per-pixel sums.
// 0.25 B read and about 1 B written per value.  Same block shape: lanes run along pixels, so the
// 16-byte code stores of a warp are contiguous; the word loads of a warp touch 32 pixel rows whose
// other words the block's other channel groups read (served by L1).
__global__ void __launch_bounds__(kCodePixels * kCodeGroups)
conv_codes_packed_kernel(const ConvArgs a, const __grid_constant__ ConvI8RPlan p,
                         const uint8_t* __restrict__ x_packed, uint4* __restrict__ codes, int* __restrict__ psum)
{
    __shared__ int sSum[kCodeGroups * kCodePixels];
    tc::pdl_trigger();
    const int px = threadIdx.x % kCodePixels, gi = threadIdx.x / kCodePixels;
    const int64_t P = (int64_t)blockIdx.x * kCodePixels + px;
    const int w = blockIdx.y;                               // phase image
    codes += (int64_t)w * (p.Cp / 16) * p.Pstride;
    psum += (int64_t)w * p.Pstride;
    const int64_t row_bytes = (int64_t)((a.C + kBlockCodes - 1) / kBlockCodes) * kBlockBytes;
    const uint32_t* src0 = nullptr;
    if (P < p.Ptot) {
        const uint32_t G = fdiv((uint32_t)P, p.div_pw);
        const int col = (int)((uint32_t)P - G * (uint32_t)p.PW) * a.stride + p.ph_c[w] - a.pad;
        const uint32_t b = fdiv(G, p.div_ph);
        const int r = (int)(G - b * (uint32_t)p.PH) * a.stride + p.ph_r[w] - a.pad;
        if (r >= 0 && r < a.H && col >= 0 && col < a.W)
            src0 = reinterpret_cast<const uint32_t*>(x_packed + (((int64_t)b * a.H + r) * a.W + col) * row_bytes);
    }
    int sum = 0;
    for (int h = gi; h < p.ngroup; h += kCodeGroups) {
        uint32_t nz = 0, sg = 0;
        if (src0 != nullptr) {
            const uint32_t* blk = src0 + (h >> 2) * 8 + (h & 3);
            nz = __ldg(blk);
            sg = __ldg(blk + 4);
            if (h * 32 + 32 > a.C) nz &= (1u << (a.C - h * 32)) - 1u;      // positions past C code to 0
        }
        uint32_t o[8];
        tc::unpack32(nz, sg, o);
        sum += __popc(nz & sg) - __popc(nz & ~sg);
        if (P < p.Pstride) {
            codes[(int64_t)(2 * h) * p.Pstride + P] = make_uint4(o[0], o[1], o[2], o[3]);
            codes[(int64_t)(2 * h + 1) * p.Pstride + P] = make_uint4(o[4], o[5], o[6], o[7]);
        }
    }
    sSum[gi * kCodePixels + px] = sum;
    __syncthreads();
    if (gi == 0 && P < p.Pstride) {
        int t = 0;
        for (int k = 0; k < kCodeGroups; ++k) t += sSum[k * kCodePixels + px];
        psum[P] = t;
    }
}

__device__ __forceinline__ void bulk_copy_g2s(uint32_t dst, const void* src, uint32_t bytes, uint32_t bar)
{
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                 ::"r"(dst), "l"(reinterpret_cast<uint64_t>(src)), "r"(bytes), "r"(bar) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx_r(uint64_t* bar, uint32_t bytes)
{
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;"
                 ::"r"(tc::smem_addr(bar)), "r"(bytes) : "memory");
}
__device__ __forceinline__ void role_wait_r(bool leader, uint64_t* bar, uint32_t parity, unsigned* status,
                                            volatile int* dead, int barrier_id, int nthreads)
{
    if (leader) wait_or_die(bar, parity, status, dead);
    asm volatile("bar.sync %0, %1;" ::"r"(barrier_id), "r"(nthreads) : "memory");
}

// ------------------------------------------------------------------------------------------------
// Kernel 2: the contraction and the epilogue.
// ------------------------------------------------------------------------------------------------
// kFused: the epilogue also applies phi, adds the skip connection, and hands the result to the next
// layer as fp32 and / or as packed Eq. 3 codes against that layer's thresholds (NextLayerArgs).
template <bool kFused>
__global__ void __launch_bounds__(kThreads, 1)
conv_i8r_kernel(const ConvArgs a, const __grid_constant__ ConvI8RPlan p, const uint4* __restrict__ codes,
                const int* __restrict__ psum, const NextLayerArgs f)
{
    extern __shared__ __align__(128) uint8_t smem[];
    uint4* sW = reinterpret_cast<uint4*>(smem + p.off_w);        // [T][Cp/16][Nq]
    float4* sC = reinterpret_cast<float4*>(smem + p.off_c);     // {c1, c2, c3, 0} per column
    uint64_t* bars = reinterpret_cast<uint64_t*>(smem + p.off_bar);
    uint64_t* slot_full = bars;                     // [kMaxSlots] bulk copies -> MMA
    uint64_t* slot_empty = bars + kMaxSlots;        // [kMaxSlots] MMA -> producer
    uint64_t* acc_full = bars + 2 * kMaxSlots;      // [kMaxAcc] MMA -> epilogue
    uint64_t* acc_empty = acc_full + kMaxAcc;       // [kMaxAcc] epilogue -> MMA
    uint32_t* slot = reinterpret_cast<uint32_t*>(smem + p.off_misc);
    volatile int* dead = reinterpret_cast<volatile int*>(smem + p.off_misc + 8);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int nchunk = p.Cp / 16;
    const int fq = blockIdx.x % p.S;                 // filter group of this CTA
    const int first_tile = blockIdx.x / p.S;         // it takes tiles first_tile, first_tile + cpg, ...
    const int n_base = fq * p.Nq;

    // ---------------------------------------------------------------- set-up (all threads)
    RTN_TL_INIT(conv_i8r)
    if (threadIdx.x == 0) RTN_TL(conv_i8r, 0);
    tc::pdl_trigger();
    if (warp == 0) tc::tmem_alloc(slot, p.tmem_cols);
    if (threadIdx.x == 32) {
        for (int i = 0; i < kMaxSlots; ++i) { tc::mbar_init(&slot_full[i], 1); tc::mbar_init(&slot_empty[i], 1); }
        for (int i = 0; i < kMaxAcc; ++i) { tc::mbar_init(&acc_full[i], 1); tc::mbar_init(&acc_empty[i], kEpiThreads); }
        tc::mbar_init_fence();
        *dead = 0;
    }
    // Nq <= 256 < the CTA's threads: one column per thread.  The operands of its epilogue constants (and the next
    // layer's thresholds) are fetched first, so that their trip to memory overlaps the filters'.
    const int col = n_base + (int)threadIdx.x;
    const bool has_col = (int)threadIdx.x < p.Nq && col < a.N;
    float ws_f = 0.f, wo_f = 0.f;
    int wsum_i = 0;
    float2 next_t = make_float2(-INFINITY, INFINITY);
    if (has_col) {
        ws_f = a.ep.w_scale[a.ep.n_wparam == 1 ? 0 : col];
        wo_f = a.ep.w_offset[a.ep.n_wparam == 1 ? 0 : col];
        wsum_i = a.w_sum[col];
        if constexpr (kFused) {
            // (as in the ternarizers: +1 is tested first)
            if (f.out_packed != nullptr)
                next_t = make_float2(f.next_lo[f.n_next == 1 ? 0 : col], f.next_hi[f.n_next == 1 ? 0 : col]);
        }
    }
    // this group's filters: bit planes -> int8, [tap][chunk][row]; rows beyond N are zero
    expand_filter_rows<2>(a.w_packed, sW, p.T, p.ngroup, p.Nq, p.div_nq, p.div_cw, n_base, a.N, -1, (int)threadIdx.x,
                          kThreads);
    if ((int)threadIdx.x < p.Nq) {
        // per-output-channel constants in double, rounded once:
        //   c1 = a_s*w_s, c2 = a_s*w_o, c3 = a_o*(w_s*S_w + K*w_o)     (K = C*kh*kw)
        const double a_s = a.ep.a_scale_val, a_o = a.ep.a_offset_val;
        float c1 = 0.f, c2 = 0.f, c3 = 0.f;
        if (has_col) {
            const double ws = ws_f, wo = wo_f;
            c1 = (float)(a_s * ws);
            c2 = (float)(a_s * wo);
            c3 = (float)(a_o * (ws * (double)wsum_i + (double)a.C * p.T * wo));
        }
        sC[threadIdx.x] = make_float4(c1, c2, c3, 0.f);
        if constexpr (kFused) reinterpret_cast<float2*>(smem + p.off_t)[threadIdx.x] = next_t;
    }
    tc::fence_smem_to_async_proxy();
    tc::tc_fence_before_sync();
    __syncthreads();
    tc::tc_fence_after_sync();
    const uint32_t tmem = *slot;
    if (threadIdx.x == 0) RTN_TL(conv_i8r, 2);
    tc::pdl_wait();         // from here on: the codes and sums of the code kernel, and out
    if (threadIdx.x == 0) RTN_TL(conv_i8r, 1);

    if (warp == 1) {
        // ------------------------------------------------------------ producer (one thread)
        if (lane == 0) {
            const uint32_t ring = tc::smem_addr(smem + p.off_slot);
            const uint32_t win_bytes = (uint32_t)p.ppix * 16u;
            uint32_t s = 0, ph = 0;             // ring slot and its phase
            bool alive = true;
            for (int tile = first_tile; tile < p.ntiles && alive; tile += p.cpg) {
                const int64_t P0 = (int64_t)tile * p.RT * p.PW;
                for (int h = 0; h < p.ngroup; h += p.gps) {
                    if (!wait_or_die(&slot_empty[s], ph ^ 1, a.status, dead)) { alive = false; break; }
                    mbar_expect_tx_r(&slot_full[s], (uint32_t)(2 * p.gps * p.nph) * win_bytes);
                    const uint32_t dst = ring + s * p.slot_bytes, bar = tc::smem_addr(&slot_full[s]);
                    for (int w = 0; w < p.nph; ++w)
                        for (int c = 0; c < 2 * p.gps; ++c)
                            bulk_copy_g2s(dst + (uint32_t)(w * 2 * p.gps + c) * win_bytes,
                                          codes + ((int64_t)w * nchunk + 2 * h + c) * p.Pstride + P0, win_bytes, bar);
                    if (++s == (uint32_t)p.nslots) { s = 0; ph ^= 1; }
                }
            }
        }
    } else if (warp == 0) {
        // ------------------------------------------------------------ MMA issue (one thread)
        if (lane == 0) {
            const uint32_t idesc = tc::idesc_i8(kTileM, (uint32_t)p.Nq);
            const uint64_t desc_hi = (uint64_t)((128u >> 4) | (1u << 14)) << 32;
            const uint32_t a_lbo_field = (((uint32_t)p.ppix * 16) >> 4) << 16;
            const uint32_t ring16 = (tc::smem_addr(smem + p.off_slot) >> 4) + a_lbo_field;
            const uint32_t slot16 = p.slot_bytes >> 4;
            const uint32_t w16 = (tc::smem_addr(sW) >> 4) + ((((uint32_t)p.Nq * 16) >> 4) << 16);
            const uint32_t wtap16 = (uint32_t)nchunk * (uint32_t)p.Nq;      // 16-byte units between taps
            // up to nine taps keep their operand offsets in registers: nothing but arithmetic between MMAs
            const bool taps_in_regs = p.T <= 9;
            uint32_t ta[9], tb[9];
            #pragma unroll
            for (int t = 0; t < 9; ++t) {
                ta[t] = taps_in_regs && t < p.T ? p.tap_shift[t] : 0u;
                tb[t] = (uint32_t)t * wtap16;
            }
            // The tensor core's queue is short: whatever this thread does between two MMAs is idle time
            // for it.  So no division in the loop (slot, phase and accumulator advance by increments),
            // and the next unit's barrier is tested before this unit's MMAs are issued: the producer
            // runs slots ahead, the test succeeds, and the next unit issues without a wait.
            uint32_t s = 0, ph = 0;             // ring slot and its phase
            int acc = 0;
            uint32_t acc_ph = 0;
            bool alive = true, have = false;    // have: slot s is known to be full
            int tl_i = 0;
            for (int tile = first_tile; tile < p.ntiles && alive; tile += p.cpg, ++tl_i) {
                if (!wait_or_die(&acc_empty[acc], acc_ph ^ 1, a.status, dead)) break;
                const uint32_t d = tmem + (uint32_t)(acc * p.Nq);
                for (int h0 = 0; h0 < p.ngroup && alive; h0 += p.gps) {
                    if (!have && !wait_or_die(&slot_full[s], ph, a.status, dead)) { alive = false; break; }
                    tc::tc_fence_after_sync();
                    if (h0 == 0 && tl_i < 8) RTN_TL(conv_i8r, 40 + 2 * tl_i);
                    const uint32_t s_cur = s;
                    if (++s == (uint32_t)p.nslots) { s = 0; ph ^= 1; }
                    have = tc::mbar_test(&slot_full[s], ph);
                  for (int hh = 0; hh < p.gps; ++hh) {
                    const int h = h0 + hh;
                    const uint32_t ag = ring16 + s_cur * slot16 + (uint32_t)(2 * hh) * (uint32_t)p.ppix;
                    const uint32_t bg = w16 + (uint32_t)(2 * h) * (uint32_t)p.Nq;
                    if (p.T == 9) {
                        // straight-line issue: one predicate set-up, then nothing but the MMAs
                        tc::mma_i8_ss(d, desc_hi | (uint64_t)(ag + ta[0]), desc_hi | (uint64_t)(bg + tb[0]), idesc, h > 0);
                        #pragma unroll
                        for (int t = 1; t < 9; ++t)
                            tc::mma_i8_ss_acc(d, desc_hi | (uint64_t)(ag + ta[t]), desc_hi | (uint64_t)(bg + tb[t]), idesc);
                    } else if (taps_in_regs) {
                        #pragma unroll
                        for (int t = 0; t < 9; ++t)
                            if (t < p.T)
                                tc::mma_i8_ss(d, desc_hi | (uint64_t)(ag + ta[t]), desc_hi | (uint64_t)(bg + tb[t]), idesc,
                                              h > 0 || t > 0);
                    } else {
                        for (int t = 0; t < p.T; ++t)
                            tc::mma_i8_ss(d, desc_hi | (uint64_t)(ag + p.tap_shift[t]),
                                          desc_hi | (uint64_t)(bg + (uint32_t)t * wtap16), idesc, h > 0 || t > 0);
                    }
                  }
                    tc::mma_commit(&slot_empty[s_cur]);
                }
                if (!alive) break;
                tc::mma_commit(&acc_full[acc]);
                if (tl_i < 8) RTN_TL(conv_i8r, 41 + 2 * tl_i);
                if (++acc == p.nAcc) { acc = 0; acc_ph ^= 1; }
            }
        }
    } else if (warp >= kEpiWarp0) {
        // ------------------------------------------------------------ epilogue: out = c1*S_xw + c2*S_x + c3
        const int q = warp & 3, half = (warp - kEpiWarp0) >> 2;
        const int64_t ostride = (int64_t)a.Ho * a.Wo;
        const int nblk16 = p.Nq / 16;
        const int blk_begin = half == 0 ? 0 : (nblk16 + 1) / 2;
        const int blk_end = half == 0 ? (nblk16 + 1) / 2 : nblk16;
        int acc = 0, tl_i = 0;
        uint32_t acc_ph = 0;
        for (int tile = first_tile; tile < p.ntiles; tile += p.cpg, ++tl_i) {
            const int g = tile * p.RT;
            const int nrows = min(p.RT, p.total_rows - g);
            role_wait_r(warp == kEpiWarp0, &acc_full[acc], acc_ph, a.status, dead, kEpiBarrier, kEpiThreads);
            const bool alive = !*dead;
            tc::tc_fence_after_sync();
            if (warp == kEpiWarp0 && lane == 0 && tl_i < 8) RTN_TL(conv_i8r, 56 + 2 * tl_i);
            const uint32_t pl = (uint32_t)(q * 32 + lane);         // pixel within the tile
            const uint32_t row = fdiv(pl, p.div_pw);
            const int wo = (int)(pl - row * (uint32_t)p.PW);
            const uint32_t G = (uint32_t)g + row;
            const uint32_t b = fdiv(G, p.div_ph);
            const int ho = (int)(G - b * (uint32_t)p.PH);
            const bool ok = alive && (int)row < nrows && b < (uint32_t)a.B && ho < a.Ho && wo < a.Wo;
            int n_inside = p.T, s_x = 0;
            if (ok) {
                const int* ps = psum + (int64_t)g * p.PW + pl;
                for (int t = 0; t < p.T; ++t) s_x += __ldg(ps + p.tap_psum[t]);
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
            const uint32_t trow = tmem + ((uint32_t)(q * 32) << 16) + (uint32_t)(acc * p.Nq);
            const int64_t obase = (((int64_t)b * a.N) * a.Ho + ho) * a.Wo + wo;
            // packed output: this pixel's row of N codes; positions from N to the end of the last
            // 128-code block are zero-filled (by the last filter group's first warp set)
            const int packed_cols = (a.N + kBlockCodes - 1) / kBlockCodes * kBlockCodes;
            uint8_t* out_row = nullptr;
            if constexpr (kFused) {
                if (ok && f.out_packed != nullptr) {
                    out_row = f.out_packed + (((int64_t)b * a.Ho + ho) * a.Wo + wo) * (int64_t)(packed_cols / 4);
                    if (fq == p.S - 1 && half == 0) zero_fill_packed_row(out_row, p.S * p.Nq, packed_cols);
                }
            }
            for (int blk = blk_begin; blk < blk_end; ++blk) {
                uint32_t v[16];
                tc::tmem_ld16(trow + (uint32_t)(blk * 16), v);
                tc::tmem_ld_wait();
                if (!ok) continue;
                const int r0 = blk * 16;                   // column of the accumulator = row of the filter group
                const int n0 = n_base + r0;
                if constexpr (kFused) {
                    uint32_t nzb, sgb;
                    next_layer_block16(a, f, v, sC + r0, reinterpret_cast<const float2*>(smem + p.off_t) + r0, fsx,
                                       border, p.T, ho, wo, n_inside, n0, obase + (int64_t)n0 * ostride, ostride,
                                       out_row != nullptr && n0 < packed_cols, nzb, sgb);
                    if (out_row != nullptr && n0 < packed_cols) {
                        uint8_t* dst = out_row + (n0 >> 7) * kBlockBytes + ((n0 & 127) >> 3);
                        *reinterpret_cast<uint16_t*>(dst) = (uint16_t)nzb;
                        *reinterpret_cast<uint16_t*>(dst + 16) = (uint16_t)sgb;
                    }
                    continue;
                }
                float* optr = a.out + obase + (int64_t)n0 * ostride;
                if (!border && a.dbg_acc == nullptr && n0 + 16 <= a.N) {
                    // results first, stores after: a shared-memory load may not be moved above a global store the
                    // compiler cannot tell apart from it, and alternating the two made every column wait for the last
                    float r[16];
                    #pragma unroll
                    for (int j = 0; j < 16; ++j) {
                        const float4 c = sC[r0 + j];
                        r[j] = fmaf(c.x, (float)(int)v[j], fmaf(c.y, fsx, c.z));
                    }
                    #pragma unroll
                    for (int j = 0; j < 16; ++j, optr += ostride) *optr = r[j];
                } else {
                    #pragma unroll
                    for (int j = 0; j < 16; ++j) {
                        const int n = n0 + j;
                        if (n >= a.N) continue;
                        const int s_xw = (int)v[j];
                        const float4 c = sC[r0 + j];
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
                        optr[(int64_t)j * ostride] = fmaf(c.x, (float)s_xw, fmaf(c.y, fsx, c3));
                        if (a.dbg_acc != nullptr) a.dbg_acc[obase + (int64_t)n * ostride] = s_xw;
                    }
                }
            }
            tc::tc_fence_before_sync();
            tc::mbar_arrive(&acc_empty[acc]);
            if (warp == kEpiWarp0 && lane == 0 && tl_i < 8) RTN_TL(conv_i8r, 57 + 2 * tl_i);
            if (++acc == p.nAcc) { acc = 0; acc_ph ^= 1; }
        }
    }
    tc::tc_fence_before_sync();
    __syncthreads();
    if (warp == 0) tc::tmem_dealloc(tmem, p.tmem_cols);
    if (threadIdx.x == 0) RTN_TL(conv_i8r, 4);
}

// Scratch of the variant that allocates nothing: one array per device, part of the module's image.
// 16 MiB holds the int8 codes of every stride-1 layer of ResNet-18 that this variant takes at batch
// 128 (512 -> 512, 3x3 on 7x7: 5.4 MB).  Every caller on a device shares it.
constexpr size_t kStaticScratchBytes = size_t(16) << 20;
static __device__ __align__(256) uint8_t g_static_scratch[kStaticScratchBytes];

// Address of the array on the current device, looked up once per device.
void* static_scratch()
{
    constexpr int kMaxDevices = 64;
    static void* addr[kMaxDevices] = {};
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return nullptr;
    if (addr[dev] == nullptr) {
        void* ptr = nullptr;
        if (cudaGetSymbolAddress(&ptr, g_static_scratch) != cudaSuccess || ptr == nullptr) {
            cudaGetLastError();
            return nullptr;
        }
        addr[dev] = ptr;
    }
    return addr[dev];
}

cudaError_t launch_with_scratch(const ConvArgs& c, const ConvI8RPlan& p, void* scratch, cudaStream_t s,
                                const NextLayerArgs* f = nullptr)
{
    uint4* codes = reinterpret_cast<uint4*>(scratch);
    int* psum = reinterpret_cast<int*>(reinterpret_cast<uint8_t*>(scratch) + p.codes_bytes);
    const dim3 blocks((unsigned)((p.Pstride + kCodePixels - 1) / kCodePixels), (unsigned)p.nph);
    if (f != nullptr && f->x_packed != nullptr) {
        conv_codes_packed_kernel<<<blocks, kCodePixels * kCodeGroups, 0, s>>>(c, p, f->x_packed, codes, psum);
    } else {
        const size_t smem1 = (size_t)p.Cp * 8 + (size_t)kCodeGroups * kCodePixels * 4;
        conv_codes_kernel<<<blocks, kCodePixels * kCodeGroups, smem1, s>>>(c, p, codes, psum);
    }
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) return e;
    if (f != nullptr) {
        e = cudaFuncSetAttribute(conv_i8r_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)p.smem_bytes);
        if (e != cudaSuccess) return e;
        return launch_pdl(conv_i8r_kernel<true>, dim3((unsigned)p.grid), dim3(kThreads), p.smem_bytes, s, c, p,
                          (const uint4*)codes, (const int*)psum, *f);
    }
    e = cudaFuncSetAttribute(conv_i8r_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)p.smem_bytes);
    if (e != cudaSuccess) return e;
    return launch_pdl(conv_i8r_kernel<false>, dim3((unsigned)p.grid), dim3(kThreads), p.smem_bytes, s, c, p,
                      (const uint4*)codes, (const int*)psum, NextLayerArgs{});
}

}  // namespace

bool conv_i8r_supported(const ConvArgs& c)
{
    ConvI8RPlan p;
    return make_plan_r(c, p, device_sm_count());
}

bool conv_i8r_next_supported(const ConvArgs& c)
{
    ConvI8RPlan p;
    return make_plan_r(c, p, device_sm_count(), true);
}

// Rough time of this variant for a shape, in microseconds (negative: not taken).  Measured on B200: about
// 8 us of fixed cost (two launches, filter expansion, the last epilogue) plus the multiply-accumulates over the
// padded pixels at 640 T/s (64 or more filters per CTA) or 370 T/s (fewer: an MMA a quarter full).
double conv_i8r_estimate_us(const ConvArgs& c)
{
    ConvI8RPlan p;
    if (!make_plan_r(c, p, device_sm_count())) return -1.0;
    const double macs = (double)p.Ptot * p.Cp * p.T * (double)(p.S * p.Nq);     // padded output pixels x K x filters
    return 8.0 + macs / ((p.Nq >= 64 ? 640.0 : 370.0) * 1e6);
}

size_t conv_i8r_scratch_bytes(const ConvArgs& c)
{
    ConvI8RPlan p;
    return make_plan_r(c, p, device_sm_count()) ? p.scratch_bytes : 0;
}

// The scratch buffer comes from the stream-ordered allocator and goes back to it right after the two
// launches, in stream order: no state in the library, safe with several streams, and legal inside a
// stream capture (the pair becomes allocation and free nodes of the graph).
cudaError_t launch_conv_i8r(const ConvArgs& c, cudaStream_t s)
{
    ConvI8RPlan p;
    if (!make_plan_r(c, p, device_sm_count())) return cudaErrorInvalidConfiguration;
    void* scratch = nullptr;
    cudaError_t e = cudaMallocAsync(&scratch, p.scratch_bytes, s);
    if (e != cudaSuccess) return e;
    e = launch_with_scratch(c, p, scratch, s);
    const cudaError_t e2 = cudaFreeAsync(scratch, s);
    return e != cudaSuccess ? e : e2;
}

// Same two launches with the scratch in the device's static array: no allocating call on this path.
// cudaErrorInvalidValue: the layer needs more scratch than the array has.
cudaError_t launch_conv_i8r_static(const ConvArgs& c, cudaStream_t s)
{
    ConvI8RPlan p;
    if (!make_plan_r(c, p, device_sm_count())) return cudaErrorInvalidConfiguration;
    if (p.scratch_bytes > kStaticScratchBytes) return cudaErrorInvalidValue;
    void* scratch = static_scratch();
    if (scratch == nullptr) return cudaErrorInvalidDevicePointer;
    return launch_with_scratch(c, p, scratch, s);
}

size_t conv_i8r_static_scratch_bytes() { return kStaticScratchBytes; }

// The two launches with the hand-over to the next layer fused into the second one's epilogue; the
// first one reads fp32 (Eq. 3 in-kernel) or packed pixel rows.  Scratch as in launch_conv_i8r.
cudaError_t launch_conv_i8r_next(const ConvArgs& c, const NextLayerArgs& f, cudaStream_t s)
{
    ConvI8RPlan p;
    if (!make_plan_r(c, p, device_sm_count(), true)) return cudaErrorInvalidConfiguration;
    void* scratch = nullptr;
    cudaError_t e = cudaMallocAsync(&scratch, p.scratch_bytes, s);
    if (e != cudaSuccess) return e;
    e = launch_with_scratch(c, p, scratch, s, &f);
    const cudaError_t e2 = cudaFreeAsync(scratch, s);
    return e != cudaSuccess ? e : e2;
}

}  // namespace rtn
