// Ternary conv2d, tensor-core variant with STREAMED filters: for layers whose int8 filter bank does
// not fit shared memory (e.g. 256 -> 256 channels, 3x3) and for 1x1 convolutions of any stride.
//
// Same arithmetic as the resident-filter kernel: fp32 NCHW input ternarized in-kernel (Eq. 3) to
// int8 codes in shared memory laid out [16-channel chunk][pixel][16 B] (K-major, no swizzle), the
// implicit GEMM of a stride-1 conv done by shifting the A window by (i*PW + j) pixels per filter
// tap, tcgen05.mma kind::i8 into int32 accumulators in tensor memory, affine epilogue fused.
// Differences:
//   * the filters are expanded from their bit planes (Table 1) to int8 one K = 32 slice at a time
//     into a ring of shared-memory stages, by the same warps that ternarized the tile, while the
//     tensor core consumes earlier slices;
//   * S_x comes from per-pixel code sums the ternarizer leaves in shared memory (summed over the
//     taps in the epilogue), so all 256 accumulator columns are free for output channels;
//   * a 1x1 convolution (any stride, no padding) uses the same code with "rows" = output rows and a
//     strided pixel gather in the ternarizer (no halo, one tap).
//
// Warp roles: warp 0 issues MMAs (one thread); warps 4..11 epilogue; warps 12..19 workers
// (ternarize the tile, then expand filter slices).  One code buffer, one accumulator set (two when
// they fit), mbarrier hand-offs with bounded waits.
#include "rtn_internal.cuh"
#include "rtn_tcgen05.cuh"
#include "rtn_conv_i8_common.cuh"

namespace rtn {

namespace {

using namespace conv_detail;

constexpr int kEpiWarp0 = 4;
constexpr int kEpiWarps = 8;
constexpr int kEpiThreads = kEpiWarps * 32;
constexpr int kWorkWarp0 = kEpiWarp0 + kEpiWarps;
constexpr int kWorkWarps = 8;
constexpr int kWorkThreads = kWorkWarps * 32;
constexpr int kThreads = (kWorkWarp0 + kWorkWarps) * 32;
constexpr int kTileM = 128;
constexpr int kMaxK = 304;                             // K = 32 slices per tile the table holds
constexpr int kMaxWStages = 8;
constexpr int kSlices = 4;                             // K = 32 slices per filter stage (one packed block)
constexpr size_t kSmemLimit = 220 * 1024;
constexpr int kWorkBarrier = 2;

struct ConvI8SPlan {
    int PW, PH;            // row length / rows per image of the pixel sequence (padded for k > 1)
    int istride, ipad;     // input pixel of sequence pixel (r, c): (r*istride - ipad, c*istride - ipad)
    int Cp, Np, T, TM, RT, halo, ppix, total_rows, grid;
    int nK;                // K = 32 slices per tile: taps * Cp/32
    int nW;                // filter ring depth
    int nAcc;              // accumulator sets (1 or 2)
    uint32_t tmem_cols;
    FastDiv div_pw, div_ph;
    uint32_t off_a, off_w, off_psum, off_lo, off_hi, off_c, off_bar, off_misc;
    size_t smem_bytes;
    uint32_t tab_a[kMaxK]; // per slice: start of the A window in 16-byte units of the code buffer
};

bool make_plan_s(const ConvArgs& c, ConvI8SPlan& p, int sms)
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
    if (p.Np > 256) return false;
    if ((int64_t)c.C * p.T > (int64_t(1) << 24)) return false;
    p.total_rows = c.B * p.PH;
    p.TM = (2 * p.Np <= 512 && (int64_t)p.total_rows * p.PW >= (int64_t)2 * 148 * kTileM) ? 2 : 1;
    p.nAcc = (2 * p.TM * p.Np <= 512) ? 2 : 1;
    p.RT = p.TM * kTileM / p.PW;
    if (p.RT < 1) return false;
    p.ppix = (p.TM * kTileM + p.halo * p.PW + (c.kw - 1) + 7) / 8 * 8;
    const int tiles = (p.total_rows + p.RT - 1) / p.RT;
    p.grid = tiles < sms ? tiles : sms;
    uint32_t cols = 32;
    while (cols < (uint32_t)(p.nAcc * p.TM * p.Np)) cols *= 2;
    p.tmem_cols = cols;
    p.div_pw = make_fastdiv((uint32_t)p.PW);
    p.div_ph = make_fastdiv((uint32_t)p.PH);
    p.nK = p.T * (p.Cp / 32);
    if (p.nK > kMaxK) return false;
    for (int i = 0; i < p.nK; ++i) {
        const int t = i / (p.Cp / 32), h = i % (p.Cp / 32);
        p.tab_a[i] = (uint32_t)(2 * h) * p.ppix + (uint32_t)((t / c.kw) * p.PW + (t % c.kw));
    }
    uint32_t o = 0;
    p.off_a = o;    o += (uint32_t)(p.Cp / 16) * p.ppix * 16;
    p.off_psum = o; o += 3u * (uint32_t)p.ppix * 4;
    p.off_lo = o;   o += (uint32_t)p.Cp * 4;
    p.off_hi = o;   o += (uint32_t)p.Cp * 4;
    o = (o + 15) / 16 * 16;
    p.off_c = o;    o += (uint32_t)p.Np * 16;
    p.off_bar = o;  o += (6 + 2 * kMaxWStages) * 8;     // a_full a_empty acc_full[2] acc_empty[2] w_full[] w_empty[]
    p.off_misc = o; o += 16;
    o = (o + 127) / 128 * 128;
    p.off_w = o;
    if (o > kSmemLimit) return false;
    const uint32_t stage = (uint32_t)p.Np * 32 * kSlices;
    const int ngroups = (p.nK + kSlices - 1) / kSlices;
    int nw = (int)((kSmemLimit - o) / stage);
    if (nw > kMaxWStages) nw = kMaxWStages;
    if (nw > ngroups) nw = ngroups;
    if (nw < 2 && ngroups > 1) return false;
    if (nw < 1) return false;
    p.nW = nw;
    p.smem_bytes = o + (uint32_t)nw * stage;
    return true;
}

__global__ void __launch_bounds__(kThreads, 1)
conv_i8s_kernel(const ConvArgs a, const __grid_constant__ ConvI8SPlan p)
{
    extern __shared__ __align__(128) uint8_t smem[];
    uint4* sA = reinterpret_cast<uint4*>(smem + p.off_a);        // [Cp/16][ppix]
    uint4* sWr = reinterpret_cast<uint4*>(smem + p.off_w);       // [nW][kSlices][2][Np]
    int* sPsum = reinterpret_cast<int*>(smem + p.off_psum);      // [3][ppix]
    float* sLo = reinterpret_cast<float*>(smem + p.off_lo);
    float* sHi = reinterpret_cast<float*>(smem + p.off_hi);
    float4* sC = reinterpret_cast<float4*>(smem + p.off_c);
    uint64_t* bars = reinterpret_cast<uint64_t*>(smem + p.off_bar);
    uint64_t* a_full = bars;            // workers -> MMA: codes of the tile written
    uint64_t* a_empty = bars + 1;       // MMA -> workers: the tile's MMAs are done
    uint64_t* acc_full = bars + 2;      // [2] MMA -> epilogue
    uint64_t* acc_empty = bars + 4;     // [2] epilogue -> MMA
    uint64_t* w_full = bars + 6;                    // [nW] workers -> MMA: filter slice expanded
    uint64_t* w_empty = bars + 6 + kMaxWStages;     // [nW] MMA -> workers: slice consumed
    uint32_t* slot = reinterpret_cast<uint32_t*>(smem + p.off_misc);
    volatile int* dead = reinterpret_cast<volatile int*>(smem + p.off_misc + 8);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int nchunk = p.Cp / 16;
    const int s0 = (int)((int64_t)blockIdx.x * p.total_rows / p.grid);
    const int s1 = (int)((int64_t)(blockIdx.x + 1) * p.total_rows / p.grid);

    tc::pdl_trigger();
    if (warp == 0) tc::tmem_alloc(slot, p.tmem_cols);
    if (threadIdx.x == 32) {
        tc::mbar_init(a_full, kWorkWarps);
        tc::mbar_init(a_empty, 1);
        for (int i = 0; i < 2; ++i) { tc::mbar_init(&acc_full[i], 1); tc::mbar_init(&acc_empty[i], kEpiThreads); }
        for (int i = 0; i < kMaxWStages; ++i) { tc::mbar_init(&w_full[i], kWorkWarps); tc::mbar_init(&w_empty[i], 1); }
        tc::mbar_init_fence();
        *dead = 0;
    }
    for (int c = threadIdx.x; c < p.Cp; c += kThreads) {
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

    if (warp >= kWorkWarp0) {
        // ------------------------------------------------------------ workers
        const int tid = threadIdx.x - kWorkWarp0 * 32;
        const int64_t cs = (int64_t)a.H * a.W;
        const bool per_layer = a.n_thr == 1;
        const float lo0 = sLo[0], hi0 = sHi[0];
        // filter row of this thread: planes of packed block j are two uint4 at Wrow + 2 j
        const int cwords = p.Cp / 32;
        const int64_t row_blocks = ((int64_t)p.T * cwords + 3) / 4;
        const uint4* Wrow = tid < a.N ? reinterpret_cast<const uint4*>(a.w_packed) + (int64_t)tid * row_blocks * 2
                                      : nullptr;
        uint32_t wcount = 0;
        int it = 0;
        for (int g = s0; g < s1; g += p.RT, ++it) {
            const int nrows = min(p.RT, s1 - g);
            const int npix = (nrows + p.halo) * p.PW;
            int* psum = sPsum + (it % 3) * p.ppix;
            wait_or_die(a_empty, (it & 1) ^ 1, a.status, dead);
            for (int i = tid; i < p.ppix; i += kWorkThreads) psum[i] = 0;
            asm volatile("bar.sync %0, %1;" ::"r"(kWorkBarrier), "r"(kWorkThreads) : "memory");
            // ---- ternarize: item = (pixel of the tile's sequence, pair of 16-channel chunks): 32 loads in flight
            for (int i = tid; i < (nchunk / 2) * npix; i += kWorkThreads) {
                const int cp = i / npix, pp = i - cp * npix;
                const uint32_t sl = fdiv((uint32_t)pp, p.div_pw);
                const int c = (int)((uint32_t)pp - sl * (uint32_t)p.PW) * p.istride - p.ipad;
                const uint32_t G = (uint32_t)g + sl;
                const uint32_t b = fdiv(G, p.div_ph);
                const int r = (int)(G - b * (uint32_t)p.PH) * p.istride - p.ipad;
                uint4 w0 = make_uint4(0, 0, 0, 0), w1 = make_uint4(0, 0, 0, 0);
                if (b < (uint32_t)a.B && r >= 0 && r < a.H && c >= 0 && c < a.W) {
                    const float* src = a.x + (((int64_t)b * a.C + cp * 32) * a.H + r) * a.W + c;
                    float v0[16], v1[16];
                    #pragma unroll
                    for (int e = 0; e < 16; ++e) {
                        v0[e] = (cp * 32 + perm16(e) < a.C) ? __ldg(src + perm16(e) * cs) : 0.0f;
                        v1[e] = (cp * 32 + 16 + perm16(e) < a.C) ? __ldg(src + (16 + perm16(e)) * cs) : 0.0f;
                    }
                    w0 = per_layer ? codes16<true>(v0, sLo, sHi, cp * 32, lo0, hi0)
                                   : codes16<false>(v0, sLo, sHi, cp * 32, lo0, hi0);
                    w1 = per_layer ? codes16<true>(v1, sLo, sHi, cp * 32 + 16, lo0, hi0)
                                   : codes16<false>(v1, sLo, sHi, cp * 32 + 16, lo0, hi0);
                    int s = __dp4a((int)w0.x, 0x01010101, __dp4a((int)w0.y, 0x01010101,
                            __dp4a((int)w0.z, 0x01010101, __dp4a((int)w0.w, 0x01010101, 0))));
                    s = __dp4a((int)w1.x, 0x01010101, __dp4a((int)w1.y, 0x01010101,
                        __dp4a((int)w1.z, 0x01010101, __dp4a((int)w1.w, 0x01010101, s))));
                    if (s != 0) atomicAdd(&psum[pp], s);
                }
                sA[(2 * cp) * p.ppix + pp] = w0;
                sA[(2 * cp + 1) * p.ppix + pp] = w1;
            }
            tc::fence_smem_to_async_proxy();
            __syncwarp();
            if (lane == 0) tc::mbar_arrive(a_full);
            // ---- filter slices of this tile, one packed block (four K = 32 slices) per ring stage; slice ks
            //      is word ks of the packed row.  The next block's planes are fetched while this one expands.
            uint4 nzn = make_uint4(0, 0, 0, 0), sgn = nzn;
            if (Wrow != nullptr) { nzn = __ldg(Wrow); sgn = __ldg(Wrow + 1); }
            for (int ks0 = 0; ks0 < p.nK; ks0 += kSlices, ++wcount) {
                const uint4 nzv = nzn, sgv = sgn;
                if (Wrow != nullptr && ks0 + kSlices < p.nK) {
                    nzn = __ldg(Wrow + 2 * ((ks0 >> 2) + 1));
                    sgn = __ldg(Wrow + 2 * ((ks0 >> 2) + 1) + 1);
                }
                const uint32_t st = wcount % (uint32_t)p.nW;
                wait_or_die(&w_empty[st], ((wcount / (uint32_t)p.nW) & 1) ^ 1, a.status, dead);
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
    } else if (warp == 0) {
        // ------------------------------------------------------------ MMA issue (one thread)
        if (lane == 0) {
            const uint32_t idesc = tc::idesc_i8(kTileM, (uint32_t)p.Np);
            const uint64_t desc_hi = (uint64_t)((128u >> 4) | (1u << 14)) << 32;
            const uint32_t a_lbo_field = (((uint32_t)p.ppix * 16) >> 4) << 16;
            const uint32_t a16 = (tc::smem_addr(sA) >> 4) + a_lbo_field;
            const uint32_t w16 = (tc::smem_addr(sWr) >> 4) + ((((uint32_t)p.Np * 16) >> 4) << 16);
            const uint32_t wslice16 = ((uint32_t)p.Np * 32) >> 4;
            const uint32_t wstage16 = wslice16 * kSlices;
            uint32_t wcount = 0;
            int it = 0;
            bool alive = true;
            for (int g = s0; g < s1 && alive; g += p.RT, ++it) {
                const int acc = p.nAcc == 2 ? (it & 1) : 0;
                const uint32_t acc_ph = p.nAcc == 2 ? ((it >> 1) & 1) : (it & 1);
                const int nrows = min(p.RT, s1 - g);
                const int ntm = (nrows * p.PW + kTileM - 1) / kTileM;
                alive = wait_or_die(a_full, it & 1, a.status, dead) &&
                        wait_or_die(&acc_empty[acc], acc_ph ^ 1, a.status, dead);
                if (!alive) break;
                for (int ks0 = 0; ks0 < p.nK; ks0 += kSlices, ++wcount) {
                    const uint32_t st = wcount % (uint32_t)p.nW;
                    if (!wait_or_die(&w_full[st], (wcount / (uint32_t)p.nW) & 1, a.status, dead)) { alive = false; break; }
                    tc::tc_fence_after_sync();
                    const int nks = min(kSlices, p.nK - ks0);
                    for (int j = 0; j < nks; ++j) {
                        const uint64_t bd = desc_hi | (uint64_t)(w16 + st * wstage16 + (uint32_t)j * wslice16);
                        const uint32_t aw = a16 + p.tab_a[ks0 + j];
                        for (int tm = 0; tm < ntm; ++tm) {
                            const uint32_t d = tmem + (uint32_t)((acc * p.TM + tm) * p.Np);
                            tc::mma_i8_ss(d, desc_hi | (uint64_t)(aw + (uint32_t)(tm * kTileM)), bd, idesc, ks0 + j > 0);
                        }
                    }
                    tc::mma_commit(&w_empty[st]);
                }
                if (!alive) break;
                tc::mma_commit(a_empty);
                tc::mma_commit(&acc_full[acc]);
            }
        }
    } else if (warp >= kEpiWarp0 && warp < kEpiWarp0 + kEpiWarps) {
        // ------------------------------------------------------------ epilogue: out = c1*S_xw + c2*S_x + c3
        const int q = warp & 3, half = (warp - kEpiWarp0) >> 2;
        const int64_t ostride = (int64_t)a.Ho * a.Wo;
        const int nblk16 = (a.N + 15) / 16;
        const int blk_begin = half == 0 ? 0 : (nblk16 + 1) / 2;
        const int blk_end = half == 0 ? (nblk16 + 1) / 2 : nblk16;
        int it = 0;
        for (int g = s0; g < s1; g += p.RT, ++it) {
            const int acc = p.nAcc == 2 ? (it & 1) : 0;
            const uint32_t acc_ph = p.nAcc == 2 ? ((it >> 1) & 1) : (it & 1);
            const int nrows = min(p.RT, s1 - g);
            const int ntm = (nrows * p.PW + kTileM - 1) / kTileM;
            const int* psum = sPsum + (it % 3) * p.ppix;
            const bool alive = wait_or_die(&acc_full[acc], acc_ph, a.status, dead);
            tc::tc_fence_after_sync();
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
                const uint32_t trow = tmem + ((uint32_t)(q * 32) << 16) + (uint32_t)((acc * p.TM + tm) * p.Np);
                float* optr = a.out + (((int64_t)b * a.N) * a.Ho + ho) * a.Wo + wo;
                int32_t* dptr = a.dbg_acc ? a.dbg_acc + (((int64_t)b * a.N) * a.Ho + ho) * a.Wo + wo : nullptr;
                for (int blk = blk_begin; blk < blk_end; ++blk) {
                    uint32_t v[16];
                    tc::tmem_ld16(trow + (uint32_t)(blk * 16), v);
                    tc::tmem_ld_wait();
                    if (!ok) continue;
                    const int n0 = blk * 16;
                    if (!border && dptr == nullptr && n0 + 16 <= a.N) {
                        #pragma unroll
                        for (int j = 0; j < 16; ++j) {
                            const float4 c = sC[n0 + j];
                            optr[(int64_t)(n0 + j) * ostride] = fmaf(c.x, (float)(int)v[j], fmaf(c.y, fsx, c.z));
                        }
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
        }
    }
    tc::tc_fence_before_sync();
    __syncthreads();
    if (warp == 0) tc::tmem_dealloc(tmem, p.tmem_cols);
}

int sm_count_s()
{
    int dev = 0, sms = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) return 148;
    if (cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || sms <= 0) return 148;
    return sms;
}

}  // namespace

bool conv_i8s_supported(const ConvArgs& c)
{
    ConvI8SPlan p;
    return make_plan_s(c, p, 148);
}

cudaError_t launch_conv_i8s(const ConvArgs& c, cudaStream_t s)
{
    ConvI8SPlan p;
    if (!make_plan_s(c, p, sm_count_s())) return cudaErrorInvalidConfiguration;
    cudaError_t e = cudaFuncSetAttribute(conv_i8s_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                         (int)p.smem_bytes);
    if (e != cudaSuccess) return e;
    return launch_pdl(conv_i8s_kernel, dim3((unsigned)p.grid), dim3(kThreads), p.smem_bytes, s, c, p);
}

}  // namespace rtn
