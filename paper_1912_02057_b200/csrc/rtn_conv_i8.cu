// Ternary conv2d (stride 1), tensor-core variant: fp32 NCHW input ternarized in-kernel (Eq. 3)
// straight to int8 {-1,0,+1} in shared memory, filters expanded from their bit planes to int8 in
// shared memory, tcgen05.mma kind::i8 into int32 accumulators in tensor memory, affine epilogue.
//
// Implicit GEMM without im2col, by a shift: lay the zero-padded images of the batch out as one
// long sequence of padded pixels, Q = (b*PH + r)*PW + c with PH = H + 2 pad, PW = W + 2 pad.  The
// output whose top-left tap sits at padded pixel Q reads, for tap (i, j), padded pixel
// Q + i*PW + j.  So for a tile of 128 consecutive Q the A operand of tap (i, j) is the SAME
// shared-memory code array, read from a start address shifted by (i*PW + j) pixels.  Outputs whose
// Q falls in the padding columns/rows (c >= Wo or r >= Ho) are computed and dropped.
//
// Shared-memory code array: [channel chunk of 16][padded pixel][16 bytes] -- K-major without
// swizzle, a core matrix (8 pixels x 16 channels) is 128 contiguous bytes wherever the window
// starts.  Filters: [tap][channel chunk][n][16 bytes].  Within a group of 32 channels both
// operands use the byte order of tc::unpack32.
#include "rtn_internal.cuh"
#include "rtn_tcgen05.cuh"

namespace rtn {

namespace {

constexpr int kThreads = 256;
constexpr int kTileM = 128;                       // pixels per MMA (TMEM lanes)
constexpr size_t kSmemLimit = 200 * 1024;

// channel (within a group of 16) held by byte e of a 16-byte chunk: tc::unpack32's order
// (0,4,8,12, 2,6,10,14, 1,5,9,13, 3,7,11,15)
__host__ __device__ constexpr int perm16(int e)
{
    return 4 * (e & 3) + ((e >> 2) == 0 ? 0 : (e >> 2) == 1 ? 2 : (e >> 2) == 2 ? 1 : 3);
}

struct ConvI8Plan {
    int PW, PH;            // padded image extent
    int Cp, Np;            // channels rounded up to 32, output channels rounded up to 16
    int T;                 // taps
    int TM;                // 128-pixel sub-tiles per CTA
    int ppix;              // padded pixels held in shared memory per CTA
    int64_t total_q;       // B*PH*PW
    uint32_t tmem_cols;
    // byte offsets into dynamic shared memory
    uint32_t off_a, off_w, off_psum, off_lo, off_hi, off_c1, off_c2, off_c3, off_bar, off_slot;
    size_t smem_bytes;
};

inline uint32_t align_up(uint32_t x, uint32_t a) { return (x + a - 1) / a * a; }

bool make_plan(const ConvArgs& c, ConvI8Plan& p)
{
    if (c.stride != 1) return false;
    if (c.Ho <= 0 || c.Wo <= 0) return false;
    p.PW = c.W + 2 * c.pad;
    p.PH = c.H + 2 * c.pad;
    p.Cp = (c.C + 31) / 32 * 32;
    p.Np = (c.N + 15) / 16 * 16;
    p.T = c.kh * c.kw;
    if (p.Np > 256) return false;
    p.total_q = (int64_t)c.B * p.PH * p.PW;
    const int64_t tiles1 = (p.total_q + kTileM - 1) / kTileM;
    p.TM = (tiles1 >= 4 * 148 && 2 * p.Np <= 512) ? 2 : 1;
    const int halo = (c.kh - 1) * p.PW + (c.kw - 1);
    p.ppix = (p.TM * kTileM + halo + 7) / 8 * 8;
    uint32_t cols = 32;
    while (cols < (uint32_t)(p.TM * p.Np)) cols *= 2;
    p.tmem_cols = cols;
    uint32_t o = 0;
    p.off_a = o;    o += (uint32_t)(p.Cp / 16) * p.ppix * 16;
    p.off_w = o;    o += (uint32_t)p.T * (p.Cp / 16) * p.Np * 16;
    p.off_psum = o; o += (uint32_t)p.ppix * 4;
    p.off_lo = o;   o += (uint32_t)p.Cp * 4;
    p.off_hi = o;   o += (uint32_t)p.Cp * 4;
    p.off_c1 = o;   o += (uint32_t)p.Np * 4;
    p.off_c2 = o;   o += (uint32_t)p.Np * 4;
    p.off_c3 = o;   o += (uint32_t)p.Np * 4;
    o = align_up(o, 8);
    p.off_bar = o;  o += 8;
    p.off_slot = o; o += 8;
    p.smem_bytes = o;
    if (p.smem_bytes > kSmemLimit) return false;
    // descriptor fields are 14 bits of 16-byte units
    if ((uint32_t)p.ppix * 16 >= (1u << 18) || (uint32_t)p.Np * 16 >= (1u << 18)) return false;
    const int64_t grid = (p.total_q + (int64_t)p.TM * kTileM - 1) / ((int64_t)p.TM * kTileM);
    if (grid > 0x7fffffff) return false;
    return true;
}

__global__ void __launch_bounds__(kThreads)
conv_i8_kernel(const ConvArgs a, const ConvI8Plan p)
{
    extern __shared__ __align__(128) uint8_t smem[];
    uint4* sA = reinterpret_cast<uint4*>(smem + p.off_a);        // [Cp/16][ppix]
    uint4* sW = reinterpret_cast<uint4*>(smem + p.off_w);        // [T][Cp/16][Np]
    int* sPsum = reinterpret_cast<int*>(smem + p.off_psum);
    float* sLo = reinterpret_cast<float*>(smem + p.off_lo);
    float* sHi = reinterpret_cast<float*>(smem + p.off_hi);
    float* sC1 = reinterpret_cast<float*>(smem + p.off_c1);
    float* sC2 = reinterpret_cast<float*>(smem + p.off_c2);
    float* sC3 = reinterpret_cast<float*>(smem + p.off_c3);
    uint64_t* bar = reinterpret_cast<uint64_t*>(smem + p.off_bar);
    uint32_t* slot = reinterpret_cast<uint32_t*>(smem + p.off_slot);

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int64_t q0 = (int64_t)blockIdx.x * p.TM * kTileM;
    const int nchunk = p.Cp / 16;
    const int img = p.PH * p.PW;

    if (warp == 0) tc::tmem_alloc(slot, p.tmem_cols);
    if (tid == 0) {
        tc::mbar_init(bar, 1);
        tc::mbar_init_fence();
    }
    for (int i = tid; i < p.ppix; i += kThreads) sPsum[i] = 0;
    for (int c = tid; c < p.Cp; c += kThreads) {
        // channel padding: thresholds that code everything to 0
        sLo[c] = c < a.C ? a.t_lo[a.n_thr == 1 ? 0 : c] : -INFINITY;
        sHi[c] = c < a.C ? a.t_hi[a.n_thr == 1 ? 0 : c] : INFINITY;
    }
    {   // per-output-channel constants in double, rounded once:
        //   c1 = a_s*w_s, c2 = a_s*w_o, c3 = a_o*(w_s*S_w + K*w_o)     (K = C*kh*kw)
        const double a_s = a.ep.a_scale_val, a_o = a.ep.a_offset_val;
        for (int n = tid; n < p.Np; n += kThreads) {
            float c1 = 0.f, c2 = 0.f, c3 = 0.f;
            if (n < a.N) {
                const double ws = a.ep.w_scale[a.ep.n_wparam == 1 ? 0 : n];
                const double wo = a.ep.w_offset[a.ep.n_wparam == 1 ? 0 : n];
                c1 = (float)(a_s * ws);
                c2 = (float)(a_s * wo);
                c3 = (float)(a_o * (ws * (double)a.w_sum[n] + (double)a.C * p.T * wo));
            }
            sC1[n] = c1; sC2[n] = c2; sC3[n] = c3;
        }
    }
    __syncthreads();

    // ---- 1. ternarize the padded pixels this tile touches: item = (chunk of 16 channels, pixel)
    for (int it = tid; it < nchunk * p.ppix; it += kThreads) {
        const int ch = it / p.ppix, pp = it % p.ppix;
        const int64_t Q = q0 + pp;
        uint32_t w[4] = {0, 0, 0, 0};
        if (Q < p.total_q) {
            const int b = (int)(Q / img);
            const int rem = (int)(Q % img);
            const int r = rem / p.PW - a.pad, c = rem % p.PW - a.pad;
            if (r >= 0 && r < a.H && c >= 0 && c < a.W) {
                const float* src = a.x + (((int64_t)b * a.C) * a.H + r) * a.W + c;
                const int64_t cs = (int64_t)a.H * a.W;
                float v[16];
                #pragma unroll
                for (int e = 0; e < 16; ++e) {
                    const int cc = ch * 16 + perm16(e);
                    v[e] = cc < a.C ? __ldg(src + cc * cs) : 0.0f;
                }
                #pragma unroll
                for (int e = 0; e < 16; ++e) {
                    const int cc = ch * 16 + perm16(e);
                    bool nz, pos;
                    ternarize(v[e], sLo[cc], sHi[cc], nz, pos);
                    const uint32_t byte = pos ? 0x01u : (nz ? 0xFFu : 0x00u);
                    w[e >> 2] |= byte << (8 * (e & 3));
                }
                const int s = __dp4a((int)w[0], 0x01010101, __dp4a((int)w[1], 0x01010101,
                              __dp4a((int)w[2], 0x01010101, __dp4a((int)w[3], 0x01010101, 0))));
                if (s != 0) atomicAdd(&sPsum[pp], s);
            }
        }
        sA[ch * p.ppix + pp] = make_uint4(w[0], w[1], w[2], w[3]);
    }

    // ---- 2. filters: bit planes -> int8, [tap][chunk][n]
    {
        const int cwords = p.Cp / 32;
        const int64_t row_words = ((int64_t)p.T * cwords + 3) / 4 * 4;          // words per plane per row
        const uint32_t* Wp = reinterpret_cast<const uint32_t*>(a.w_packed);
        for (int it = tid; it < p.T * cwords * p.Np; it += kThreads) {
            const int n = it % p.Np;
            const int wd = it / p.Np;                    // word index in the row: t*cwords + cw
            uint32_t nz = 0, sg = 0;
            if (n < a.N) {
                const uint32_t* blk = Wp + ((int64_t)n * (row_words / 4) + wd / 4) * 8;
                nz = __ldg(blk + (wd & 3));
                sg = __ldg(blk + 4 + (wd & 3));
            }
            uint32_t o[8];
            tc::unpack32(nz, sg, o);
            const int t = wd / cwords, cw = wd % cwords;
            uint4* dst = sW + ((int64_t)(t * nchunk + 2 * cw) * p.Np + n);
            dst[0] = make_uint4(o[0], o[1], o[2], o[3]);
            dst[p.Np] = make_uint4(o[4], o[5], o[6], o[7]);
        }
    }
    tc::fence_smem_to_async_proxy();
    tc::tc_fence_before_sync();
    __syncthreads();
    tc::tc_fence_after_sync();
    const uint32_t tmem = *slot;

    // ---- 3. MMAs: for every sub-tile, tap and group of 32 channels
    if (tid == 0) {
        const uint32_t idesc = tc::idesc_i8(kTileM, (uint32_t)p.Np);
        const uint32_t a_base = tc::smem_addr(sA), w_base = tc::smem_addr(sW);
        const uint32_t a_lbo = (uint32_t)p.ppix * 16, w_lbo = (uint32_t)p.Np * 16;
        for (int tm = 0; tm < p.TM; ++tm) {
            bool acc = false;
            for (int t = 0; t < p.T; ++t) {
                const int shift = (t / a.kw) * p.PW + (t % a.kw);
                for (int h = 0; h < p.Cp / 32; ++h) {
                    const uint64_t ad = tc::smem_desc_kmajor(
                        a_base + (uint32_t)(2 * h) * a_lbo + (uint32_t)(tm * kTileM + shift) * 16, a_lbo, 128);
                    const uint64_t bd = tc::smem_desc_kmajor(
                        w_base + (uint32_t)((t * nchunk + 2 * h) * p.Np) * 16, w_lbo, 128);
                    tc::mma_i8_ss(tmem + (uint32_t)(tm * p.Np), ad, bd, idesc, acc);
                    acc = true;
                }
            }
        }
        tc::mma_commit(bar);
    }
    const bool alive = tc::mbar_wait(bar, 0, a.status);
    tc::tc_fence_after_sync();

    // ---- 4. epilogue: out = c1*S_xw + c2*S_x + c3
    {
        const int q = warp & 3, part = warp >> 2;
        for (int tm = 0; tm < p.TM; ++tm) {
            const int pl = tm * kTileM + q * 32 + lane;          // local padded pixel
            const int64_t Q = q0 + pl;
            const int b = (int)(Q / img);
            const int rem = (int)(Q % img);
            const int ho = rem / p.PW, wo = rem % p.PW;
            const bool ok = alive && Q < p.total_q && ho < a.Ho && wo < a.Wo;
            int s_x = 0;
            int n_inside = p.T;
            if (ok) {
                for (int t = 0; t < p.T; ++t) s_x += sPsum[pl + (t / a.kw) * p.PW + (t % a.kw)];
                if (a.pad_mode == RTN_PAD_VALUE_ZERO) {
                    n_inside = 0;
                    for (int t = 0; t < p.T; ++t) {
                        const int h = ho - a.pad + t / a.kw, v = wo - a.pad + t % a.kw;
                        n_inside += (h >= 0 && h < a.H && v >= 0 && v < a.W);
                    }
                }
            }
            const bool border = n_inside < p.T;
            const float fsx = (float)s_x;
            const int64_t obase = (((int64_t)b * a.N) * a.Ho + ho) * a.Wo + wo;
            const int64_t ostride = (int64_t)a.Ho * a.Wo;
            for (int c0 = part * 16; c0 < p.Np; c0 += 32) {
                uint32_t v[16];
                tc::tmem_ld16(tmem + ((uint32_t)(q * 32) << 16) + (uint32_t)(tm * p.Np + c0), v);
                tc::tmem_ld_wait();
                if (!ok) continue;
                #pragma unroll
                for (int j = 0; j < 16; ++j) {
                    const int n = c0 + j;
                    if (n >= a.N) break;
                    const int s_xw = (int)v[j];
                    float c3 = sC3[n];
                    if (border) {
                        // value-zero padding at an image border: S_w and K over inside taps only
                        int s_w = 0;
                        for (int t = 0; t < p.T; ++t) {
                            const int h = ho - a.pad + t / a.kw, vv = wo - a.pad + t % a.kw;
                            if (h >= 0 && h < a.H && vv >= 0 && vv < a.W) s_w += a.w_sum[(1 + t) * a.N + n];
                        }
                        const double ws = a.ep.w_scale[a.ep.n_wparam == 1 ? 0 : n];
                        const double wo_ = a.ep.w_offset[a.ep.n_wparam == 1 ? 0 : n];
                        c3 = (float)((double)a.ep.a_offset_val * (ws * (double)s_w + (double)a.C * n_inside * wo_));
                    }
                    a.out[obase + n * ostride] = fmaf(sC1[n], (float)s_xw, fmaf(sC2[n], fsx, c3));
                    if (a.dbg_acc != nullptr) a.dbg_acc[obase + n * ostride] = s_xw;
                }
            }
        }
    }
    tc::tc_fence_before_sync();
    __syncthreads();
    if (warp == 0) tc::tmem_dealloc(tmem, p.tmem_cols);
}

}  // namespace

bool conv_i8_supported(const ConvArgs& c)
{
    ConvI8Plan p;
    return make_plan(c, p);
}

cudaError_t launch_conv_i8(const ConvArgs& c, cudaStream_t s)
{
    ConvI8Plan p;
    if (!make_plan(c, p)) return cudaErrorInvalidConfiguration;
    cudaError_t e = cudaFuncSetAttribute(conv_i8_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                         (int)p.smem_bytes);
    if (e != cudaSuccess) return e;
    const int64_t grid = (p.total_q + (int64_t)p.TM * kTileM - 1) / ((int64_t)p.TM * kTileM);
    conv_i8_kernel<<<(unsigned)grid, kThreads, p.smem_bytes, s>>>(c, p);
    return cudaGetLastError();
}

}  // namespace rtn
