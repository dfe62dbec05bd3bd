// Ternary conv2d as an implicit GEMM, bit-plane variant (any filter size, stride, padding).
//
// One CTA: one image, an 8x8 tile of output pixels, 64 output channels.  Per pass over at most
// 256 input channels it
//   1. ternarizes the fp32 input patch the tile needs (Eq. 3) into channel-packed bit planes in
//      shared memory (bit c mod 32 of word c div 32 of a pixel; code 0 outside the image) and
//      records each pixel's code sum,
//   2. copies the matching slice of the packed filters into shared memory,
//   3. evaluates Eq. 9 for 16 outputs per thread: the im2col patch is never built, a filter tap
//      (i, j) just reads the plane words of the pixel shifted by (i, j).
// The epilogue is the four-term affine form in double, rounded once to fp32.
#include "rtn_internal.cuh"

namespace rtn {

constexpr int kTH = 8, kTW = 8;           // output tile
constexpr int kNB = 64;                   // output channels per CTA
constexpr int kCW = 8;                    // channel words (of 32) per pass

__global__ void __launch_bounds__(256)
conv_popc_kernel(const ConvArgs a, int PH, int PW)
{
    extern __shared__ uint32_t smem[];
    const int T = a.kh * a.kw;
    const int PP = PH * PW;                                   // patch pixels
    uint32_t* sP = smem;                                      // [2][kCW][PP]
    uint32_t* sW = sP + 2 * kCW * PP;                         // [2][T][kCW][kNB]
    int* sSum = reinterpret_cast<int*>(sW + 2 * T * kCW * kNB);   // [PP]

    const int tid = threadIdx.x;
    const int tx = tid & 15, ty = tid >> 4;
    const int tiles_w = (a.Wo + kTW - 1) / kTW;
    const int ho0 = (blockIdx.x / tiles_w) * kTH, wo0 = (blockIdx.x % tiles_w) * kTW;
    const int n0 = blockIdx.y * kNB;
    const int b = blockIdx.z;
    const int h0 = ho0 * a.stride - a.pad, v0 = wo0 * a.stride - a.pad;   // patch origin
    const int cwords = (a.C + 31) / 32;
    const int64_t w_row_words = ((int64_t)T * cwords + 3) / 4 * 4;        // words per plane per row
    const uint32_t* __restrict__ Wp = reinterpret_cast<const uint32_t*>(a.w_packed);
    const float lo0 = a.t_lo[0], hi0 = a.t_hi[0];

    int pbase[4];                      // patch index of each of my pixels' (0,0) tap
    #pragma unroll
    for (int i = 0; i < 4; ++i) {
        const int p = tx + 16 * i;
        pbase[i] = ((p >> 3) * a.stride) * PW + (p & 7) * a.stride;
    }
    int cnt_c[4][4], cnt_d[4][4], s_x[4];
    #pragma unroll
    for (int i = 0; i < 4; ++i) {
        s_x[i] = 0;
        #pragma unroll
        for (int j = 0; j < 4; ++j) { cnt_c[i][j] = 0; cnt_d[i][j] = 0; }
    }

    for (int cw0 = 0; cw0 < cwords; cw0 += kCW) {
        const int ncw = min(kCW, cwords - cw0);
        __syncthreads();
        for (int i = tid; i < PP; i += 256) sSum[i] = 0;
        __syncthreads();
        // 1. ternarize the patch: item = (channel word, patch pixel), pixel fastest
        for (int it = tid; it < ncw * PP; it += 256) {
            const int cw = it / PP, pp = it % PP;
            const int h = h0 + pp / PW, v = v0 + pp % PW;
            uint32_t nz = 0, sg = 0;
            if (h >= 0 && h < a.H && v >= 0 && v < a.W) {
                const int c0 = (cw0 + cw) * 32;
                const float* src = a.x + (((int64_t)b * a.C + c0) * a.H + h) * a.W + v;
                const int cmax = min(32, a.C - c0);
                for (int c = 0; c < cmax; ++c) {
                    const float val = __ldg(src + (int64_t)c * a.H * a.W);
                    const float lo = a.n_thr == 1 ? lo0 : __ldg(a.t_lo + c0 + c);
                    const float hi = a.n_thr == 1 ? hi0 : __ldg(a.t_hi + c0 + c);
                    bool z, p;
                    ternarize(val, lo, hi, z, p);
                    nz |= (uint32_t)z << c;
                    sg |= (uint32_t)p << c;
                }
            }
            sP[(0 * kCW + cw) * PP + pp] = nz;
            sP[(1 * kCW + cw) * PP + pp] = sg;
            const int s = __popc(nz & sg) - __popc(nz & ~sg);
            if (s != 0) atomicAdd(&sSum[pp], s);
        }
        // 2. filter slice: sW[plane][t][cw][n]
        for (int it = tid; it < 2 * T * ncw * kNB; it += 256) {
            const int n = it % kNB;
            int r = it / kNB;
            const int cw = r % ncw; r /= ncw;
            const int t = r % T;
            const int plane = r / T;
            uint32_t v = 0;
            if (n0 + n < a.N) {
                const int64_t wd = (int64_t)t * cwords + cw0 + cw;     // word index in the row
                v = __ldg(Wp + ((int64_t)(n0 + n) * (w_row_words / 4) + wd / 4) * 8 + plane * 4 + wd % 4);
            }
            sW[((plane * T + t) * kCW + cw) * kNB + n] = v;
        }
        __syncthreads();
        // 3. Eq. 9
        for (int t = 0; t < T; ++t) {
            const int off = (t / a.kw) * PW + (t % a.kw);
            #pragma unroll
            for (int i = 0; i < 4; ++i) s_x[i] += sSum[pbase[i] + off];
            for (int cw = 0; cw < ncw; ++cw) {
                uint32_t a1[4], a2[4], w1[4], w2[4];
                #pragma unroll
                for (int i = 0; i < 4; ++i) {
                    a1[i] = sP[(0 * kCW + cw) * PP + pbase[i] + off];
                    a2[i] = sP[(1 * kCW + cw) * PP + pbase[i] + off];
                }
                #pragma unroll
                for (int j = 0; j < 4; ++j) {
                    w1[j] = sW[((0 * T + t) * kCW + cw) * kNB + ty + 16 * j];
                    w2[j] = sW[((1 * T + t) * kCW + cw) * kNB + ty + 16 * j];
                }
                #pragma unroll
                for (int i = 0; i < 4; ++i)
                    #pragma unroll
                    for (int j = 0; j < 4; ++j) {
                        const uint32_t c = a1[i] & w1[j];
                        const uint32_t d = (a2[i] ^ w2[j]) & c;
                        cnt_c[i][j] += __popc(c);
                        cnt_d[i][j] += __popc(d);
                    }
            }
        }
    }

    // Epilogue
    const EpilogueParams& ep = a.ep;
    const double a_s = ep.a_scale_val, a_o = ep.a_offset_val;
    #pragma unroll
    for (int i = 0; i < 4; ++i) {
        const int p = tx + 16 * i;
        const int ho = ho0 + (p >> 3), wo = wo0 + (p & 7);
        if (ho >= a.Ho || wo >= a.Wo) continue;
        // taps inside the image (all of them for interior pixels)
        int n_inside = 0;
        for (int t = 0; t < T; ++t) {
            const int h = ho * a.stride - a.pad + t / a.kw, v = wo * a.stride - a.pad + t % a.kw;
            n_inside += (h >= 0 && h < a.H && v >= 0 && v < a.W);
        }
        const bool border = (a.pad_mode == RTN_PAD_VALUE_ZERO) && (n_inside < T);
        #pragma unroll
        for (int j = 0; j < 4; ++j) {
            const int n = n0 + ty + 16 * j;
            if (n >= a.N) continue;
            int s_w = a.w_sum[n];
            double k_eff = (double)a.C * T;
            if (border) {
                s_w = 0;
                for (int t = 0; t < T; ++t) {
                    const int h = ho * a.stride - a.pad + t / a.kw, v = wo * a.stride - a.pad + t % a.kw;
                    if (h >= 0 && h < a.H && v >= 0 && v < a.W) s_w += a.w_sum[(1 + t) * a.N + n];
                }
                k_eff = (double)a.C * n_inside;
            }
            const int s_xw = cnt_c[i][j] - 2 * cnt_d[i][j];
            const double w_s = ep.w_scale[ep.n_wparam == 1 ? 0 : n];
            const double w_o = ep.w_offset[ep.n_wparam == 1 ? 0 : n];
            const int64_t o = (((int64_t)b * a.N + n) * a.Ho + ho) * a.Wo + wo;
            a.out[o] = epilogue_f64(s_xw, s_x[i], s_w, k_eff, a_s, a_o, w_s, w_o);
            if (a.dbg_acc != nullptr) a.dbg_acc[o] = s_xw;
        }
    }
}

static size_t conv_popc_smem(const ConvArgs& c, int& PH, int& PW)
{
    PH = (kTH - 1) * c.stride + c.kh;
    PW = (kTW - 1) * c.stride + c.kw;
    const size_t PP = (size_t)PH * PW, T = (size_t)c.kh * c.kw;
    return 4 * (2 * kCW * PP + 2 * T * kCW * kNB + PP);
}

bool conv_popc_supported(const ConvArgs& c)
{
    int PH, PW;
    return conv_popc_smem(c, PH, PW) <= 200 * 1024 && c.B <= 65535 && (c.N + kNB - 1) / kNB <= 65535;
}

cudaError_t launch_conv_popc(const ConvArgs& c, cudaStream_t s)
{
    int PH, PW;
    const size_t smem = conv_popc_smem(c, PH, PW);
    if (!conv_popc_supported(c)) return cudaErrorInvalidConfiguration;
    cudaError_t e = cudaFuncSetAttribute(conv_popc_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                         (int)smem);
    if (e != cudaSuccess) return e;
    const int tiles = ((c.Ho + kTH - 1) / kTH) * ((c.Wo + kTW - 1) / kTW);
    dim3 grid((unsigned)tiles, (unsigned)((c.N + kNB - 1) / kNB), (unsigned)c.B);
    conv_popc_kernel<<<grid, 256, smem, s>>>(c, PH, PW);
    return cudaGetLastError();
}

}  // namespace rtn
