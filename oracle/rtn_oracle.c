/*
 * TEST INFRASTRUCTURE -- not part of the product.
 *
 * Plain, slow CPU oracle for the forward ternary-by-ternary contraction of the
 * Reparameterized Ternary Network (RTN, arXiv 1912.02057).  Every function is the
 * definition written out: exact integer sums in int64 by nested loops, floating
 * point in double.  No blocking, no bit tricks (except orc_dot_eq9, which IS the
 * paper's bit formula and exists so that tests can pin it against the plain sum),
 * no code shared with the CUDA library.  OpenMP pragmas only split the outermost
 * loop over independent outputs; they change no arithmetic.
 *
 * Only the tests, the smoke check and the benchmark's CPU-baseline leg may call
 * this file.
 *
 * Notation (paper, section "Efficient Computation Pattern"):
 *   x  activation code in {-1,0,+1}   (paper: A^t)
 *   w  weight code in {-1,0,+1}       (paper: W^t)
 *   a_s, a_o  activation scale / offset (paper: gamma, beta; Eq. 4)
 *   w_s, w_o  weight scale / offset     (paper: alpha; the paper fixes w_o = 0, Eq. 5 ff.)
 *   S_xw = sum_k x*w,  S_x = sum_k x,  S_w = sum_k w
 */
#include <stdint.h>
#include <stddef.h>
#include <math.h>

/* ------------------------------------------------------------------------- */
/* Eq. 3: ternarize against a threshold pair.  With the BN transform A' = kA+b  */
/* (Eq. 2, k > 0) the thresholds are t_hi = (0.5-b)/k and t_lo = -(0.5+b)/k.    */
/* Both comparisons are strict (Eq. 1 and Eq. 3 use > and <), so a value equal  */
/* to a threshold, and a NaN, give code 0.  The +1 case is tested first, as the */
/* equation lists it first.                                                     */
/* Tensor viewed as [outer][chan][inner]; threshold index = chan (n_thr==chan)  */
/* or 0 (n_thr==1).                                                             */
/* ------------------------------------------------------------------------- */
void orc_ternarize(const float *a, int64_t outer, int64_t chan, int64_t inner,
                   const float *t_lo, const float *t_hi, int64_t n_thr,
                   int8_t *codes)
{
    for (int64_t o = 0; o < outer; ++o)
        for (int64_t c = 0; c < chan; ++c) {
            const float lo = t_lo[n_thr == 1 ? 0 : c];
            const float hi = t_hi[n_thr == 1 ? 0 : c];
            for (int64_t i = 0; i < inner; ++i) {
                const int64_t idx = (o * chan + c) * inner + i;
                const float v = a[idx];
                int8_t t = 0;
                if (v > hi) t = 1;
                else if (v < lo) t = -1;
                codes[idx] = t;
            }
        }
}

/* Eq. 1 applied to the BN-transformed value of Eq. 2, evaluated in double:     */
/* Q(k*A + b) with Q(v) = sign(v) if |v| > 0.5 else 0.  Used to pin Eq. 3.      */
void orc_ternarize_eq1_of_eq2(const double *a, int64_t n, double k, double b, int8_t *codes)
{
    for (int64_t i = 0; i < n; ++i) {
        const double v = k * a[i] + b;
        int8_t t = 0;
        if (fabs(v) > 0.5) t = (v > 0.0) ? 1 : -1;
        codes[i] = t;
    }
}

/* ------------------------------------------------------------------------- */
/* Table 1: two-bit encoding.  first bit = "is non-zero", second bit = sign,    */
/* rows 00->0, 01->0, 10->-1, 11->+1.  One bit per byte here, for readability.  */
/* The encoder always emits the canonical zero 00.                              */
/* ------------------------------------------------------------------------- */
void orc_encode_bits(const int8_t *codes, int64_t n, uint8_t *bit1, uint8_t *bit2)
{
    for (int64_t i = 0; i < n; ++i) {
        bit1[i] = (codes[i] != 0);
        bit2[i] = (codes[i] > 0);
    }
}

void orc_decode_bits(const uint8_t *bit1, const uint8_t *bit2, int64_t n, int8_t *codes)
{
    for (int64_t i = 0; i < n; ++i) {
        if (!bit1[i]) codes[i] = 0;              /* 00 and 01 */
        else codes[i] = bit2[i] ? 1 : -1;        /* 11 and 10 */
    }
}

/* Eq. 9: (W^t)^T A^t = bC(c) - 2*bC((W2 xor A2) and c),  c = W1 and A1.        */
int64_t orc_dot_eq9(const uint8_t *w1, const uint8_t *w2,
                    const uint8_t *a1, const uint8_t *a2, int64_t n)
{
    int64_t count_c = 0, count_d = 0;
    for (int64_t i = 0; i < n; ++i) {
        const uint8_t c = w1[i] & a1[i];
        const uint8_t d = (uint8_t)((w2[i] ^ a2[i]) & c);
        count_c += c;
        count_d += d;
    }
    return count_c - 2 * count_d;
}

/* ------------------------------------------------------------------------- */
/* The library's packed operand format (its public header defines it; this is   */
/* an independent writer of the same format):                                   */
/*   a row of K codes occupies ceil(K/128) blocks of 32 bytes;                  */
/*   block j, bytes 0..15  = first-bit plane of codes 128j..128j+127,           */
/*   block j, bytes 16..31 = second-bit plane of the same codes;                */
/*   code 128j+i sits in bit (i mod 8) of byte (i div 8) of its plane;          */
/*   positions past K hold 00.                                                  */
/* ------------------------------------------------------------------------- */
int64_t orc_packed_row_bytes(int64_t K) { return ((K + 127) / 128) * 32; }

void orc_pack_rows(const int8_t *codes, int64_t rows, int64_t K, uint8_t *out)
{
    const int64_t rb = orc_packed_row_bytes(K);
    for (int64_t r = 0; r < rows; ++r) {
        uint8_t *row = out + r * rb;
        for (int64_t i = 0; i < rb; ++i) row[i] = 0;
        for (int64_t k = 0; k < K; ++k) {
            const int8_t t = codes[r * K + k];
            const int64_t blk = k / 128, i = k % 128;
            if (t != 0) row[blk * 32 + i / 8] |= (uint8_t)(1u << (i % 8));
            if (t > 0)  row[blk * 32 + 16 + i / 8] |= (uint8_t)(1u << (i % 8));
        }
    }
}

void orc_unpack_rows(const uint8_t *packed, int64_t rows, int64_t K, int8_t *codes)
{
    const int64_t rb = orc_packed_row_bytes(K);
    for (int64_t r = 0; r < rows; ++r) {
        const uint8_t *row = packed + r * rb;
        for (int64_t k = 0; k < K; ++k) {
            const int64_t blk = k / 128, i = k % 128;
            const int b1 = (row[blk * 32 + i / 8] >> (i % 8)) & 1;
            const int b2 = (row[blk * 32 + 16 + i / 8] >> (i % 8)) & 1;
            codes[r * K + k] = (int8_t)(b1 ? (b2 ? 1 : -1) : 0);
        }
    }
}

/* Convolution filters [N][C][kh][kw] are stored as rows of length                  */
/* kh*kw*Cw, Cw = C rounded up to 32, in (kh, kw, c) order (the im2col patch of the */
/* paper's section "Methodology", with the channel innermost); channel padding = 0. */
void orc_conv_weight_rows(const int8_t *w, int64_t N, int64_t C, int64_t kh, int64_t kw,
                          int8_t *rows /* [N][kh*kw*Cw] */)
{
    const int64_t Cw = ((C + 31) / 32) * 32;
    const int64_t Kc = kh * kw * Cw;
    for (int64_t n = 0; n < N; ++n)
        for (int64_t i = 0; i < kh; ++i)
            for (int64_t j = 0; j < kw; ++j)
                for (int64_t c = 0; c < Cw; ++c)
                    rows[n * Kc + (i * kw + j) * Cw + c] =
                        (c < C) ? w[((n * C + c) * kh + i) * kw + j] : 0;
}

/* ------------------------------------------------------------------------- */
/* GEMM sums, by definition.  x [M][K], w [N][K], codes as int8.               */
/* ------------------------------------------------------------------------- */
void orc_gemm_sums(const int8_t *x, const int8_t *w, int64_t M, int64_t N, int64_t K,
                   int64_t *S_xw /* [M][N] */, int64_t *S_x /* [M] */, int64_t *S_w /* [N] */)
{
    #pragma omp parallel for schedule(static)
    for (int64_t m = 0; m < M; ++m) {
        int64_t sx = 0;
        for (int64_t k = 0; k < K; ++k) sx += x[m * K + k];
        S_x[m] = sx;
        for (int64_t n = 0; n < N; ++n) {
            int64_t s = 0;
            for (int64_t k = 0; k < K; ++k)
                s += (int64_t)x[m * K + k] * (int64_t)w[n * K + k];
            S_xw[m * N + n] = s;
        }
    }
    for (int64_t n = 0; n < N; ++n) {
        int64_t sw = 0;
        for (int64_t k = 0; k < K; ++k) sw += w[n * K + k];
        S_w[n] = sw;
    }
}

/* ------------------------------------------------------------------------- */
/* Affine epilogue.  sum_k (a_s*x + a_o)(w_s*w + w_o) expanded:                 */
/*   a_s*w_s*S_xw + a_s*w_o*S_x + a_o*w_s*S_w + K*a_o*w_o                       */
/* (Eq. 10 is the w_o = 0 case: alpha*gamma*S_xw + alpha*beta*S_w.)             */
/* a_* per layer (n_aparam==1) or per row; w_* per layer or per column.         */
/* mag receives sum of |term_i|, the scale the fp32 tolerance is stated against.*/
/* ------------------------------------------------------------------------- */
void orc_epilogue(const int64_t *S_xw, const int64_t *S_x, const int64_t *S_w,
                  int64_t M, int64_t N, int64_t K,
                  const float *a_s, const float *a_o, int64_t n_aparam,
                  const float *w_s, const float *w_o, int64_t n_wparam,
                  double *out, double *mag)
{
    for (int64_t m = 0; m < M; ++m) {
        const double as = a_s[n_aparam == 1 ? 0 : m], ao = a_o[n_aparam == 1 ? 0 : m];
        for (int64_t n = 0; n < N; ++n) {
            const double ws = w_s[n_wparam == 1 ? 0 : n], wo = w_o[n_wparam == 1 ? 0 : n];
            const double t1 = as * ws * (double)S_xw[m * N + n];
            const double t2 = as * wo * (double)S_x[m];
            const double t3 = ao * ws * (double)S_w[n];
            const double t4 = (double)K * ao * wo;
            out[m * N + n] = t1 + t2 + t3 + t4;
            if (mag) mag[m * N + n] = fabs(t1) + fabs(t2) + fabs(t3) + fabs(t4);
        }
    }
}

/* ------------------------------------------------------------------------- */
/* Convolution, by definition, one output point at a time.                      */
/* x codes [B][C][H][W], w codes [N][C][kh][kw], out [B][N][Ho][Wo].            */
/* pad_mode 0 (code-zero): a tap outside the image has CODE 0, i.e. real value  */
/*   a_o; S_w and K run over all C*kh*kw taps, so the constant of Eq. 10 is one */
/*   number per output channel, as the paper says it can be pre-stored.         */
/* pad_mode 1 (value-zero): a tap outside the image contributes nothing; S_w and*/
/*   K run over the taps inside the image only.                                 */
/* ------------------------------------------------------------------------- */
typedef struct {
    int64_t S_xw, S_x, S_w, K_eff;
} orc_conv_sums;

static orc_conv_sums conv_point(const int8_t *x, const int8_t *w,
                                int64_t C, int64_t H, int64_t W, int64_t kh, int64_t kw,
                                int64_t stride, int64_t pad, int pad_mode,
                                int64_t b, int64_t n, int64_t ho, int64_t wo)
{
    orc_conv_sums s = {0, 0, 0, 0};
    for (int64_t c = 0; c < C; ++c)
        for (int64_t i = 0; i < kh; ++i)
            for (int64_t j = 0; j < kw; ++j) {
                const int64_t h = ho * stride - pad + i;
                const int64_t v = wo * stride - pad + j;
                const int inside = (h >= 0 && h < H && v >= 0 && v < W);
                const int64_t wc = w[((n * C + c) * kh + i) * kw + j];
                if (inside) {
                    const int64_t xc = x[((b * C + c) * H + h) * W + v];
                    s.S_xw += xc * wc;
                    s.S_x += xc;
                    s.S_w += wc;
                    s.K_eff += 1;
                } else if (pad_mode == 0) {
                    s.S_w += wc;      /* code 0 there: adds nothing to S_xw, S_x */
                    s.K_eff += 1;
                }
            }
    return s;
}

static double conv_value(orc_conv_sums s, double as, double ao, double ws, double wo, double *mag)
{
    const double t1 = as * ws * (double)s.S_xw;
    const double t2 = as * wo * (double)s.S_x;
    const double t3 = ao * ws * (double)s.S_w;
    const double t4 = (double)s.K_eff * ao * wo;
    if (mag) *mag = fabs(t1) + fabs(t2) + fabs(t3) + fabs(t4);
    return t1 + t2 + t3 + t4;
}

int64_t orc_conv_out_dim(int64_t in, int64_t k, int64_t stride, int64_t pad)
{
    return (in + 2 * pad - k) / stride + 1;
}

void orc_conv2d(const int8_t *x, const int8_t *w,
                int64_t B, int64_t C, int64_t H, int64_t W,
                int64_t N, int64_t kh, int64_t kw, int64_t stride, int64_t pad, int pad_mode,
                float a_s, float a_o, const float *w_s, const float *w_o, int64_t n_wparam,
                int64_t *S_xw /* [B][N][Ho][Wo], nullable */,
                double *out /* same shape */, double *mag /* nullable */)
{
    const int64_t Ho = orc_conv_out_dim(H, kh, stride, pad);
    const int64_t Wo = orc_conv_out_dim(W, kw, stride, pad);
    #pragma omp parallel for collapse(2) schedule(static)
    for (int64_t b = 0; b < B; ++b)
        for (int64_t n = 0; n < N; ++n) {
            const double ws = w_s[n_wparam == 1 ? 0 : n], wo = w_o[n_wparam == 1 ? 0 : n];
            for (int64_t ho = 0; ho < Ho; ++ho)
                for (int64_t q = 0; q < Wo; ++q) {
                    const orc_conv_sums s =
                        conv_point(x, w, C, H, W, kh, kw, stride, pad, pad_mode, b, n, ho, q);
                    const int64_t o = ((b * N + n) * Ho + ho) * Wo + q;
                    if (S_xw) S_xw[o] = s.S_xw;
                    out[o] = conv_value(s, a_s, a_o, ws, wo, mag ? &mag[o] : NULL);
                }
        }
}

/* The same definition at a list of output points (b, n, ho, wo), for checking  */
/* samples of outputs too large to compute in full.                             */
void orc_conv2d_points(const int8_t *x, const int8_t *w,
                       int64_t B, int64_t C, int64_t H, int64_t W,
                       int64_t N, int64_t kh, int64_t kw, int64_t stride, int64_t pad, int pad_mode,
                       float a_s, float a_o, const float *w_s, const float *w_o, int64_t n_wparam,
                       const int64_t *pts /* [n_pts][4] */, int64_t n_pts,
                       int64_t *S_xw /* [n_pts] */, double *out, double *mag)
{
    (void)B; (void)N;
    #pragma omp parallel for schedule(static)
    for (int64_t p = 0; p < n_pts; ++p) {
        const int64_t b = pts[4 * p], n = pts[4 * p + 1], ho = pts[4 * p + 2], q = pts[4 * p + 3];
        const double ws = w_s[n_wparam == 1 ? 0 : n], wo = w_o[n_wparam == 1 ? 0 : n];
        const orc_conv_sums s =
            conv_point(x, w, C, H, W, kh, kw, stride, pad, pad_mode, b, n, ho, q);
        S_xw[p] = s.S_xw;
        out[p] = conv_value(s, a_s, a_o, ws, wo, mag ? &mag[p] : NULL);
    }
}

/* Per-tap weight code sums [1 + kh*kw][N]: entry 0 = sum over all taps and     */
/* channels, entry 1+t = sum over channels of tap t (t = i*kw + j).             */
void orc_conv_weight_sums(const int8_t *w, int64_t N, int64_t C, int64_t kh, int64_t kw,
                          int64_t *sums)
{
    const int64_t T = kh * kw;
    for (int64_t n = 0; n < N; ++n) {
        int64_t tot = 0;
        for (int64_t t = 0; t < T; ++t) {
            int64_t s = 0;
            for (int64_t c = 0; c < C; ++c) s += w[(n * C + c) * T + t];
            sums[(1 + t) * N + n] = s;
            tot += s;
        }
        sums[n] = tot;
    }
}

/* Materialised im2col (oracle-side only): rows (b,ho,wo), columns (c,kh,kw) in */
/* the filter's own memory order, code 0 outside the image.  Used to pin        */
/* orc_conv2d (code-zero mode) against orc_gemm_sums.                           */
void orc_im2col(const int8_t *x, int64_t B, int64_t C, int64_t H, int64_t W,
                int64_t kh, int64_t kw, int64_t stride, int64_t pad, int8_t *cols)
{
    const int64_t Ho = orc_conv_out_dim(H, kh, stride, pad);
    const int64_t Wo = orc_conv_out_dim(W, kw, stride, pad);
    const int64_t K = C * kh * kw;
    for (int64_t b = 0; b < B; ++b)
        for (int64_t ho = 0; ho < Ho; ++ho)
            for (int64_t q = 0; q < Wo; ++q) {
                int8_t *row = cols + ((b * Ho + ho) * Wo + q) * K;
                for (int64_t c = 0; c < C; ++c)
                    for (int64_t i = 0; i < kh; ++i)
                        for (int64_t j = 0; j < kw; ++j) {
                            const int64_t h = ho * stride - pad + i, v = q * stride - pad + j;
                            const int inside = (h >= 0 && h < H && v >= 0 && v < W);
                            row[(c * kh + i) * kw + j] =
                                inside ? x[((b * C + c) * H + h) * W + v] : 0;
                        }
            }
}

/* Direct evaluation, term by term in double, of sum_k (a_s*x_k + a_o)(w_s*w_k + w_o). */
/* Independent of the four-term expansion; for tiny inputs only.                       */
double orc_direct_dot(const int8_t *x, const int8_t *w, int64_t K,
                      double a_s, double a_o, double w_s, double w_o)
{
    double acc = 0.0;
    for (int64_t k = 0; k < K; ++k)
        acc += (a_s * (double)x[k] + a_o) * (w_s * (double)w[k] + w_o);
    return acc;
}

/* ------------------------------------------------------------------------- */
/* What a ternary layer hands to the next one.  Eq. 10 wraps the affine form in */
/* phi (ReLU); the residual block then adds its skip connection; the next       */
/* layer's BN (placed after the ReLU, section "Activation Ternarization") is    */
/* folded into a threshold pair per channel and Eq. 3 ternarizes:               */
/*     y    = phi(pre) + skip          (phi and skip each optional)             */
/*     code = +1 if y > t_hi[n], -1 if y < t_lo[n], else 0                      */
/* y is evaluated in double.  The code is decided on y rounded to fp32 with     */
/* fp32 comparisons, the precision the layer's consumer decides in.  margin is  */
/* the distance of the double y to the nearer threshold: where it is below the  */
/* fp32 rounding error of y, the neighbouring code is as valid.                 */
/* Tensors are [B][N][inner]; thresholds per layer (n_thr == 1) or channel n.   */
/* ------------------------------------------------------------------------- */
void orc_next_layer(const double *pre, const float *skip /* nullable */, int relu,
                    int64_t B, int64_t N, int64_t inner,
                    const float *t_lo, const float *t_hi, int64_t n_thr,
                    double *y /* out */, int8_t *codes /* out */, double *margin /* out */)
{
    for (int64_t b = 0; b < B; ++b)
        for (int64_t n = 0; n < N; ++n) {
            const float lo = t_lo[n_thr == 1 ? 0 : n];
            const float hi = t_hi[n_thr == 1 ? 0 : n];
            for (int64_t i = 0; i < inner; ++i) {
                const int64_t idx = (b * N + n) * inner + i;
                double v = pre[idx];
                if (relu && !(v > 0.0)) v = 0.0;
                if (skip) v += (double)skip[idx];
                y[idx] = v;
                const float vf = (float)v;
                int8_t t = 0;
                if (vf > hi) t = 1;
                else if (vf < lo) t = -1;
                codes[idx] = t;
                const double d_hi = fabs(v - (double)hi), d_lo = fabs(v - (double)lo);
                margin[idx] = d_hi < d_lo ? d_hi : d_lo;
            }
        }
}

/* ------------------------------------------------------------------------- */
/* The paper's comparison workload: 2-bit quaternary weights and activations    */
/* (Table 1, last column: bits (b1, b2) stand for the value 2*b1 + b2 in        */
/* {0, 1, 2, 3}), dot product in the DoReFa-Net pattern the section "Efficient  */
/* Computation Pattern" cites: AND between each bit plane of the two inputs,    */
/* popcount, power-of-two shifts, four partial sums.                            */
/* ------------------------------------------------------------------------- */
void orc_quaternary_decode(const uint8_t *bit1, const uint8_t *bit2, int64_t n, uint8_t *values)
{
    for (int64_t i = 0; i < n; ++i) values[i] = (uint8_t)(2 * (bit1[i] != 0) + (bit2[i] != 0));
}

void orc_quaternary_encode(const uint8_t *values, int64_t n, uint8_t *bit1, uint8_t *bit2)
{
    for (int64_t i = 0; i < n; ++i) {
        bit1[i] = (uint8_t)((values[i] >> 1) & 1);
        bit2[i] = (uint8_t)(values[i] & 1);
    }
}

/* The definition: plain sums of products of the values, int64. */
void orc_quaternary_gemm(const uint8_t *x, const uint8_t *w, int64_t M, int64_t N, int64_t K,
                         int64_t *S /* [M][N] */)
{
    #pragma omp parallel for schedule(static)
    for (int64_t m = 0; m < M; ++m)
        for (int64_t n = 0; n < N; ++n) {
            int64_t s = 0;
            for (int64_t k = 0; k < K; ++k) s += (int64_t)x[m * K + k] * (int64_t)w[n * K + k];
            S[m * N + n] = s;
        }
}

/* The bit formula (exists to be pinned against the plain sum):                 */
/*   x.w = 4 bC(X1&W1) + 2 bC(X1&W2) + 2 bC(X2&W1) + bC(X2&W2)                  */
int64_t orc_dot_quaternary_bits(const uint8_t *x1, const uint8_t *x2,
                                const uint8_t *w1, const uint8_t *w2, int64_t n)
{
    int64_t c11 = 0, c12 = 0, c21 = 0, c22 = 0;
    for (int64_t i = 0; i < n; ++i) {
        c11 += (x1[i] & w1[i]) & 1;
        c12 += (x1[i] & w2[i]) & 1;
        c21 += (x2[i] & w1[i]) & 1;
        c22 += (x2[i] & w2[i]) & 1;
    }
    return (c11 << 2) + (c12 << 1) + (c21 << 1) + c22;
}

/* Packed rows of quaternary values: the library's block-plane format with      */
/* plane 1 = first bit (weight 2) and plane 2 = second bit (weight 1).          */
void orc_pack_quaternary_rows(const uint8_t *values, int64_t rows, int64_t K, uint8_t *out)
{
    const int64_t rb = orc_packed_row_bytes(K);
    for (int64_t r = 0; r < rows; ++r) {
        uint8_t *row = out + r * rb;
        for (int64_t i = 0; i < rb; ++i) row[i] = 0;
        for (int64_t k = 0; k < K; ++k) {
            const uint8_t v = values[r * K + k];
            uint8_t *blk = row + (k / 128) * 32;
            const int64_t i = k % 128;
            if (v & 2) blk[i / 8] |= (uint8_t)(1u << (i % 8));
            if (v & 1) blk[16 + i / 8] |= (uint8_t)(1u << (i % 8));
        }
    }
}
