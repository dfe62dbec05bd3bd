/*
 * rtn.h -- C ABI of librtn_b200: the forward ternary-by-ternary contraction of the
 * Reparameterized Ternary Network (RTN, arXiv 1912.02057) on NVIDIA B200 (sm_100a).
 *
 * Path: ternarize + pack (Eq. 1-3, Table 1)  ->  packed ternary GEMM / implicit-GEMM conv2d
 * (Eq. 9)  ->  affine scale/offset epilogue (Eq. 10, generalised to a weight offset).
 *
 * Conventions
 *   - Every data pointer is a DEVICE pointer unless its comment says "host".  The caller owns
 *     every input and output buffer.  The library keeps no state besides one device status word (see
 *     rtn_last_device_status) and, per device, the fixed scratch array of rtn_ternary_conv2d_noalloc.
 *     Convolutions that take the two-kernel path (rtn_conv_kernel_launches / rtn_conv_next_kernel_launches
 *     say which) borrow a scratch buffer from the stream-ordered allocator for the duration of the call
 *     (cudaMallocAsync / cudaFreeAsync on `stream`), and so does the tensor-core GEMM for its expanded
 *     operands (rtn_gemm_kernel_launches); nothing else is allocated.
 *   - `stream` is a cudaStream_t passed as void* (NULL = the default stream).  Calls only
 *     enqueue work and return without synchronising, except rtn_pack_weights and
 *     rtn_last_device_status, which synchronise the stream.
 *   - Errors are return codes; argument errors are found on the host before any launch and
 *     leave every buffer untouched.  Nothing throws, aborts or traps.
 *   - Codes: x (activation) and w (weight) in {-1, 0, +1}.  S_xw = sum_k x*w, S_x = sum_k x,
 *     S_w = sum_k w (exact int32; |S| <= K <= 2^24).
 *
 * Packed operand format (Table 1 and the bit-plane vectors W1, W2, A1, A2 of Eq. 9)
 *   A row of K codes occupies ceil(K/128) blocks of 32 bytes (2 bits per code):
 *     block j, bytes  0..15 : plane 1 ("non-zero" bit) of codes 128j .. 128j+127
 *     block j, bytes 16..31 : plane 2 ("sign" bit, 1 = positive) of the same codes
 *   Code 128j+i sits in bit (i mod 8) of byte (i div 8) of its plane (little-endian words:
 *   bit (i mod 32) of 32-bit word (i div 32)).  Table 1: 00 -> 0, 01 -> 0, 10 -> -1, 11 -> +1.
 *   The packers emit the canonical zero 00 and zero-fill positions past K; every consumer also
 *   accepts 01 as zero.  Rows are contiguous: row stride = rtn_packed_row_bytes(K).  Packed
 *   buffers must be 16-byte aligned.
 *   Convolution filters [N][C][kh][kw] are packed as rows of length rtn_conv_packed_k(C,kh,kw)
 *   = kh*kw*Cw, Cw = C rounded up to 32, in (kh, kw, c) order with zero codes in the channel
 *   padding (the im2col patch of the paper's "Methodology" section, channel innermost).
 */
#ifndef RTN_H_
#define RTN_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
    RTN_OK = 0,
    RTN_ERR_NULL = 1,           /* a required pointer is NULL                                  */
    RTN_ERR_SHAPE = 2,          /* a size is <= 0, too large, or inconsistent                  */
    RTN_ERR_ALIGN = 3,          /* a buffer misses its alignment                               */
    RTN_ERR_VALUE = 4,          /* a weight code outside {-1,0,+1}, or a bad enum value        */
    RTN_ERR_UNSUPPORTED = 5,    /* the requested variant cannot run this shape                 */
    RTN_ERR_CUDA = 6,           /* a CUDA runtime call failed (launch, attribute, copy)        */
    RTN_ERR_DEVICE_TIMEOUT = 7  /* a bounded device-side wait gave up (see last_device_status) */
} rtn_status;

/* Treatment of filter taps that fall outside the image.  The paper never mentions padding; the
 * constant term C of Eq. 10 can be stored ahead of time, as the paper has it, only under
 * RTN_PAD_CODE_ZERO: an outside tap has CODE 0, i.e. real value a_offset, and S_w and K cover
 * all C*kh*kw taps.  RTN_PAD_VALUE_ZERO makes an outside tap contribute nothing (what a
 * floating-point conv2d on the de-quantised tensor does): S_w and K then cover inside taps only. */
typedef enum { RTN_PAD_CODE_ZERO = 0, RTN_PAD_VALUE_ZERO = 1 } rtn_pad_mode;

/* Kernel family.  POPC: Eq. 9 evaluated with AND/XOR/popcount on the packed planes.
 * I8: planes expanded to int8 in shared memory and contracted on the tensor cores
 * (tcgen05 kind::i8).  AUTO picks per shape.  Both give identical integers. */
typedef enum { RTN_VARIANT_AUTO = 0, RTN_VARIANT_POPC = 1, RTN_VARIANT_I8 = 2 } rtn_variant;

/* Bytes of one packed row of K codes: ceil(K/128)*32.  0 if K <= 0. */
size_t rtn_packed_row_bytes(int64_t K);
/* Bytes of a packed operand of `rows` rows. */
size_t rtn_packed_bytes(int64_t rows, int64_t K);
/* Length of a packed convolution filter row: kh*kw*roundup(C,32).  0 on bad arguments. */
int64_t rtn_conv_packed_k(int64_t C, int64_t kh, int64_t kw);
/* Output extent of a convolution: (in + 2*pad - k)/stride + 1 (0 if not positive). */
int64_t rtn_conv_out_dim(int64_t in, int64_t k, int64_t stride, int64_t pad);

/* Weight ternary codes -> packed planes and code sums (Table 1; W1, W2 of Eq. 9; the
 * pre-stored 1 (x) W^t of Eq. 10).  Offline step.
 *   w_codes  int8 [N][C][kh][kw] in {-1,0,+1} (a GEMM weight [N][K] is C=K, kh=kw=1)
 *   w_packed out, N rows of rtn_conv_packed_k(C,kh,kw) codes, 16-byte aligned
 *   w_sum    out, int32 [1 + kh*kw][N]: row 0 = S_w over all taps and channels, row 1+t = sum
 *            over the channels of tap t = i*kw + j (used by RTN_PAD_VALUE_ZERO at borders)
 * Synchronises `stream`.  Returns RTN_ERR_VALUE if any code is outside {-1,0,+1} (outputs are
 * then unspecified). */
rtn_status rtn_pack_weights(const int8_t* w_codes, int64_t N, int64_t C, int64_t kh, int64_t kw,
                            void* w_packed, int32_t* w_sum, void* stream);

/* fp32 activations -> ternary codes (Eq. 3) -> packed planes (Table 1), plus S_x per row.
 *   a        fp32 [M][K] row-major
 *   t_lo,t_hi  n_thr thresholds (n_thr == 1: per layer; n_thr == K: per input feature k).
 *            code = +1 if a > t_hi, else -1 if a < t_lo, else 0; comparisons are strict and
 *            done in fp32, so a value equal to a threshold, and a NaN, code to 0.  With the BN
 *            transform k*a+b of Eq. 2 (k > 0): t_hi = (0.5-b)/k, t_lo = -(0.5+b)/k.
 *   a_packed out, M packed rows of K codes, 16-byte aligned
 *   a_sum    out, int32 [M] = S_x (may be NULL) */
rtn_status rtn_ternarize_pack_act(const float* a, int64_t M, int64_t K,
                                  const float* t_lo, const float* t_hi, int64_t n_thr,
                                  void* a_packed, int32_t* a_sum, void* stream);

/* Packed ternary GEMM with the affine epilogue (Eq. 9 then Eq. 10 with a weight offset):
 *   out[m][n] = a_s*w_s*S_xw + a_s*w_o*S_x[m] + a_o*w_s*S_w[n] + K*a_o*w_o
 *             = sum_k (a_s*x[m][k] + a_o) * (w_s*w[n][k] + w_o)
 *   a_packed M rows, w_packed N rows of K codes (w_packed from rtn_pack_weights with C=K)
 *   a_sum    int32 [M] (S_x), w_sum int32 [N] (row 0 of rtn_pack_weights' w_sum)
 *   a_scale,a_offset  n_aparam floats: 1 (per layer: gamma, beta of Eq. 4) or M (per row)
 *   w_scale,w_offset  n_wparam floats: 1 or N (per output channel: alpha of Eq. 5; the paper
 *                     has w_offset = 0)
 *   out      fp32 [M][N] row-major
 *   dbg_acc  NULL, or int32 [M][N] that receives the raw S_xw */
rtn_status rtn_ternary_gemm(const void* a_packed, const int32_t* a_sum,
                            const void* w_packed, const int32_t* w_sum,
                            int64_t M, int64_t N, int64_t K,
                            const float* a_scale, const float* a_offset, int64_t n_aparam,
                            const float* w_scale, const float* w_offset, int64_t n_wparam,
                            float* out, int32_t* dbg_acc, rtn_variant variant, void* stream);

/* Ternary conv2d as an implicit GEMM (im2col never materialised), input ternarized in-kernel:
 *   x        fp32 [B][C][H][W]; code per Eq. 3 with thresholds per layer (n_thr == 1) or per
 *            input channel (n_thr == C)
 *   w_packed,w_sum  from rtn_pack_weights(w_codes, N, C, kh, kw)
 *   a_scale,a_offset  per-layer gamma, beta (by value); w_scale,w_offset as in the GEMM
 *   out      fp32 [B][N][Ho][Wo], Ho = rtn_conv_out_dim(H,kh,stride,pad), same for Wo
 *   dbg_acc  NULL, or int32 of out's shape that receives the raw S_xw
 * out[b][n][ho][wo] = sum over taps of (a_s*x + a_o)*(w_s*w + w_o) under pad_mode's rule.
 * Stream order: x, out and dbg_acc are ordered after all earlier work of the stream, as usual.  The
 * tensor-core kernels start their set-up while the stream's previous kernel is still draining
 * (programmatic dependent launch), and that set-up reads the layer's parameters: t_lo, t_hi,
 * w_packed, w_sum, w_scale, w_offset must therefore not be buffers that an earlier
 * rtn_ternary_conv2d call of the same stream writes (its out or dbg_acc), unless the stream was
 * synchronized or ran another kernel in between (they are constants of the layer in every intended
 * use). */
rtn_status rtn_ternary_conv2d(const float* x, int64_t B, int64_t C, int64_t H, int64_t W,
                              const float* t_lo, const float* t_hi, int64_t n_thr,
                              const void* w_packed, const int32_t* w_sum,
                              int64_t N, int64_t kh, int64_t kw, int64_t stride, int64_t pad,
                              rtn_pad_mode pad_mode, float a_scale, float a_offset,
                              const float* w_scale, const float* w_offset, int64_t n_wparam,
                              float* out, int32_t* dbg_acc, rtn_variant variant, void* stream);

/* Variant of rtn_ternary_conv2d that allocates nothing (the paper has no counterpart; it is for
 * callers that must not touch an allocator on the hot path).  It always takes the two-kernel
 * tensor-core path (int8 codes of the input in a scratch buffer, filter bank split over CTAs),
 * the path rtn_ternary_conv2d chooses for strided 3x3 layers and, by its cost estimate, for some 1x1
 * stride-2 layers and wide layers at large batch, and gives the same bits.  The scratch is one array of 16 MiB per device, part of the library's image; the
 * call performs no cudaMalloc, cudaMallocAsync, cudaFree or other allocating routine.
 *   - RTN_ERR_UNSUPPORTED: a shape the path does not take (e.g. 3x3 with stride 3), or a layer whose codes
 *     (about B*(H+2pad)*(W+2pad)*(C rounded up to 32) bytes) exceed the array.
 *   - The array is shared by every caller on the device: two calls whose kernels may overlap in
 *     time (different streams, or different host threads on different streams) race on it.
 *     Issue them on one stream, or order them with events.
 *   - The first call on a device does set-up (address of the array, kernel attributes) and must come
 *     before any stream capture; later calls can be captured.
 * Arguments, layouts and the stream-order rule are those of rtn_ternary_conv2d. */
rtn_status rtn_ternary_conv2d_noalloc(const float* x, int64_t B, int64_t C, int64_t H, int64_t W,
                              const float* t_lo, const float* t_hi, int64_t n_thr,
                              const void* w_packed, const int32_t* w_sum,
                              int64_t N, int64_t kh, int64_t kw, int64_t stride, int64_t pad,
                              rtn_pad_mode pad_mode, float a_scale, float a_offset,
                              const float* w_scale, const float* w_offset, int64_t n_wparam,
                              float* out, int32_t* dbg_acc, void* stream);

/* Ternary conv2d that hands its result to the next layer from its epilogue (Eq. 10 with its phi;
 * section "Activation Ternarization": BN sits after the ReLU, so the next layer's BN folds into
 * that layer's threshold pair of Eq. 3).  Per output value:
 *     y    = phi(affine form of rtn_ternary_conv2d) + skip      phi = ReLU if relu == 1, else identity
 *     out        <- y (fp32)                                    if out != NULL
 *     out_packed <- +1 if y > next_t_hi, -1 if y < next_t_lo, else 0, as a packed pixel row
 *                                                               if out_packed != NULL
 * so a layer whose only consumer is the next ternary layer writes 2 bits per value instead of 32.
 *   x ... n_wparam   as in rtn_ternary_conv2d
 *   skip        NULL, or fp32 [B][N][Ho][Wo] (the residual block's skip connection), added after phi
 *   out         NULL, or fp32 [B][N][Ho][Wo]
 *   next_t_lo, next_t_hi   thresholds of the NEXT layer's ternarizer: n_next_thr = 1 (per layer) or N
 *               (per channel of this layer's output); strict fp32 comparisons on the fp32 y, +1 first;
 *               required when out_packed != NULL
 *   out_packed  NULL, or B*Ho*Wo packed rows of N codes each (rtn_packed_bytes(B*Ho*Wo, N) bytes,
 *               16-byte aligned): pixel (b, ho, wo) is row (b*Ho + ho)*Wo + wo, channel n is code n of
 *               the row; canonical zeros, zero fill past N.  This is the x_packed of
 *               rtn_ternary_conv2d_packed.
 *   dbg_acc     NULL, or int32 [B][N][Ho][Wo] raw S_xw
 * At least one of out, out_packed must be given.  Runs on the tensor cores only: the one-kernel variant with
 * the filters resident in shared memory where they fit (stride 1), else the streamed-filter variant or the
 * two-kernel variant with int8 codes in a scratch buffer from the stream-ordered allocator
 * (rtn_conv_next_kernel_launches says how many launches a shape takes); RTN_ERR_UNSUPPORTED for shapes none of
 * the three takes (e.g. 3x3 with stride 3).  Stream-order rule as for rtn_ternary_conv2d; the next-layer
 * thresholds count as parameters of the layer. */
rtn_status rtn_ternary_conv2d_fused(const float* x, int64_t B, int64_t C, int64_t H, int64_t W,
                                    const float* t_lo, const float* t_hi, int64_t n_thr,
                                    const void* w_packed, const int32_t* w_sum,
                                    int64_t N, int64_t kh, int64_t kw, int64_t stride, int64_t pad,
                                    rtn_pad_mode pad_mode, float a_scale, float a_offset,
                                    const float* w_scale, const float* w_offset, int64_t n_wparam,
                                    int relu, const float* skip, float* out,
                                    const float* next_t_lo, const float* next_t_hi, int64_t n_next_thr,
                                    void* out_packed, int32_t* dbg_acc, void* stream);

/* The same layer on an input that is already ternary: packed pixel rows (Table 1 planes; A1, A2 of
 * Eq. 9 with the channel as the fast index), as written by the out_packed of the layer before or by
 * rtn_ternarize_pack_act on an fp32 [B*H*W][C] (NHWC) matrix.
 *   x_packed    B*H*W packed rows of C codes: pixel (b, h, w) is row (b*H + h)*W + w; 16-byte aligned
 * Everything else as in rtn_ternary_conv2d_fused (there are no thresholds for the input: it is codes). */
rtn_status rtn_ternary_conv2d_packed(const void* x_packed, int64_t B, int64_t C, int64_t H, int64_t W,
                                     const void* w_packed, const int32_t* w_sum,
                                     int64_t N, int64_t kh, int64_t kw, int64_t stride, int64_t pad,
                                     rtn_pad_mode pad_mode, float a_scale, float a_offset,
                                     const float* w_scale, const float* w_offset, int64_t n_wparam,
                                     int relu, const float* skip, float* out,
                                     const float* next_t_lo, const float* next_t_hi, int64_t n_next_thr,
                                     void* out_packed, int32_t* dbg_acc, void* stream);

/* The paper's comparison workload (section "Efficient Computation Pattern", Table 1's last column and the
 * DoReFa-Net pattern it cites): 2-bit quaternary values q = 2*b1 + b2 in {0,1,2,3}, dot products by AND
 * between each bit plane of the two inputs, popcount, power-of-two shifts and four partial sums:
 *     x.w = 4 bC(X1&W1) + 2 bC(X1&W2) + 2 bC(X2&W1) + bC(X2&W2).
 * Same packed operand format, with plane 1 = first bit (weight 2) and plane 2 = second bit (weight 1).
 *
 * rtn_pack_quaternary: q_values uint8 [rows][K] in {0..3} -> packed rows (16-byte aligned).  Synchronises
 *   `stream`; RTN_ERR_VALUE if a value is above 3 (output then unspecified).
 * rtn_quaternary_gemm: out[m][n] = sum_k x[m][k] * w[n][k], exact int32 ([M][N] row-major; <= 9 K). */
rtn_status rtn_pack_quaternary(const uint8_t* q_values, int64_t rows, int64_t K, void* packed, void* stream);
rtn_status rtn_quaternary_gemm(const void* a_packed, const void* w_packed, int64_t M, int64_t N, int64_t K,
                               int32_t* out, void* stream);

/* The variant RTN_VARIANT_AUTO resolves to for a shape (never AUTO). */
rtn_variant rtn_choose_gemm_variant(int64_t M, int64_t N, int64_t K);
/* Slices of K that RTN_VARIANT_AUTO cuts a GEMM shape into (1 = none).  A linear layer with few rows and
 * columns and a long K (linear layers are covered by the pattern of section "Efficient Computation
 * Pattern" as much as convolutions) has too few output tiles to fill the GPU: the bit-plane kernel then works on slices of K in
 * parallel, adds their exact integer parts into the output buffer and applies the affine form in place
 * (3 launches instead of 1; the integers do not depend on the order of the additions). */
int64_t rtn_gemm_k_slices(int64_t M, int64_t N, int64_t K);
/* Kernel launches of one rtn_ternary_gemm call with RTN_VARIANT_AUTO: 1; 2 when the tensor-core kernel first
 * expands the weight operand into a scratch buffer (stream-ordered allocation of about N*K bytes; shapes with
 * two or more row tiles; with two or more column tiles as well the activations too, M*K bytes more) or when K
 * is cut into slices (plus a memset). */
int64_t rtn_gemm_kernel_launches(int64_t M, int64_t N, int64_t K);
rtn_variant rtn_choose_conv_variant(int64_t B, int64_t C, int64_t H, int64_t W, int64_t N,
                                    int64_t kh, int64_t kw, int64_t stride, int64_t pad);
/* Kernel launches one rtn_ternary_conv2d call with RTN_VARIANT_AUTO makes for a shape: 1, or 2 on the
 * path that first writes the input's int8 codes to a scratch buffer. */
int64_t rtn_conv_kernel_launches(int64_t B, int64_t C, int64_t H, int64_t W, int64_t N,
                                 int64_t kh, int64_t kw, int64_t stride, int64_t pad);

/* Kernel launches of one rtn_ternary_conv2d_fused / rtn_ternary_conv2d_packed call for a shape: 1 (one-kernel
 * variant with the filters resident in shared memory), 2 (int8 codes in a scratch buffer first), or 0 if
 * the entry points do not take the shape (they would return RTN_ERR_UNSUPPORTED). */
int64_t rtn_conv_next_kernel_launches(int64_t B, int64_t C, int64_t H, int64_t W, int64_t N,
                                      int64_t kh, int64_t kw, int64_t stride, int64_t pad);

/* Synchronises `stream`, then reads and clears the device status word of the current device.
 * RTN_OK, or RTN_ERR_DEVICE_TIMEOUT if a kernel's bounded wait (on an mbarrier of the
 * tensor-core pipeline) ran out since the last call; that kernel's output is then invalid. */
rtn_status rtn_last_device_status(void* stream);

/* Self-test of the bounded waits (the safety net behind RTN_ERR_DEVICE_TIMEOUT): launches one small kernel
 * whose single waiting thread polls, `polls` times (1..4096, each poll parks the thread for up to about 2 us),
 * an mbarrier that nothing arrives on, with the same wait routine the tensor-core kernels use.  The wait must
 * give up: *gave_up (device int32) receives 1, and the next rtn_last_device_status returns
 * RTN_ERR_DEVICE_TIMEOUT once.  Nothing traps or spins without limit; the context stays usable.  Only enqueues. */
rtn_status rtn_selftest_wait_timeout(int64_t polls, int32_t* gave_up, void* stream);

/* Peak probes (measurement aids; the paper has no counterpart).  The contraction kernels are judged against two
 * ceilings that no memory copy measures: the int8 tensor-pipe rate and the issue rate of the AND / XOR /
 * popcount pattern of Eq. 9.  Each probe launches rtn_probe_ctas() CTAs (one per multiprocessor) that run
 * nothing but that work on on-chip operands, and writes the SM-clock cycles of each CTA's loop to `cycles`
 * (device int64 [rtn_probe_ctas()], 8-byte aligned); time the launch with events for the rate in seconds.
 *   rtn_probe_peak_i8   n_mma (1..2^22) tcgen05.mma kind::i8 of M = 128, N = 256, K = 32 per CTA, operands in
 *                       shared memory, one accumulator; rtn_probe_i8_ops_per_mma() = 2*128*256*32 operations each.
 *                       The final wait is bounded like every other (rtn_last_device_status reports a time-out).
 *   rtn_probe_i8_rate   the same loop with accumulators of n_cols columns (a multiple of 16 in 16..256): what one
 *                       instruction of that width costs when nothing else is in the way (narrow instructions do not
 *                       get cheaper in proportion); 2*128*n_cols*32 operations each.
 *   rtn_probe_peak_popc rounds (1..2^24) rounds per thread of 64 word pairs, 1024 threads per CTA, registers
 *                       only; rtn_probe_popc_ops_per_round() operations (2 per code pair) per CTA and round.
 *                       `sink`: device int32 the kernel never writes in practice (keeps the loop alive).
 *   rtn_probe_copy      copies `bytes` (a multiple of 16; both pointers 16-byte aligned) from src to dst with two
 *                       CTAs of 1024 threads per multiprocessor, 16 bytes per thread and trip: the time a kernel
 *                       that only moves a layer's input and output takes at that size.
 * All only enqueue. */
int64_t rtn_probe_ctas(void);
int64_t rtn_probe_i8_ops_per_mma(void);
int64_t rtn_probe_popc_ops_per_round(void);
rtn_status rtn_probe_peak_i8(int64_t n_mma, int64_t* cycles, void* stream);
rtn_status rtn_probe_i8_rate(int64_t n_cols, int64_t n_mma, int64_t* cycles, void* stream);
rtn_status rtn_probe_peak_popc(int64_t rounds, int64_t* cycles, int32_t* sink, void* stream);
rtn_status rtn_probe_copy(const void* src, void* dst, int64_t bytes, void* stream);

/* Static text for a status code. */
const char* rtn_status_string(rtn_status s);

#ifdef __cplusplus
}
#endif
#endif /* RTN_H_ */
