// Internal declarations shared by the translation units of librtn_b200 (not installed).
#pragma once
#include <cstring>
#include <cuda_runtime.h>
#include <stdint.h>
#include "rtn.h"

namespace rtn {

// Bits of the device status word.
constexpr unsigned kStatusBadWeightCode = 1u;   // rtn_pack_weights met a code outside {-1,0,+1}
constexpr unsigned kStatusWaitTimeout   = 2u;   // a bounded mbarrier wait gave up

// Packed format: 128 codes per 32-byte block (16 B plane 1 "non-zero", 16 B plane 2 "sign").
constexpr int kBlockCodes = 128;
constexpr int kBlockBytes = 32;

inline int64_t blocks_of(int64_t K) { return (K + kBlockCodes - 1) / kBlockCodes; }

// Arguments of the affine epilogue, common to GEMM and conv.
//   out = a_s*w_s*S_xw + a_s*w_o*S_x + a_o*w_s*S_w + K*a_o*w_o      (Eq. 10 plus a weight offset)
struct EpilogueParams {
    const float* a_scale;   // device, n_aparam entries (GEMM) -- or NULL when by value (conv)
    const float* a_offset;
    int64_t n_aparam;
    float a_scale_val;      // used when a_scale == NULL
    float a_offset_val;
    const float* w_scale;   // device, n_wparam entries
    const float* w_offset;
    int64_t n_wparam;
};

struct GemmArgs {
    const uint8_t* a_packed;
    const int32_t* a_sum;
    const uint8_t* w_packed;
    const int32_t* w_sum;
    int64_t M, N, K;
    EpilogueParams ep;
    float* out;
    int32_t* dbg_acc;
    unsigned* status;       // device status word
};

struct ConvArgs {
    const float* x;
    int B, C, H, W;
    const float* t_lo;
    const float* t_hi;
    int n_thr;
    const uint8_t* w_packed;
    const int32_t* w_sum;   // [1 + kh*kw][N]
    int N, kh, kw, stride, pad, Ho, Wo;
    int pad_mode;
    EpilogueParams ep;
    float* out;
    int32_t* dbg_acc;
    unsigned* status;
};

// What a conv layer hands to the next one, fused into its epilogue (every member optional):
//   y = phi(affine form) + skip;  out <- y (fp32);  out_packed <- Eq. 3 codes of y against the
//   NEXT layer's thresholds, as packed pixel rows.  x_packed != NULL: the layer's own input comes as
//   packed pixel rows ([B*H*W] rows of C codes) instead of fp32 (ConvArgs::x, t_lo, t_hi unused).
struct NextLayerArgs {
    const uint8_t* x_packed;
    int relu;               // phi of Eq. 10
    const float* skip;      // fp32 [B][N][Ho][Wo], added after phi
    const float* next_lo;   // thresholds of the next layer's ternarizer: n_next = 1 or N entries
    const float* next_hi;
    int n_next;
    uint8_t* out_packed;    // [B*Ho*Wo] packed rows of N codes
};

// Multiprocessors of the current device, asked once per device.  Plans, *_supported answers, launch counts,
// scratch sizes and the launchers all size their grids with this number, so they agree on any part.  Without a
// usable device (a host-only query) the answer is a B200's 148.
inline int device_sm_count()
{
    constexpr int kSlots = 64;
    static int cached[kSlots];
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) { cudaGetLastError(); return 148; }
    if (dev >= 0 && dev < kSlots && cached[dev] > 0) return cached[dev];
    int sms = 0;
    if (cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || sms <= 0) {
        cudaGetLastError();
        return 148;
    }
    if (dev >= 0 && dev < kSlots) cached[dev] = sms;
    return sms;
}

// Device address of the current device's status word (NULL on failure); defined with the C ABI.
unsigned* device_status_word();

// Launchers (each returns the cudaError_t of its launch).
cudaError_t launch_pack_weights(const int8_t* w, int64_t N, int64_t C, int kh, int kw,
                                uint8_t* packed, int32_t* w_sum, unsigned* status, cudaStream_t s);
cudaError_t launch_ternarize_pack(const float* a, int64_t M, int64_t K, const float* t_lo,
                                  const float* t_hi, int64_t n_thr, uint8_t* packed, int32_t* a_sum,
                                  cudaStream_t s);
cudaError_t launch_gemm_popc(const GemmArgs& g, cudaStream_t s);
int gemm_popc_slices(int64_t M, int64_t N, int64_t K);     // K slices the bit-plane GEMM cuts a shape into (1 = none)
bool conv_popc_supported(const ConvArgs& c);
cudaError_t launch_conv_popc(const ConvArgs& c, cudaStream_t s);

// The paper's 2-bit quaternary comparison workload (AND / popcount / shift pattern).
cudaError_t launch_pack_quaternary(const uint8_t* q, int64_t rows, int64_t K, uint8_t* packed, unsigned* status,
                                   cudaStream_t s);
cudaError_t launch_gemm_quaternary(const uint8_t* a, const uint8_t* w, int64_t M, int64_t N, int64_t K, int32_t* out,
                                   cudaStream_t s);

// Tensor-core (tcgen05 kind::i8) variants; *_supported say whether a shape can run there.
bool gemm_i8_supported(int64_t M, int64_t N, int64_t K);
cudaError_t launch_gemm_i8(const GemmArgs& g, cudaStream_t s);
int gemm_i8_launches(int64_t M, int64_t N, int64_t K);     // 1, or 2 when the weights are expanded into scratch first
bool conv_i8_supported(const ConvArgs& c);       // filters resident in shared memory (stride 1)
cudaError_t launch_conv_i8(const ConvArgs& c, cudaStream_t s);
bool conv_i8s_supported(const ConvArgs& c);      // filters streamed (large layers, 1x1 of any stride)
cudaError_t launch_conv_i8s(const ConvArgs& c, cudaStream_t s);
int conv_i8s_launches(const ConvArgs& c);       // 1, or 2 when the filter bank is expanded into scratch first (0: not taken)
bool conv_i8r_supported(const ConvArgs& c);      // two kernels: int8 codes in a scratch buffer, filter bank split over CTAs
size_t conv_i8r_scratch_bytes(const ConvArgs& c);
cudaError_t launch_conv_i8r(const ConvArgs& c, cudaStream_t s);     // scratch from the stream-ordered allocator
cudaError_t launch_conv_i8r_static(const ConvArgs& c, cudaStream_t s);      // scratch in a static device array
size_t conv_i8r_static_scratch_bytes();
// Two-kernel path with the fused hand-over to the next layer (and, optionally, packed input).
bool conv_i8_next_supported(const ConvArgs& c);    // one-kernel variant (filters resident)
cudaError_t launch_conv_i8_next(const ConvArgs& c, const NextLayerArgs& f, cudaStream_t s);
bool conv_i8s_next_supported(const ConvArgs& c);   // streamed-filter variant
int conv_i8s_next_launches(const ConvArgs& c);
cudaError_t launch_conv_i8s_next(const ConvArgs& c, const NextLayerArgs& f, cudaStream_t s);
bool conv_i8r_next_supported(const ConvArgs& c);
cudaError_t launch_conv_i8r_next(const ConvArgs& c, const NextLayerArgs& f, cudaStream_t s);
inline bool conv_i8_any_supported(const ConvArgs& c)
{
    return conv_i8_supported(c) || conv_i8s_supported(c) || conv_i8r_supported(c);
}
// Rough times (us; negative: shape not taken) behind the choice between the streamed-filter variant, whose
// time is set by the filter stream and hardly moves with the batch, and the split-bank variant, whose time
// grows with the pixels.
double conv_i8s_estimate_us(const ConvArgs& c);
double conv_i8r_estimate_us(const ConvArgs& c);
inline bool conv_prefers_streamed(const ConvArgs& c)
{
    const double ts = conv_i8s_estimate_us(c), tr = conv_i8r_estimate_us(c);
    // a strided 1x1 layer: the streamed-filter kernel gathers only the pixels some tap lands on, in one launch; the
    // split-bank pair reads and codes the whole input first (measured 22.8 against 24.9 us on 128 -> 256 at 28 x 28, batch 128)
    if (ts >= 0.0 && c.kh == 1 && c.kw == 1 && c.stride > 1) return true;
    return ts >= 0.0 && (tr < 0.0 || ts <= 0.95 * tr);     // the estimates are rough: a tie goes to the split bank
}
inline cudaError_t launch_conv_i8_any(const ConvArgs& c, cudaStream_t s)
{
    if (conv_i8_supported(c)) return launch_conv_i8(c, s);
    if (conv_i8s_supported(c) && (!conv_i8r_supported(c) || conv_prefers_streamed(c))) return launch_conv_i8s(c, s);
    return launch_conv_i8r(c, s);
}

// ----------------------------------------------------------------------------------------------
// Device helpers
// ----------------------------------------------------------------------------------------------
#ifdef __CUDACC__

// Eq. 3, strict comparisons in fp32; the +1 case is tested first.  Returns (nz, positive).
__device__ __forceinline__ void ternarize(float v, float lo, float hi, bool& nz, bool& pos)
{
    pos = v > hi;
    nz = pos || (v < lo);
}

// Epilogue in double, rounded once to fp32 (used by the POPC kernels).
__device__ __forceinline__ float epilogue_f64(int s_xw, int s_x, int s_w, double k_eff,
                                              double a_s, double a_o, double w_s, double w_o)
{
    const double r = a_s * w_s * (double)s_xw + a_s * w_o * (double)s_x
                   + a_o * w_s * (double)s_w + k_eff * a_o * w_o;
    return (float)r;
}

// Launch that allows the kernel's CTAs to start while the stream's previous kernel is still
// draining (programmatic dependent launch); the kernel orders itself with tc::pdl_wait().  Inside a
// stream capture the launch becomes a programmatic edge of the graph.
template <typename... KArgs, typename... Args>
inline cudaError_t launch_pdl(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem_bytes, cudaStream_t s,
                              Args&&... args)
{
    cudaLaunchConfig_t cfg;
    memset(&cfg, 0, sizeof(cfg));
    cfg.gridDim = grid;
    cfg.blockDim = block;
    cfg.dynamicSmemBytes = smem_bytes;
    cfg.stream = s;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, kernel, static_cast<KArgs>(args)...);
}

#endif  // __CUDACC__

}  // namespace rtn
