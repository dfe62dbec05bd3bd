// C ABI of librtn_b200 (declared in rtn.h): argument checks, variant choice, launches.
#include "rtn_internal.cuh"
#include "rtn_tcgen05.cuh"

#include <limits.h>

namespace {

// One status word per device, living in device memory for the life of the library.
__device__ unsigned g_status_word;

constexpr int kMaxDevices = 64;
unsigned* g_status_ptr[kMaxDevices];

// Device address of the status word of the current device (NULL on failure).
unsigned* status_word()
{
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return nullptr;
    if (g_status_ptr[dev] == nullptr) {
        void* p = nullptr;
        if (cudaGetSymbolAddress(&p, g_status_word) != cudaSuccess) return nullptr;
        if (cudaMemset(p, 0, sizeof(unsigned)) != cudaSuccess) return nullptr;
        g_status_ptr[dev] = static_cast<unsigned*>(p);
    }
    return g_status_ptr[dev];
}

// Self-test of the give-up path of the bounded waits: one thread waits, with the library's wait routine and a
// caller-chosen number of polls, on an mbarrier that nothing ever arrives on.  The wait must come back false
// and leave the time-out bit in the status word; `result` receives 1 if it did, 0 if the wait claimed success.
__global__ void selftest_wait_kernel(unsigned* status, uint32_t polls, int* result)
{
    __shared__ uint64_t bar;
    if (threadIdx.x == 0) {
        rtn::tc::mbar_init(&bar, 1);
        rtn::tc::mbar_init_fence();
        const bool completed = rtn::tc::mbar_wait(&bar, 0, status, polls);
        *result = completed ? 0 : 1;
    }
}

inline bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }
inline bool aligned4(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 3u) == 0; }

constexpr int64_t kMaxK = int64_t(1) << 24;       // |S| <= K must stay exact in fp32 and int32
constexpr int64_t kMaxDim = int64_t(1) << 31;

rtn_status check_params(const float* s, const float* o, int64_t n, int64_t full)
{
    if (s == nullptr || o == nullptr) return RTN_ERR_NULL;
    if (n != 1 && n != full) return RTN_ERR_SHAPE;
    if (!aligned4(s) || !aligned4(o)) return RTN_ERR_ALIGN;
    return RTN_OK;
}

}  // namespace

namespace rtn {
unsigned* device_status_word() { return status_word(); }
}

extern "C" {

size_t rtn_packed_row_bytes(int64_t K)
{
    if (K <= 0) return 0;
    return (size_t)rtn::blocks_of(K) * rtn::kBlockBytes;
}

size_t rtn_packed_bytes(int64_t rows, int64_t K)
{
    if (rows <= 0 || K <= 0) return 0;
    return (size_t)rows * rtn_packed_row_bytes(K);
}

int64_t rtn_conv_packed_k(int64_t C, int64_t kh, int64_t kw)
{
    if (C <= 0 || kh <= 0 || kw <= 0) return 0;
    return kh * kw * ((C + 31) / 32 * 32);
}

int64_t rtn_conv_out_dim(int64_t in, int64_t k, int64_t stride, int64_t pad)
{
    if (in <= 0 || k <= 0 || stride <= 0 || pad < 0) return 0;
    const int64_t span = in + 2 * pad - k;
    if (span < 0) return 0;
    return span / stride + 1;
}

const char* rtn_status_string(rtn_status s)
{
    switch (s) {
        case RTN_OK: return "RTN_OK";
        case RTN_ERR_NULL: return "RTN_ERR_NULL: a required pointer is NULL";
        case RTN_ERR_SHAPE: return "RTN_ERR_SHAPE: bad or inconsistent size";
        case RTN_ERR_ALIGN: return "RTN_ERR_ALIGN: buffer alignment";
        case RTN_ERR_VALUE: return "RTN_ERR_VALUE: weight code outside {-1,0,+1} or bad enum";
        case RTN_ERR_UNSUPPORTED: return "RTN_ERR_UNSUPPORTED: variant cannot run this shape";
        case RTN_ERR_CUDA: return "RTN_ERR_CUDA: CUDA runtime call failed";
        case RTN_ERR_DEVICE_TIMEOUT: return "RTN_ERR_DEVICE_TIMEOUT: bounded device wait gave up";
    }
    return "unknown rtn_status";
}

rtn_status rtn_pack_weights(const int8_t* w_codes, int64_t N, int64_t C, int64_t kh, int64_t kw,
                            void* w_packed, int32_t* w_sum, void* stream)
{
    if (w_codes == nullptr || w_packed == nullptr || w_sum == nullptr) return RTN_ERR_NULL;
    if (N <= 0 || C <= 0 || kh <= 0 || kw <= 0 || kh > 64 || kw > 64 || N >= kMaxDim) return RTN_ERR_SHAPE;
    if (C > kMaxK || rtn_conv_packed_k(C, kh, kw) > kMaxK) return RTN_ERR_SHAPE;
    if (!aligned16(w_packed) || !aligned4(w_sum)) return RTN_ERR_ALIGN;
    unsigned* st = status_word();
    if (st == nullptr) return RTN_ERR_CUDA;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    if (rtn::launch_pack_weights(w_codes, N, C, (int)kh, (int)kw, static_cast<uint8_t*>(w_packed),
                                 w_sum, st, s) != cudaSuccess) return RTN_ERR_CUDA;
    unsigned h = 0;
    if (cudaMemcpyAsync(&h, st, sizeof(h), cudaMemcpyDeviceToHost, s) != cudaSuccess) return RTN_ERR_CUDA;
    if (cudaStreamSynchronize(s) != cudaSuccess) return RTN_ERR_CUDA;
    if (h & rtn::kStatusBadWeightCode) {
        const unsigned keep = h & ~rtn::kStatusBadWeightCode;
        cudaMemcpyAsync(st, &keep, sizeof(keep), cudaMemcpyHostToDevice, s);
        cudaStreamSynchronize(s);
        return RTN_ERR_VALUE;
    }
    return RTN_OK;
}

rtn_status rtn_ternarize_pack_act(const float* a, int64_t M, int64_t K,
                                  const float* t_lo, const float* t_hi, int64_t n_thr,
                                  void* a_packed, int32_t* a_sum, void* stream)
{
    if (a == nullptr || t_lo == nullptr || t_hi == nullptr || a_packed == nullptr) return RTN_ERR_NULL;
    if (M <= 0 || K <= 0 || M >= kMaxDim || K > kMaxK) return RTN_ERR_SHAPE;
    if (n_thr != 1 && n_thr != K) return RTN_ERR_SHAPE;
    if (!aligned16(a_packed) || !aligned4(a) || !aligned4(t_lo) || !aligned4(t_hi) ||
        (a_sum != nullptr && !aligned4(a_sum))) return RTN_ERR_ALIGN;
    if (rtn::launch_ternarize_pack(a, M, K, t_lo, t_hi, n_thr, static_cast<uint8_t*>(a_packed), a_sum,
                                   static_cast<cudaStream_t>(stream)) != cudaSuccess) return RTN_ERR_CUDA;
    return RTN_OK;
}

rtn_variant rtn_choose_gemm_variant(int64_t M, int64_t N, int64_t K)
{
    if (!rtn::gemm_i8_supported(M, N, K)) return RTN_VARIANT_POPC;
    // Tiny problems finish inside one wave of the bit-plane kernel before the tensor-core
    // pipeline has filled; everything else is far faster on the tensor cores.
    if (M * N <= 128 * 128 && K <= 1024) return RTN_VARIANT_POPC;
    // A linear layer with few rows and columns and a long K is one or two tiles for the tensor-core
    // kernel, whose single CTA then walks all of K; the bit-plane kernel cuts K into slices instead.
    if (M * N <= 64 * 256 && rtn::gemm_popc_slices(M, N, K) > 1) return RTN_VARIANT_POPC;
    return RTN_VARIANT_I8;
}

int64_t rtn_gemm_k_slices(int64_t M, int64_t N, int64_t K)
{
    if (M <= 0 || N <= 0 || K <= 0) return 0;
    return rtn_choose_gemm_variant(M, N, K) == RTN_VARIANT_POPC ? rtn::gemm_popc_slices(M, N, K) : 1;
}

int64_t rtn_gemm_kernel_launches(int64_t M, int64_t N, int64_t K)
{
    if (M <= 0 || N <= 0 || K <= 0) return 0;
    if (rtn_choose_gemm_variant(M, N, K) == RTN_VARIANT_I8) return rtn::gemm_i8_launches(M, N, K);
    return rtn::gemm_popc_slices(M, N, K) > 1 ? 2 : 1;
}

rtn_status rtn_ternary_gemm(const void* a_packed, const int32_t* a_sum,
                            const void* w_packed, const int32_t* w_sum,
                            int64_t M, int64_t N, int64_t K,
                            const float* a_scale, const float* a_offset, int64_t n_aparam,
                            const float* w_scale, const float* w_offset, int64_t n_wparam,
                            float* out, int32_t* dbg_acc, rtn_variant variant, void* stream)
{
    if (a_packed == nullptr || a_sum == nullptr || w_packed == nullptr || w_sum == nullptr ||
        out == nullptr) return RTN_ERR_NULL;
    if (M <= 0 || N <= 0 || K <= 0 || M >= kMaxDim || N >= kMaxDim || K > kMaxK) return RTN_ERR_SHAPE;
    rtn_status st = check_params(a_scale, a_offset, n_aparam, M);
    if (st != RTN_OK) return st;
    st = check_params(w_scale, w_offset, n_wparam, N);
    if (st != RTN_OK) return st;
    if (!aligned16(a_packed) || !aligned16(w_packed) || !aligned4(a_sum) || !aligned4(w_sum) ||
        !aligned4(out) || (dbg_acc != nullptr && !aligned4(dbg_acc))) return RTN_ERR_ALIGN;
    if (variant != RTN_VARIANT_AUTO && variant != RTN_VARIANT_POPC && variant != RTN_VARIANT_I8)
        return RTN_ERR_VALUE;
    if (variant == RTN_VARIANT_AUTO) variant = rtn_choose_gemm_variant(M, N, K);
    if (variant == RTN_VARIANT_I8 && !rtn::gemm_i8_supported(M, N, K)) return RTN_ERR_UNSUPPORTED;
    if (variant == RTN_VARIANT_POPC && ((M + 15) / 16 > INT_MAX || (N + 63) / 64 > 65535))
        return RTN_ERR_UNSUPPORTED;

    rtn::GemmArgs g;
    g.a_packed = static_cast<const uint8_t*>(a_packed);
    g.a_sum = a_sum;
    g.w_packed = static_cast<const uint8_t*>(w_packed);
    g.w_sum = w_sum;
    g.M = M; g.N = N; g.K = K;
    g.ep = rtn::EpilogueParams{a_scale, a_offset, n_aparam, 0.f, 0.f, w_scale, w_offset, n_wparam};
    g.out = out;
    g.dbg_acc = dbg_acc;
    g.status = status_word();
    if (g.status == nullptr) return RTN_ERR_CUDA;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    const cudaError_t e = (variant == RTN_VARIANT_I8) ? rtn::launch_gemm_i8(g, s)
                                                      : rtn::launch_gemm_popc(g, s);
    return e == cudaSuccess ? RTN_OK : RTN_ERR_CUDA;
}

static rtn_status fill_conv_args(rtn::ConvArgs& c, const float* x, int64_t B, int64_t C, int64_t H,
                                 int64_t W, const float* t_lo, const float* t_hi, int64_t n_thr,
                                 const void* w_packed, const int32_t* w_sum, int64_t N, int64_t kh,
                                 int64_t kw, int64_t stride, int64_t pad, rtn_pad_mode pad_mode,
                                 float a_scale, float a_offset, const float* w_scale,
                                 const float* w_offset, int64_t n_wparam, float* out, int32_t* dbg_acc,
                                 bool packed_in = false, bool out_optional = false)
{
    // packed_in: the input is packed pixel rows (x is not used, nor are the thresholds)
    if (w_packed == nullptr || w_sum == nullptr || (out == nullptr && !out_optional)) return RTN_ERR_NULL;
    if (!packed_in && (x == nullptr || t_lo == nullptr || t_hi == nullptr)) return RTN_ERR_NULL;
    const int64_t lim = 1 << 20;
    if (B <= 0 || C <= 0 || H <= 0 || W <= 0 || N <= 0 || kh <= 0 || kw <= 0 || stride <= 0 || pad < 0 ||
        B > lim || C > lim || H > lim || W > lim || N > lim || kh > 64 || kw > 64 || stride > 64 ||
        pad > 64) return RTN_ERR_SHAPE;
    if (!packed_in && n_thr != 1 && n_thr != C) return RTN_ERR_SHAPE;
    const int64_t Ho = rtn_conv_out_dim(H, kh, stride, pad), Wo = rtn_conv_out_dim(W, kw, stride, pad);
    if (Ho <= 0 || Wo <= 0) return RTN_ERR_SHAPE;
    if (rtn_conv_packed_k(C, kh, kw) > kMaxK) return RTN_ERR_SHAPE;
    if (B * C * H * W >= (int64_t(1) << 40) || B * N * Ho * Wo >= (int64_t(1) << 40)) return RTN_ERR_SHAPE;
    if (pad_mode != RTN_PAD_CODE_ZERO && pad_mode != RTN_PAD_VALUE_ZERO) return RTN_ERR_VALUE;
    rtn_status st = check_params(w_scale, w_offset, n_wparam, N);
    if (st != RTN_OK) return st;
    if (!aligned16(w_packed) || !aligned4(out) || !aligned4(w_sum) ||
        (dbg_acc != nullptr && !aligned4(dbg_acc))) return RTN_ERR_ALIGN;
    if (!packed_in && (!aligned4(x) || !aligned4(t_lo) || !aligned4(t_hi))) return RTN_ERR_ALIGN;
    c.x = x; c.B = (int)B; c.C = (int)C; c.H = (int)H; c.W = (int)W;
    c.t_lo = t_lo; c.t_hi = t_hi; c.n_thr = (int)n_thr;
    c.w_packed = static_cast<const uint8_t*>(w_packed); c.w_sum = w_sum;
    c.N = (int)N; c.kh = (int)kh; c.kw = (int)kw; c.stride = (int)stride; c.pad = (int)pad;
    c.Ho = (int)Ho; c.Wo = (int)Wo; c.pad_mode = (int)pad_mode;
    c.ep = rtn::EpilogueParams{nullptr, nullptr, 1, a_scale, a_offset, w_scale, w_offset, n_wparam};
    c.out = out; c.dbg_acc = dbg_acc; c.status = nullptr;
    return RTN_OK;
}

rtn_variant rtn_choose_conv_variant(int64_t B, int64_t C, int64_t H, int64_t W, int64_t N,
                                    int64_t kh, int64_t kw, int64_t stride, int64_t pad)
{
    rtn::ConvArgs c{};
    c.B = (int)B; c.C = (int)C; c.H = (int)H; c.W = (int)W; c.N = (int)N; c.kh = (int)kh; c.kw = (int)kw;
    c.stride = (int)stride; c.pad = (int)pad;
    c.Ho = (int)rtn_conv_out_dim(H, kh, stride, pad); c.Wo = (int)rtn_conv_out_dim(W, kw, stride, pad);
    return rtn::conv_i8_any_supported(c) ? RTN_VARIANT_I8 : RTN_VARIANT_POPC;
}

int64_t rtn_conv_kernel_launches(int64_t B, int64_t C, int64_t H, int64_t W, int64_t N,
                                 int64_t kh, int64_t kw, int64_t stride, int64_t pad)
{
    rtn::ConvArgs c{};
    c.B = (int)B; c.C = (int)C; c.H = (int)H; c.W = (int)W; c.N = (int)N; c.kh = (int)kh; c.kw = (int)kw;
    c.stride = (int)stride; c.pad = (int)pad;
    c.Ho = (int)rtn_conv_out_dim(H, kh, stride, pad); c.Wo = (int)rtn_conv_out_dim(W, kw, stride, pad);
    if (rtn::conv_i8_supported(c)) return 1;
    if (rtn::conv_i8s_supported(c) && (!rtn::conv_i8r_supported(c) || rtn::conv_prefers_streamed(c)))
        return rtn::conv_i8s_launches(c);
    return rtn::conv_i8r_supported(c) ? 2 : 1;
}

int64_t rtn_conv_next_kernel_launches(int64_t B, int64_t C, int64_t H, int64_t W, int64_t N,
                                      int64_t kh, int64_t kw, int64_t stride, int64_t pad)
{
    rtn::ConvArgs c{};
    c.B = (int)B; c.C = (int)C; c.H = (int)H; c.W = (int)W; c.N = (int)N; c.kh = (int)kh; c.kw = (int)kw;
    c.stride = (int)stride; c.pad = (int)pad;
    c.Ho = (int)rtn_conv_out_dim(H, kh, stride, pad); c.Wo = (int)rtn_conv_out_dim(W, kw, stride, pad);
    if (rtn::conv_i8_next_supported(c)) return 1;
    if (rtn::conv_i8s_next_supported(c) && (!rtn::conv_i8r_next_supported(c) || rtn::conv_prefers_streamed(c)))
        return rtn::conv_i8s_next_launches(c);
    return rtn::conv_i8r_next_supported(c) ? 2 : 0;
}

rtn_status rtn_ternary_conv2d(const float* x, int64_t B, int64_t C, int64_t H, int64_t W,
                              const float* t_lo, const float* t_hi, int64_t n_thr,
                              const void* w_packed, const int32_t* w_sum,
                              int64_t N, int64_t kh, int64_t kw, int64_t stride, int64_t pad,
                              rtn_pad_mode pad_mode, float a_scale, float a_offset,
                              const float* w_scale, const float* w_offset, int64_t n_wparam,
                              float* out, int32_t* dbg_acc, rtn_variant variant, void* stream)
{
    rtn::ConvArgs c{};
    rtn_status st = fill_conv_args(c, x, B, C, H, W, t_lo, t_hi, n_thr, w_packed, w_sum, N, kh, kw,
                                   stride, pad, pad_mode, a_scale, a_offset, w_scale, w_offset,
                                   n_wparam, out, dbg_acc);
    if (st != RTN_OK) return st;
    if (variant != RTN_VARIANT_AUTO && variant != RTN_VARIANT_POPC && variant != RTN_VARIANT_I8)
        return RTN_ERR_VALUE;
    if (variant == RTN_VARIANT_AUTO) variant = rtn::conv_i8_any_supported(c) ? RTN_VARIANT_I8 : RTN_VARIANT_POPC;
    if (variant == RTN_VARIANT_I8 && !rtn::conv_i8_any_supported(c)) return RTN_ERR_UNSUPPORTED;
    if (variant == RTN_VARIANT_POPC && !rtn::conv_popc_supported(c)) return RTN_ERR_UNSUPPORTED;
    c.status = status_word();
    if (c.status == nullptr) return RTN_ERR_CUDA;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    const cudaError_t e = (variant == RTN_VARIANT_I8) ? rtn::launch_conv_i8_any(c, s)
                                                      : rtn::launch_conv_popc(c, s);
    return e == cudaSuccess ? RTN_OK : RTN_ERR_CUDA;
}

rtn_status rtn_ternary_conv2d_noalloc(const float* x, int64_t B, int64_t C, int64_t H, int64_t W,
                                      const float* t_lo, const float* t_hi, int64_t n_thr,
                                      const void* w_packed, const int32_t* w_sum,
                                      int64_t N, int64_t kh, int64_t kw, int64_t stride, int64_t pad,
                                      rtn_pad_mode pad_mode, float a_scale, float a_offset,
                                      const float* w_scale, const float* w_offset, int64_t n_wparam,
                                      float* out, int32_t* dbg_acc, void* stream)
{
    rtn::ConvArgs c{};
    rtn_status st = fill_conv_args(c, x, B, C, H, W, t_lo, t_hi, n_thr, w_packed, w_sum, N, kh, kw,
                                   stride, pad, pad_mode, a_scale, a_offset, w_scale, w_offset,
                                   n_wparam, out, dbg_acc);
    if (st != RTN_OK) return st;
    if (!rtn::conv_i8r_supported(c)) return RTN_ERR_UNSUPPORTED;
    if (rtn::conv_i8r_scratch_bytes(c) > rtn::conv_i8r_static_scratch_bytes()) return RTN_ERR_UNSUPPORTED;
    c.status = status_word();
    if (c.status == nullptr) return RTN_ERR_CUDA;
    const cudaError_t e = rtn::launch_conv_i8r_static(c, static_cast<cudaStream_t>(stream));
    return e == cudaSuccess ? RTN_OK : RTN_ERR_CUDA;
}

// Common tail of the two entry points that hand the result to the next layer.
static rtn_status conv_next(rtn::ConvArgs& c, const void* x_packed, int relu, const float* skip,
                            const float* next_t_lo, const float* next_t_hi, int64_t n_next_thr,
                            void* out_packed, void* stream)
{
    if (c.out == nullptr && out_packed == nullptr) return RTN_ERR_NULL;
    if (relu != 0 && relu != 1) return RTN_ERR_VALUE;
    if (out_packed != nullptr) {
        if (next_t_lo == nullptr || next_t_hi == nullptr) return RTN_ERR_NULL;
        if (n_next_thr != 1 && n_next_thr != c.N) return RTN_ERR_SHAPE;
        if (!aligned16(out_packed) || !aligned4(next_t_lo) || !aligned4(next_t_hi)) return RTN_ERR_ALIGN;
    }
    if ((x_packed != nullptr && !aligned16(x_packed)) || (skip != nullptr && !aligned4(skip))) return RTN_ERR_ALIGN;
    const bool one_kernel = rtn::conv_i8_next_supported(c);
    const bool streamed = !one_kernel && rtn::conv_i8s_next_supported(c) &&
                          (!rtn::conv_i8r_next_supported(c) || rtn::conv_prefers_streamed(c));
    if (!one_kernel && !streamed && !rtn::conv_i8r_next_supported(c)) return RTN_ERR_UNSUPPORTED;
    rtn::NextLayerArgs f{};
    f.x_packed = static_cast<const uint8_t*>(x_packed);
    f.relu = relu;
    f.skip = skip;
    f.next_lo = next_t_lo; f.next_hi = next_t_hi; f.n_next = (int)n_next_thr;
    f.out_packed = static_cast<uint8_t*>(out_packed);
    c.status = status_word();
    if (c.status == nullptr) return RTN_ERR_CUDA;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    const cudaError_t e = one_kernel ? rtn::launch_conv_i8_next(c, f, s)
                        : streamed ? rtn::launch_conv_i8s_next(c, f, s) : rtn::launch_conv_i8r_next(c, f, s);
    return e == cudaSuccess ? RTN_OK : RTN_ERR_CUDA;
}

rtn_status rtn_ternary_conv2d_fused(const float* x, int64_t B, int64_t C, int64_t H, int64_t W,
                                    const float* t_lo, const float* t_hi, int64_t n_thr,
                                    const void* w_packed, const int32_t* w_sum,
                                    int64_t N, int64_t kh, int64_t kw, int64_t stride, int64_t pad,
                                    rtn_pad_mode pad_mode, float a_scale, float a_offset,
                                    const float* w_scale, const float* w_offset, int64_t n_wparam,
                                    int relu, const float* skip, float* out,
                                    const float* next_t_lo, const float* next_t_hi, int64_t n_next_thr,
                                    void* out_packed, int32_t* dbg_acc, void* stream)
{
    rtn::ConvArgs c{};
    rtn_status st = fill_conv_args(c, x, B, C, H, W, t_lo, t_hi, n_thr, w_packed, w_sum, N, kh, kw,
                                   stride, pad, pad_mode, a_scale, a_offset, w_scale, w_offset,
                                   n_wparam, out, dbg_acc, false, true);
    if (st != RTN_OK) return st;
    return conv_next(c, nullptr, relu, skip, next_t_lo, next_t_hi, n_next_thr, out_packed, stream);
}

rtn_status rtn_ternary_conv2d_packed(const void* x_packed, int64_t B, int64_t C, int64_t H, int64_t W,
                                     const void* w_packed, const int32_t* w_sum,
                                     int64_t N, int64_t kh, int64_t kw, int64_t stride, int64_t pad,
                                     rtn_pad_mode pad_mode, float a_scale, float a_offset,
                                     const float* w_scale, const float* w_offset, int64_t n_wparam,
                                     int relu, const float* skip, float* out,
                                     const float* next_t_lo, const float* next_t_hi, int64_t n_next_thr,
                                     void* out_packed, int32_t* dbg_acc, void* stream)
{
    if (x_packed == nullptr) return RTN_ERR_NULL;
    rtn::ConvArgs c{};
    rtn_status st = fill_conv_args(c, nullptr, B, C, H, W, nullptr, nullptr, 1, w_packed, w_sum, N, kh, kw,
                                   stride, pad, pad_mode, a_scale, a_offset, w_scale, w_offset,
                                   n_wparam, out, dbg_acc, true, true);
    if (st != RTN_OK) return st;
    return conv_next(c, x_packed, relu, skip, next_t_lo, next_t_hi, n_next_thr, out_packed, stream);
}

rtn_status rtn_pack_quaternary(const uint8_t* q_values, int64_t rows, int64_t K, void* packed, void* stream)
{
    if (q_values == nullptr || packed == nullptr) return RTN_ERR_NULL;
    if (rows <= 0 || K <= 0 || rows >= kMaxDim || K > kMaxK) return RTN_ERR_SHAPE;
    if (!aligned16(packed)) return RTN_ERR_ALIGN;
    unsigned* st = status_word();
    if (st == nullptr) return RTN_ERR_CUDA;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    if (rtn::launch_pack_quaternary(q_values, rows, K, static_cast<uint8_t*>(packed), st, s) != cudaSuccess)
        return RTN_ERR_CUDA;
    unsigned h = 0;
    if (cudaMemcpyAsync(&h, st, sizeof(h), cudaMemcpyDeviceToHost, s) != cudaSuccess) return RTN_ERR_CUDA;
    if (cudaStreamSynchronize(s) != cudaSuccess) return RTN_ERR_CUDA;
    if (h & rtn::kStatusBadWeightCode) {
        const unsigned keep = h & ~rtn::kStatusBadWeightCode;
        cudaMemcpyAsync(st, &keep, sizeof(keep), cudaMemcpyHostToDevice, s);
        cudaStreamSynchronize(s);
        return RTN_ERR_VALUE;
    }
    return RTN_OK;
}

rtn_status rtn_quaternary_gemm(const void* a_packed, const void* w_packed, int64_t M, int64_t N, int64_t K,
                               int32_t* out, void* stream)
{
    if (a_packed == nullptr || w_packed == nullptr || out == nullptr) return RTN_ERR_NULL;
    if (M <= 0 || N <= 0 || K <= 0 || M >= kMaxDim || N >= kMaxDim || K > kMaxK) return RTN_ERR_SHAPE;
    if (!aligned16(a_packed) || !aligned16(w_packed) || !aligned4(out)) return RTN_ERR_ALIGN;
    if ((M + 15) / 16 > INT_MAX || (N + 15) / 16 > 65535) return RTN_ERR_UNSUPPORTED;
    const cudaError_t e = rtn::launch_gemm_quaternary(static_cast<const uint8_t*>(a_packed),
                                                      static_cast<const uint8_t*>(w_packed), M, N, K, out,
                                                      static_cast<cudaStream_t>(stream));
    return e == cudaSuccess ? RTN_OK : RTN_ERR_CUDA;
}

rtn_status rtn_selftest_wait_timeout(int64_t polls, int32_t* gave_up, void* stream)
{
    if (gave_up == nullptr) return RTN_ERR_NULL;
    if (polls < 1 || polls > 4096) return RTN_ERR_SHAPE;
    if (!aligned4(gave_up)) return RTN_ERR_ALIGN;
    unsigned* st = status_word();
    if (st == nullptr) return RTN_ERR_CUDA;
    selftest_wait_kernel<<<1, 32, 0, static_cast<cudaStream_t>(stream)>>>(st, (uint32_t)polls, gave_up);
    return cudaGetLastError() == cudaSuccess ? RTN_OK : RTN_ERR_CUDA;
}

rtn_status rtn_last_device_status(void* stream)
{
    unsigned* st = status_word();
    if (st == nullptr) return RTN_ERR_CUDA;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    unsigned h = 0;
    if (cudaMemcpyAsync(&h, st, sizeof(h), cudaMemcpyDeviceToHost, s) != cudaSuccess) return RTN_ERR_CUDA;
    if (cudaStreamSynchronize(s) != cudaSuccess) return RTN_ERR_CUDA;
    if (h != 0) {
        if (cudaMemsetAsync(st, 0, sizeof(unsigned), s) != cudaSuccess) return RTN_ERR_CUDA;
        if (cudaStreamSynchronize(s) != cudaSuccess) return RTN_ERR_CUDA;
    }
    return (h & rtn::kStatusWaitTimeout) ? RTN_ERR_DEVICE_TIMEOUT : RTN_OK;
}

}  // extern "C"
