"""ctypes binding of ``librtn_b200.so`` (C ABI: ``include/rtn.h``), same names as the C entry points.

Argument marshalling only: torch supplies device memory and the current stream; every step of
the path runs in the library's CUDA kernels.  There is no fallback: if the shared library is
missing, the first call raises.
"""
import ctypes as C
import os

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
_LIB_NAME = "librtn_b200.so"

PAD_CODE_ZERO, PAD_VALUE_ZERO = 0, 1
VARIANT_AUTO, VARIANT_POPC, VARIANT_I8 = 0, 1, 2

_STATUS = {0: "RTN_OK", 1: "RTN_ERR_NULL", 2: "RTN_ERR_SHAPE", 3: "RTN_ERR_ALIGN",
           4: "RTN_ERR_VALUE", 5: "RTN_ERR_UNSUPPORTED", 6: "RTN_ERR_CUDA",
           7: "RTN_ERR_DEVICE_TIMEOUT"}


class RtnError(RuntimeError):
    def __init__(self, code, where):
        self.code = int(code)
        super().__init__(f"{where}: {_STATUS.get(self.code, self.code)}")


def lib_path():
    """The product library; RTN_B200_LIBRARY names another build of it (the instrumented one of
    paper_1912_02057_b200.timeline)."""
    return os.environ.get("RTN_B200_LIBRARY") or os.path.join(_HERE, _LIB_NAME)


_lib = None

_i64, _vp, _f32, _int = C.c_int64, C.c_void_p, C.c_float, C.c_int


def lib():
    """The loaded shared library.  Raises if it has not been built (python -m paper_1912_02057_b200.build)."""
    global _lib
    if _lib is None:
        path = lib_path()
        if not os.path.exists(path):
            raise RuntimeError(
                f"{path} is missing: build it with `python -m paper_1912_02057_b200.build` "
                "(nvcc, sm_100a).  There is no CPU or PyTorch fallback.")
        L = C.CDLL(path)
        L.rtn_packed_row_bytes.restype = C.c_size_t
        L.rtn_packed_row_bytes.argtypes = [_i64]
        L.rtn_packed_bytes.restype = C.c_size_t
        L.rtn_packed_bytes.argtypes = [_i64, _i64]
        L.rtn_conv_packed_k.restype = _i64
        L.rtn_conv_packed_k.argtypes = [_i64, _i64, _i64]
        L.rtn_conv_out_dim.restype = _i64
        L.rtn_conv_out_dim.argtypes = [_i64] * 4
        L.rtn_pack_weights.restype = _int
        L.rtn_pack_weights.argtypes = [_vp, _i64, _i64, _i64, _i64, _vp, _vp, _vp]
        L.rtn_ternarize_pack_act.restype = _int
        L.rtn_ternarize_pack_act.argtypes = [_vp, _i64, _i64, _vp, _vp, _i64, _vp, _vp, _vp]
        L.rtn_ternary_gemm.restype = _int
        L.rtn_ternary_gemm.argtypes = [_vp, _vp, _vp, _vp, _i64, _i64, _i64, _vp, _vp, _i64,
                                       _vp, _vp, _i64, _vp, _vp, _int, _vp]
        L.rtn_ternary_conv2d.restype = _int
        L.rtn_ternary_conv2d.argtypes = [_vp, _i64, _i64, _i64, _i64, _vp, _vp, _i64, _vp, _vp,
                                         _i64, _i64, _i64, _i64, _i64, _int, _f32, _f32,
                                         _vp, _vp, _i64, _vp, _vp, _int, _vp]
        L.rtn_ternary_conv2d_noalloc.restype = _int
        L.rtn_ternary_conv2d_noalloc.argtypes = [_vp, _i64, _i64, _i64, _i64, _vp, _vp, _i64, _vp, _vp,
                                                 _i64, _i64, _i64, _i64, _i64, _int, _f32, _f32,
                                                 _vp, _vp, _i64, _vp, _vp, _vp]
        _tail = [_int, _vp, _vp, _vp, _vp, _i64, _vp, _vp, _vp]      # relu ... stream
        L.rtn_ternary_conv2d_fused.restype = _int
        L.rtn_ternary_conv2d_fused.argtypes = [_vp, _i64, _i64, _i64, _i64, _vp, _vp, _i64, _vp, _vp,
                                               _i64, _i64, _i64, _i64, _i64, _int, _f32, _f32,
                                               _vp, _vp, _i64] + _tail
        L.rtn_ternary_conv2d_packed.restype = _int
        L.rtn_ternary_conv2d_packed.argtypes = [_vp, _i64, _i64, _i64, _i64, _vp, _vp,
                                                _i64, _i64, _i64, _i64, _i64, _int, _f32, _f32,
                                                _vp, _vp, _i64] + _tail
        L.rtn_pack_quaternary.restype = _int
        L.rtn_pack_quaternary.argtypes = [_vp, _i64, _i64, _vp, _vp]
        L.rtn_quaternary_gemm.restype = _int
        L.rtn_quaternary_gemm.argtypes = [_vp, _vp, _i64, _i64, _i64, _vp, _vp]
        L.rtn_choose_gemm_variant.restype = _int
        L.rtn_choose_gemm_variant.argtypes = [_i64] * 3
        L.rtn_gemm_kernel_launches.restype = _i64
        L.rtn_gemm_kernel_launches.argtypes = [_i64] * 3
        L.rtn_gemm_k_slices.restype = _i64
        L.rtn_gemm_k_slices.argtypes = [_i64] * 3
        L.rtn_choose_conv_variant.restype = _int
        L.rtn_choose_conv_variant.argtypes = [_i64] * 9
        L.rtn_conv_kernel_launches.restype = _i64
        L.rtn_conv_kernel_launches.argtypes = [_i64] * 9
        L.rtn_conv_next_kernel_launches.restype = _i64
        L.rtn_conv_next_kernel_launches.argtypes = [_i64] * 9
        L.rtn_last_device_status.restype = _int
        L.rtn_last_device_status.argtypes = [_vp]
        L.rtn_probe_ctas.restype = _i64
        L.rtn_probe_ctas.argtypes = []
        L.rtn_probe_i8_ops_per_mma.restype = _i64
        L.rtn_probe_i8_ops_per_mma.argtypes = []
        L.rtn_probe_popc_ops_per_round.restype = _i64
        L.rtn_probe_popc_ops_per_round.argtypes = []
        L.rtn_probe_peak_i8.restype = _int
        L.rtn_probe_peak_i8.argtypes = [_i64, _vp, _vp]
        L.rtn_probe_i8_rate.restype = _int
        L.rtn_probe_i8_rate.argtypes = [_i64, _i64, _vp, _vp]
        L.rtn_probe_peak_popc.restype = _int
        L.rtn_probe_peak_popc.argtypes = [_i64, _vp, _vp, _vp]
        L.rtn_probe_copy.restype = _int
        L.rtn_probe_copy.argtypes = [_vp, _vp, _i64, _vp]
        L.rtn_selftest_wait_timeout.restype = _int
        L.rtn_selftest_wait_timeout.argtypes = [_i64, _vp, _vp]
        L.rtn_status_string.restype = C.c_char_p
        L.rtn_status_string.argtypes = [_int]
        _lib = L
    return _lib


def _ptr(t, dtype=None, allow_none=False):
    if t is None:
        if allow_none:
            return None
        raise ValueError("tensor required")
    if not t.is_cuda:
        raise ValueError("expected a CUDA tensor")
    if dtype is not None and t.dtype != dtype:
        raise ValueError(f"expected dtype {dtype}, got {t.dtype}")
    if not t.is_contiguous():
        raise ValueError("expected a contiguous tensor")
    return C.c_void_p(t.data_ptr())


def _stream(stream):
    if stream is None:
        stream = torch.cuda.current_stream()
    return C.c_void_p(stream.cuda_stream)


def _check(code, where):
    if code != 0:
        raise RtnError(code, where)


def rtn_packed_row_bytes(K):
    return int(lib().rtn_packed_row_bytes(int(K)))


def rtn_packed_bytes(rows, K):
    return int(lib().rtn_packed_bytes(int(rows), int(K)))


def rtn_conv_packed_k(Cin, kh, kw):
    return int(lib().rtn_conv_packed_k(int(Cin), int(kh), int(kw)))


def rtn_conv_out_dim(n, k, stride, pad):
    return int(lib().rtn_conv_out_dim(int(n), int(k), int(stride), int(pad)))


def rtn_pack_weights(w_codes, stream=None):
    """int8 codes [N,K] or [N,C,kh,kw] on the device -> (w_packed uint8 [N, row_bytes], w_sum int32 [1+kh*kw, N])."""
    if w_codes.dim() == 2:
        N, Cin = w_codes.shape
        kh = kw = 1
    else:
        N, Cin, kh, kw = w_codes.shape
    Kc = rtn_conv_packed_k(Cin, kh, kw)
    w_packed = torch.empty((N, rtn_packed_row_bytes(Kc)), dtype=torch.uint8, device=w_codes.device)
    w_sum = torch.empty((1 + kh * kw, N), dtype=torch.int32, device=w_codes.device)
    _check(lib().rtn_pack_weights(_ptr(w_codes, torch.int8), N, Cin, kh, kw, _ptr(w_packed),
                                  _ptr(w_sum), _stream(stream)), "rtn_pack_weights")
    return w_packed, w_sum


def rtn_ternarize_pack_act(a, t_lo, t_hi, want_sum=True, out=None, out_sum=None, stream=None):
    """fp32 [M,K] -> (a_packed uint8 [M, row_bytes], a_sum int32 [M] or None)."""
    M, K = a.shape
    a_packed = out if out is not None else torch.empty((M, rtn_packed_row_bytes(K)),
                                                       dtype=torch.uint8, device=a.device)
    a_sum = out_sum if out_sum is not None else (
        torch.empty((M,), dtype=torch.int32, device=a.device) if want_sum else None)
    _check(lib().rtn_ternarize_pack_act(_ptr(a, torch.float32), M, K, _ptr(t_lo, torch.float32),
                                        _ptr(t_hi, torch.float32), t_lo.numel(), _ptr(a_packed),
                                        _ptr(a_sum, torch.int32, allow_none=True), _stream(stream)),
           "rtn_ternarize_pack_act")
    return a_packed, a_sum


def rtn_ternary_gemm(a_packed, a_sum, w_packed, w_sum, M, N, K, a_scale, a_offset, w_scale,
                     w_offset, out=None, dbg_acc=None, variant=VARIANT_AUTO, stream=None):
    """Packed ternary GEMM + affine epilogue -> fp32 [M,N].  ``dbg_acc`` (int32 [M,N]) receives raw S_xw."""
    if out is None:
        out = torch.empty((M, N), dtype=torch.float32, device=a_packed.device)
    _check(lib().rtn_ternary_gemm(
        _ptr(a_packed), _ptr(a_sum, torch.int32), _ptr(w_packed), _ptr(w_sum, torch.int32),
        M, N, K, _ptr(a_scale, torch.float32), _ptr(a_offset, torch.float32), a_scale.numel(),
        _ptr(w_scale, torch.float32), _ptr(w_offset, torch.float32), w_scale.numel(),
        _ptr(out, torch.float32), _ptr(dbg_acc, torch.int32, allow_none=True), int(variant),
        _stream(stream)), "rtn_ternary_gemm")
    return out


def rtn_ternary_conv2d(x, t_lo, t_hi, w_packed, w_sum, N, kh, kw, stride, pad, pad_mode,
                       a_scale, a_offset, w_scale, w_offset, out=None, dbg_acc=None,
                       variant=VARIANT_AUTO, stream=None):
    """fp32 NCHW input ternarized in-kernel -> fp32 [B,N,Ho,Wo]."""
    B, Cin, H, W = x.shape
    Ho, Wo = rtn_conv_out_dim(H, kh, stride, pad), rtn_conv_out_dim(W, kw, stride, pad)
    if out is None:
        out = torch.empty((B, N, Ho, Wo), dtype=torch.float32, device=x.device)
    _check(lib().rtn_ternary_conv2d(
        _ptr(x, torch.float32), B, Cin, H, W, _ptr(t_lo, torch.float32), _ptr(t_hi, torch.float32),
        t_lo.numel(), _ptr(w_packed), _ptr(w_sum, torch.int32), N, kh, kw, stride, pad,
        int(pad_mode), float(a_scale), float(a_offset), _ptr(w_scale, torch.float32),
        _ptr(w_offset, torch.float32), w_scale.numel(), _ptr(out, torch.float32),
        _ptr(dbg_acc, torch.int32, allow_none=True), int(variant), _stream(stream)),
        "rtn_ternary_conv2d")
    return out


def rtn_ternary_conv2d_noalloc(x, t_lo, t_hi, w_packed, w_sum, N, kh, kw, stride, pad, pad_mode,
                               a_scale, a_offset, w_scale, w_offset, out, dbg_acc=None, stream=None):
    """rtn_ternary_conv2d on the two-kernel tensor-core path with the library's static scratch array;
    ``out`` is the caller's (nothing is allocated here either)."""
    B, Cin, H, W = x.shape
    _check(lib().rtn_ternary_conv2d_noalloc(
        _ptr(x, torch.float32), B, Cin, H, W, _ptr(t_lo, torch.float32), _ptr(t_hi, torch.float32),
        t_lo.numel(), _ptr(w_packed), _ptr(w_sum, torch.int32), N, kh, kw, stride, pad,
        int(pad_mode), float(a_scale), float(a_offset), _ptr(w_scale, torch.float32),
        _ptr(w_offset, torch.float32), w_scale.numel(), _ptr(out, torch.float32),
        _ptr(dbg_acc, torch.int32, allow_none=True), _stream(stream)),
        "rtn_ternary_conv2d_noalloc")
    return out


def _next_tail(relu, skip, out, next_t_lo, next_t_hi, out_packed, dbg_acc, stream):
    n_next = next_t_lo.numel() if next_t_lo is not None else 1
    return (int(bool(relu)), _ptr(skip, torch.float32, allow_none=True),
            _ptr(out, torch.float32, allow_none=True), _ptr(next_t_lo, torch.float32, allow_none=True),
            _ptr(next_t_hi, torch.float32, allow_none=True), n_next,
            _ptr(out_packed, torch.uint8, allow_none=True), _ptr(dbg_acc, torch.int32, allow_none=True),
            _stream(stream))


def rtn_ternary_conv2d_fused(x, t_lo, t_hi, w_packed, w_sum, N, kh, kw, stride, pad, pad_mode,
                             a_scale, a_offset, w_scale, w_offset, relu=False, skip=None, out=None,
                             next_t_lo=None, next_t_hi=None, out_packed=None, dbg_acc=None, stream=None):
    """fp32 NCHW input; y = phi(conv) + skip goes to ``out`` (fp32 [B,N,Ho,Wo]) and / or, ternarized
    against the next layer's thresholds, to ``out_packed`` (uint8 [B*Ho*Wo, row_bytes(N)]).  The
    caller passes the buffers it wants filled."""
    B, Cin, H, W = x.shape
    _check(lib().rtn_ternary_conv2d_fused(
        _ptr(x, torch.float32), B, Cin, H, W, _ptr(t_lo, torch.float32), _ptr(t_hi, torch.float32),
        t_lo.numel(), _ptr(w_packed), _ptr(w_sum, torch.int32), N, kh, kw, stride, pad,
        int(pad_mode), float(a_scale), float(a_offset), _ptr(w_scale, torch.float32),
        _ptr(w_offset, torch.float32), w_scale.numel(),
        *_next_tail(relu, skip, out, next_t_lo, next_t_hi, out_packed, dbg_acc, stream)),
        "rtn_ternary_conv2d_fused")
    return out, out_packed


def rtn_ternary_conv2d_packed(x_packed, B, Cin, H, W, w_packed, w_sum, N, kh, kw, stride, pad, pad_mode,
                              a_scale, a_offset, w_scale, w_offset, relu=False, skip=None, out=None,
                              next_t_lo=None, next_t_hi=None, out_packed=None, dbg_acc=None, stream=None):
    """The same layer on packed pixel rows (uint8 [B*H*W, row_bytes(Cin)])."""
    _check(lib().rtn_ternary_conv2d_packed(
        _ptr(x_packed, torch.uint8), B, Cin, H, W, _ptr(w_packed), _ptr(w_sum, torch.int32), N, kh, kw,
        stride, pad, int(pad_mode), float(a_scale), float(a_offset), _ptr(w_scale, torch.float32),
        _ptr(w_offset, torch.float32), w_scale.numel(),
        *_next_tail(relu, skip, out, next_t_lo, next_t_hi, out_packed, dbg_acc, stream)),
        "rtn_ternary_conv2d_packed")
    return out, out_packed


def rtn_pack_quaternary(q_values, stream=None):
    """uint8 values [rows,K] in {0..3} on the device -> packed rows uint8 [rows, row_bytes]."""
    rows, K = q_values.shape
    packed = torch.empty((rows, rtn_packed_row_bytes(K)), dtype=torch.uint8, device=q_values.device)
    _check(lib().rtn_pack_quaternary(_ptr(q_values, torch.uint8), rows, K, _ptr(packed), _stream(stream)),
           "rtn_pack_quaternary")
    return packed


def rtn_quaternary_gemm(a_packed, w_packed, M, N, K, out=None, stream=None):
    """Packed 2-bit x 2-bit GEMM (the paper's comparison workload) -> exact int32 [M,N]."""
    if out is None:
        out = torch.empty((M, N), dtype=torch.int32, device=a_packed.device)
    _check(lib().rtn_quaternary_gemm(_ptr(a_packed), _ptr(w_packed), M, N, K, _ptr(out, torch.int32),
                                     _stream(stream)), "rtn_quaternary_gemm")
    return out


def rtn_choose_gemm_variant(M, N, K):
    return int(lib().rtn_choose_gemm_variant(M, N, K))


def rtn_gemm_kernel_launches(M, N, K):
    return int(lib().rtn_gemm_kernel_launches(M, N, K))


def rtn_gemm_k_slices(M, N, K):
    return int(lib().rtn_gemm_k_slices(M, N, K))


def rtn_choose_conv_variant(B, Cin, H, W, N, kh, kw, stride, pad):
    return int(lib().rtn_choose_conv_variant(B, Cin, H, W, N, kh, kw, stride, pad))


def rtn_conv_kernel_launches(B, Cin, H, W, N, kh, kw, stride, pad):
    return int(lib().rtn_conv_kernel_launches(B, Cin, H, W, N, kh, kw, stride, pad))


def rtn_conv_next_kernel_launches(B, Cin, H, W, N, kh, kw, stride, pad):
    return int(lib().rtn_conv_next_kernel_launches(B, Cin, H, W, N, kh, kw, stride, pad))


def rtn_last_device_status(stream=None):
    return int(lib().rtn_last_device_status(_stream(stream)))


def rtn_selftest_wait_timeout(polls=1024, stream=None):
    """Runs the library's bounded wait on an mbarrier nothing arrives on.  Returns the device int32 tensor that
    receives 1 when the wait gave up; the next rtn_last_device_status then reports RTN_ERR_DEVICE_TIMEOUT once."""
    gave_up = torch.zeros((1,), dtype=torch.int32, device="cuda")
    _check(lib().rtn_selftest_wait_timeout(int(polls), _ptr(gave_up, torch.int32), _stream(stream)),
           "rtn_selftest_wait_timeout")
    return gave_up


def rtn_probe_peak_i8(n_mma, stream=None):
    """Launches the int8 tensor-pipe probe; returns (cycles int64 [CTAs] on the device, operations per CTA)."""
    ctas = int(lib().rtn_probe_ctas())
    cycles = torch.zeros((ctas,), dtype=torch.int64, device="cuda")
    _check(lib().rtn_probe_peak_i8(int(n_mma), _ptr(cycles, torch.int64), _stream(stream)), "rtn_probe_peak_i8")
    return cycles, int(n_mma) * int(lib().rtn_probe_i8_ops_per_mma())


def rtn_probe_i8_rate(n_cols, n_mma, stream=None):
    """The tensor-pipe probe with accumulators of n_cols columns; returns (cycles int64 [CTAs] on the device,
    operations per CTA)."""
    ctas = int(lib().rtn_probe_ctas())
    cycles = torch.zeros((ctas,), dtype=torch.int64, device="cuda")
    _check(lib().rtn_probe_i8_rate(int(n_cols), int(n_mma), _ptr(cycles, torch.int64), _stream(stream)), "rtn_probe_i8_rate")
    return cycles, int(n_mma) * 2 * 128 * int(n_cols) * 32


def rtn_probe_peak_popc(rounds, stream=None):
    """Launches the AND / XOR / popcount probe; returns (cycles int64 [CTAs] on the device, operations per CTA)."""
    ctas = int(lib().rtn_probe_ctas())
    cycles = torch.zeros((ctas,), dtype=torch.int64, device="cuda")
    sink = torch.zeros((1,), dtype=torch.int32, device="cuda")
    _check(lib().rtn_probe_peak_popc(int(rounds), _ptr(cycles, torch.int64), _ptr(sink, torch.int32), _stream(stream)),
           "rtn_probe_peak_popc")
    return cycles, int(rounds) * int(lib().rtn_probe_popc_ops_per_round())


def rtn_probe_copy(src, dst, stream=None):
    """Plain device copy of src into dst (same size, a multiple of 16 bytes) by the library's copy probe."""
    nbytes = src.numel() * src.element_size()
    _check(lib().rtn_probe_copy(_ptr(src), _ptr(dst), nbytes, _stream(stream)), "rtn_probe_copy")
    return dst
