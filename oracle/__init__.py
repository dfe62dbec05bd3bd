"""TEST INFRASTRUCTURE -- CPU oracle for the RTN forward ternary contraction.

numpy-facing wrappers around ``rtn_oracle.c`` (plain C, exact int64 sums, double epilogue).
Shares nothing with the CUDA library.  Only the tests, the smoke check and the benchmark's
CPU-baseline leg may import this package; the product never does.

Each wrapper names the passage of the paper (arXiv 1912.02057) its C function follows.
"""
import ctypes as C
import os

import numpy as np

from . import build as _build

_lib = None


def _L():
    global _lib
    if _lib is None:
        _lib = C.CDLL(_build.build())
        _lib.orc_dot_eq9.restype = C.c_int64
        _lib.orc_packed_row_bytes.restype = C.c_int64
        _lib.orc_packed_row_bytes.argtypes = [C.c_int64]
        _lib.orc_conv_out_dim.restype = C.c_int64
        _lib.orc_conv_out_dim.argtypes = [C.c_int64] * 4
        _lib.orc_direct_dot.restype = C.c_double
        _lib.orc_dot_quaternary_bits.restype = C.c_int64
    return _lib


def _p(a):
    return None if a is None else a.ctypes.data_as(C.c_void_p)


def _i64(v):
    return C.c_int64(int(v))


def _arr(a, dtype):
    return np.ascontiguousarray(a, dtype=dtype)


def _param(v, dtype=np.float32):
    return np.atleast_1d(np.ascontiguousarray(v, dtype=dtype))


def threads() -> int:
    """Number of OpenMP threads the oracle's outer loops use."""
    return int(os.environ.get("OMP_NUM_THREADS", os.cpu_count() or 1))


# ----------------------------------------------------------------------------- Eq. 1-3
def ternarize(a, t_lo, t_hi, channel_axis=None):
    """Eq. 3: +1 if A > t_hi, -1 if A < t_lo, else 0 (strict comparisons, fp32 compares).

    ``t_lo``/``t_hi`` are scalars (per layer) or vectors along ``channel_axis``.
    """
    a = _arr(a, np.float32)
    lo, hi = _param(t_lo), _param(t_hi)
    assert lo.shape == hi.shape
    if lo.size == 1:
        outer, chan, inner = 1, 1, a.size
    else:
        ax = channel_axis % a.ndim
        assert a.shape[ax] == lo.size
        outer = int(np.prod(a.shape[:ax], dtype=np.int64))
        chan = a.shape[ax]
        inner = int(np.prod(a.shape[ax + 1:], dtype=np.int64))
    codes = np.empty(a.shape, np.int8)
    _L().orc_ternarize(_p(a), _i64(outer), _i64(chan), _i64(inner), _p(lo), _p(hi),
                       _i64(lo.size), _p(codes))
    return codes


def ternarize_eq1_of_eq2(a, k, b):
    """Eq. 1 applied to Eq. 2's transformed value k*A+b, in double (pins Eq. 3)."""
    a = _arr(a, np.float64)
    codes = np.empty(a.shape, np.int8)
    _L().orc_ternarize_eq1_of_eq2(_p(a), _i64(a.size), C.c_double(k), C.c_double(b), _p(codes))
    return codes


# ----------------------------------------------------------------------------- Table 1, Eq. 9
def encode_bits(codes):
    """Table 1: code -> (first bit = non-zero, second bit = sign); canonical zero 00."""
    codes = _arr(codes, np.int8)
    b1 = np.empty(codes.shape, np.uint8)
    b2 = np.empty(codes.shape, np.uint8)
    _L().orc_encode_bits(_p(codes), _i64(codes.size), _p(b1), _p(b2))
    return b1, b2


def decode_bits(b1, b2):
    """Table 1 read backwards: 00,01 -> 0; 10 -> -1; 11 -> +1."""
    b1, b2 = _arr(b1, np.uint8), _arr(b2, np.uint8)
    codes = np.empty(b1.shape, np.int8)
    _L().orc_decode_bits(_p(b1), _p(b2), _i64(b1.size), _p(codes))
    return codes


def dot_eq9(w1, w2, a1, a2):
    """Eq. 9: bC(c) - 2 bC((W2 xor A2) and c), c = W1 and A1, on one-bit-per-byte vectors."""
    w1, w2, a1, a2 = (_arr(v, np.uint8) for v in (w1, w2, a1, a2))
    return int(_L().orc_dot_eq9(_p(w1), _p(w2), _p(a1), _p(a2), _i64(w1.size)))


# ----------------------------------------------------------------------------- packed format
def packed_row_bytes(K):
    return int(_L().orc_packed_row_bytes(int(K)))


def pack_rows(codes):
    """codes [rows, K] -> bytes [rows, ceil(K/128)*32] in the library's block-plane format."""
    codes = _arr(codes, np.int8)
    rows, K = codes.shape
    out = np.empty((rows, packed_row_bytes(K)), np.uint8)
    _L().orc_pack_rows(_p(codes), _i64(rows), _i64(K), _p(out))
    return out


def unpack_rows(packed, K):
    packed = _arr(packed, np.uint8)
    rows = packed.shape[0]
    assert packed.shape[1] == packed_row_bytes(K)
    codes = np.empty((rows, K), np.int8)
    _L().orc_unpack_rows(_p(packed), _i64(rows), _i64(K), _p(codes))
    return codes


def conv_weight_rows(w):
    """Filters [N, C, kh, kw] -> rows [N, kh*kw*Cw] in (kh, kw, c) order, Cw = C rounded up to 32."""
    w = _arr(w, np.int8)
    N, Cc, kh, kw = w.shape
    Cw = (Cc + 31) // 32 * 32
    rows = np.empty((N, kh * kw * Cw), np.int8)
    _L().orc_conv_weight_rows(_p(w), _i64(N), _i64(Cc), _i64(kh), _i64(kw), _p(rows))
    return rows


def conv_weight_sums(w):
    """Per-tap weight code sums [1 + kh*kw, N]; row 0 is the total (1 (x) W^t of Eq. 10)."""
    w = _arr(w, np.int8)
    N, Cc, kh, kw = w.shape
    sums = np.empty((1 + kh * kw, N), np.int64)
    _L().orc_conv_weight_sums(_p(w), _i64(N), _i64(Cc), _i64(kh), _i64(kw), _p(sums))
    return sums


# ----------------------------------------------------------------------------- GEMM
def gemm_sums(x, w):
    """S_xw [M,N], S_x [M], S_w [N] as exact int64 sums (the definition's triple loop)."""
    x, w = _arr(x, np.int8), _arr(w, np.int8)
    M, K = x.shape
    N, K2 = w.shape
    assert K == K2
    S_xw = np.empty((M, N), np.int64)
    S_x = np.empty(M, np.int64)
    S_w = np.empty(N, np.int64)
    _L().orc_gemm_sums(_p(x), _p(w), _i64(M), _i64(N), _i64(K), _p(S_xw), _p(S_x), _p(S_w))
    return S_xw, S_x, S_w


def epilogue(S_xw, S_x, S_w, K, a_s, a_o, w_s, w_o):
    """Four-term expansion of sum_k (a_s x + a_o)(w_s w + w_o) in double (Eq. 10 when w_o = 0).

    Returns (out, mag) with mag = sum of |term|, the scale of the fp32 tolerance.
    """
    S_xw, S_x, S_w = _arr(S_xw, np.int64), _arr(S_x, np.int64), _arr(S_w, np.int64)
    M, N = S_xw.shape
    a_s, a_o, w_s, w_o = _param(a_s), _param(a_o), _param(w_s), _param(w_o)
    assert a_s.size == a_o.size and a_s.size in (1, M)
    assert w_s.size == w_o.size and w_s.size in (1, N)
    out = np.empty((M, N), np.float64)
    mag = np.empty((M, N), np.float64)
    _L().orc_epilogue(_p(S_xw), _p(S_x), _p(S_w), _i64(M), _i64(N), _i64(K),
                      _p(a_s), _p(a_o), _i64(a_s.size), _p(w_s), _p(w_o), _i64(w_s.size),
                      _p(out), _p(mag))
    return out, mag


def gemm(x, w, a_s, a_o, w_s, w_o):
    """codes x [M,K], w [N,K] -> (S_xw int64, out double, mag double)."""
    S_xw, S_x, S_w = gemm_sums(x, w)
    out, mag = epilogue(S_xw, S_x, S_w, x.shape[1], a_s, a_o, w_s, w_o)
    return S_xw, out, mag


def direct_dot(x, w, a_s, a_o, w_s, w_o):
    """sum_k (a_s x_k + a_o)(w_s w_k + w_o), term by term in double (tiny inputs)."""
    x, w = _arr(x, np.int8), _arr(w, np.int8)
    assert x.shape == w.shape and x.ndim == 1
    return float(_L().orc_direct_dot(_p(x), _p(w), _i64(x.size), C.c_double(a_s), C.c_double(a_o),
                                     C.c_double(w_s), C.c_double(w_o)))


# ----------------------------------------------------------------------------- conv
PAD_CODE_ZERO = 0   # a tap outside the image has code 0 (real value a_o)
PAD_VALUE_ZERO = 1  # a tap outside the image contributes nothing


def conv_out_dim(n, k, stride, pad):
    return int(_L().orc_conv_out_dim(int(n), int(k), int(stride), int(pad)))


def conv2d(x, w, stride, pad, pad_mode, a_s, a_o, w_s, w_o):
    """codes x [B,C,H,W], w [N,C,kh,kw] -> (S_xw int64, out double, mag double), [B,N,Ho,Wo]."""
    x, w = _arr(x, np.int8), _arr(w, np.int8)
    B, Cc, H, W = x.shape
    N, C2, kh, kw = w.shape
    assert Cc == C2
    Ho, Wo = conv_out_dim(H, kh, stride, pad), conv_out_dim(W, kw, stride, pad)
    w_s, w_o = _param(w_s), _param(w_o)
    assert w_s.size == w_o.size and w_s.size in (1, N)
    S = np.empty((B, N, Ho, Wo), np.int64)
    out = np.empty((B, N, Ho, Wo), np.float64)
    mag = np.empty((B, N, Ho, Wo), np.float64)
    _L().orc_conv2d(_p(x), _p(w), _i64(B), _i64(Cc), _i64(H), _i64(W), _i64(N), _i64(kh), _i64(kw),
                    _i64(stride), _i64(pad), C.c_int(pad_mode), C.c_float(a_s), C.c_float(a_o),
                    _p(w_s), _p(w_o), _i64(w_s.size), _p(S), _p(out), _p(mag))
    return S, out, mag


def conv2d_points(x, w, stride, pad, pad_mode, a_s, a_o, w_s, w_o, pts):
    """The same definition at sampled output points pts [n,4] = (b, n, ho, wo)."""
    x, w = _arr(x, np.int8), _arr(w, np.int8)
    B, Cc, H, W = x.shape
    N, C2, kh, kw = w.shape
    assert Cc == C2
    pts = _arr(pts, np.int64)
    n_pts = pts.shape[0]
    w_s, w_o = _param(w_s), _param(w_o)
    S = np.empty(n_pts, np.int64)
    out = np.empty(n_pts, np.float64)
    mag = np.empty(n_pts, np.float64)
    _L().orc_conv2d_points(_p(x), _p(w), _i64(B), _i64(Cc), _i64(H), _i64(W), _i64(N), _i64(kh),
                           _i64(kw), _i64(stride), _i64(pad), C.c_int(pad_mode), C.c_float(a_s),
                           C.c_float(a_o), _p(w_s), _p(w_o), _i64(w_s.size), _p(pts), _i64(n_pts),
                           _p(S), _p(out), _p(mag))
    return S, out, mag


def im2col(x, kh, kw, stride, pad):
    """Materialised patches [B*Ho*Wo, C*kh*kw] with code 0 outside the image (oracle-side only)."""
    x = _arr(x, np.int8)
    B, Cc, H, W = x.shape
    Ho, Wo = conv_out_dim(H, kh, stride, pad), conv_out_dim(W, kw, stride, pad)
    cols = np.empty((B * Ho * Wo, Cc * kh * kw), np.int8)
    _L().orc_im2col(_p(x), _i64(B), _i64(Cc), _i64(H), _i64(W), _i64(kh), _i64(kw), _i64(stride),
                    _i64(pad), _p(cols))
    return cols


# ----------------------------------------------------------------------------- next layer's input
def next_layer(pre, relu, skip, t_lo, t_hi):
    """Eq. 10's phi (ReLU, optional), the block's skip connection (optional), then the next layer's
    ternarizer (Eq. 3 with that layer's BN folded into per-channel thresholds).

    ``pre`` [B,N,...] double (a conv's affine output); ``skip`` fp32 of the same shape or None.
    Returns (y double, codes int8, margin double): y = phi(pre) + skip, codes decided on fp32(y),
    margin = distance of y to the nearer threshold.
    """
    pre = _arr(pre, np.float64)
    B, N = pre.shape[:2]
    inner = int(np.prod(pre.shape[2:], dtype=np.int64))
    lo, hi = _param(t_lo), _param(t_hi)
    assert lo.size == hi.size and lo.size in (1, N)
    sk = None if skip is None else _arr(skip, np.float32)
    assert sk is None or sk.shape == pre.shape
    y = np.empty(pre.shape, np.float64)
    codes = np.empty(pre.shape, np.int8)
    margin = np.empty(pre.shape, np.float64)
    _L().orc_next_layer(_p(pre), _p(sk), C.c_int(1 if relu else 0), _i64(B), _i64(N), _i64(inner),
                        _p(lo), _p(hi), _i64(lo.size), _p(y), _p(codes), _p(margin))
    return y, codes, margin


def pack_nhwc(codes):
    """Activation codes [B,C,H,W] -> packed pixel rows [B*H*W, ceil(C/128)*32]: one row of C codes
    per pixel in the block-plane format (Table 1 planes), pixels in (b, h, w) order."""
    codes = _arr(codes, np.int8)
    B, Cc, H, W = codes.shape
    return pack_rows(np.ascontiguousarray(codes.transpose(0, 2, 3, 1)).reshape(B * H * W, Cc))


def unpack_nhwc(packed, B, Cc, H, W):
    """Inverse of pack_nhwc: packed pixel rows -> codes [B,C,H,W]."""
    rows = unpack_rows(np.asarray(packed, np.uint8).reshape(B * H * W, packed_row_bytes(Cc)), Cc)
    return np.ascontiguousarray(rows.reshape(B, H, W, Cc).transpose(0, 3, 1, 2))


# ----------------------------------------------------------------------------- 2-bit comparison workload
def quaternary_decode(b1, b2):
    """Table 1, last column: bits (b1, b2) -> 2*b1 + b2 in {0,1,2,3}."""
    b1, b2 = _arr(b1, np.uint8), _arr(b2, np.uint8)
    v = np.empty(b1.shape, np.uint8)
    _L().orc_quaternary_decode(_p(b1), _p(b2), _i64(b1.size), _p(v))
    return v


def quaternary_encode(values):
    values = _arr(values, np.uint8)
    b1, b2 = np.empty(values.shape, np.uint8), np.empty(values.shape, np.uint8)
    _L().orc_quaternary_encode(_p(values), _i64(values.size), _p(b1), _p(b2))
    return b1, b2


def quaternary_gemm(x, w):
    """values x [M,K], w [N,K] in {0..3} -> exact int64 dot products [M,N] (the definition)."""
    x, w = _arr(x, np.uint8), _arr(w, np.uint8)
    M, K = x.shape
    N, K2 = w.shape
    assert K == K2
    S = np.empty((M, N), np.int64)
    _L().orc_quaternary_gemm(_p(x), _p(w), _i64(M), _i64(N), _i64(K), _p(S))
    return S


def dot_quaternary_bits(x1, x2, w1, w2):
    """DoReFa pattern: 4 bC(X1&W1) + 2 bC(X1&W2) + 2 bC(X2&W1) + bC(X2&W2) on one-bit-per-byte vectors."""
    x1, x2, w1, w2 = (_arr(v, np.uint8) for v in (x1, x2, w1, w2))
    return int(_L().orc_dot_quaternary_bits(_p(x1), _p(x2), _p(w1), _p(w2), _i64(x1.size)))


def pack_quaternary_rows(values):
    """values [rows, K] in {0..3} -> packed rows: plane 1 = first bit (weight 2), plane 2 = second bit."""
    values = _arr(values, np.uint8)
    rows, K = values.shape
    out = np.empty((rows, packed_row_bytes(K)), np.uint8)
    _L().orc_pack_quaternary_rows(_p(values), _i64(rows), _i64(K), _p(out))
    return out


# ----------------------------------------------------------------------------- tolerance
REL_TOL = 1e-5
ABS_TOL = 1e-6


def within_tolerance(got, ref, mag):
    """Elementwise: |err| <= 1e-5 |ref|  or  |err| <= 1e-6 max(1, sum |term_i|)."""
    err = np.abs(np.asarray(got, np.float64) - ref)
    return (err <= REL_TOL * np.abs(ref)) | (err <= ABS_TOL * np.maximum(1.0, mag))


def strict_miss(got, ref):
    """How far the outputs are from the rule without the sum-of-terms relaxation: (count, largest |err|) over the
    outputs with |err| > 1e-5 |ref| and |err| > 1e-6.  Reported next to the tolerance verdict, never a verdict."""
    ref = np.asarray(ref, np.float64)
    err = np.abs(np.asarray(got, np.float64) - ref)
    miss = (err > REL_TOL * np.abs(ref)) & (err > ABS_TOL)
    return int(miss.sum()), float(err[miss].max()) if miss.any() else 0.0
