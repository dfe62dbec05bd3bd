"""The shared library loads without a GPU and exports every entry point rtn.h declares; argument
errors are reported on the host before anything is launched."""
import ctypes
import os
import re

import paper_1912_02057_b200 as rtn

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def declared_functions():
    text = open(os.path.join(ROOT, "include", "rtn.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(rtn_[a-z0-9_]+)\s*\(", text)))


def test_library_exports_every_declared_symbol():
    names = declared_functions()
    assert {"rtn_pack_weights", "rtn_ternarize_pack_act", "rtn_ternary_gemm",
            "rtn_ternary_conv2d"} <= set(names)
    L = ctypes.CDLL(rtn.lib_path())
    for n in names:
        assert hasattr(L, n), n


def test_size_helpers():
    assert rtn.rtn_packed_row_bytes(1) == 32
    assert rtn.rtn_packed_row_bytes(128) == 32
    assert rtn.rtn_packed_row_bytes(129) == 64
    assert rtn.rtn_packed_row_bytes(576) == 160
    assert rtn.rtn_packed_row_bytes(0) == 0
    assert rtn.rtn_packed_bytes(64, 576) == 64 * 160
    assert rtn.rtn_conv_packed_k(64, 3, 3) == 576
    assert rtn.rtn_conv_packed_k(3, 7, 7) == 49 * 32
    assert rtn.rtn_conv_packed_k(0, 3, 3) == 0
    assert rtn.rtn_conv_out_dim(56, 3, 1, 1) == 56
    assert rtn.rtn_conv_out_dim(56, 3, 2, 1) == 28
    assert rtn.rtn_conv_out_dim(28, 1, 2, 0) == 14
    assert rtn.rtn_conv_out_dim(2, 3, 1, 0) == 0


def test_argument_errors_come_back_as_codes_without_a_gpu():
    L = rtn.lib()
    vp = ctypes.c_void_p
    # NULL pointers
    assert L.rtn_pack_weights(None, 4, 4, 1, 1, None, None, None) == 1
    assert L.rtn_ternarize_pack_act(None, 4, 4, None, None, 1, None, None, None) == 1
    fake = vp(0x1000)          # never dereferenced: the checks below fail before any launch
    odd = vp(0x1004)
    assert L.rtn_pack_weights(fake, 0, 4, 1, 1, fake, fake, None) == 2
    assert L.rtn_pack_weights(fake, 4, 4, 1, 1, odd, fake, None) == 3
    assert L.rtn_ternarize_pack_act(fake, 4, 4, fake, fake, 3, fake, None, None) == 2
    assert L.rtn_ternarize_pack_act(fake, 4, 4, fake, fake, 1, odd, None, None) == 3
    gemm = lambda M, N, K, na, nw, variant, a=fake: L.rtn_ternary_gemm(
        a, fake, fake, fake, M, N, K, fake, fake, na, fake, fake, nw, fake, None, variant, None)
    assert gemm(0, 4, 4, 1, 1, 0) == 2
    assert gemm(4, 4, 1 << 25, 1, 1, 0) == 2
    assert gemm(4, 4, 4, 3, 1, 0) == 2
    assert gemm(4, 4, 4, 1, 5, 0) == 2
    assert gemm(4, 4, 4, 1, 1, 0, a=odd) == 3
    assert gemm(4, 4, 4, 1, 1, 9) == 4
    conv = lambda C, k, stride, pad, mode, nthr=1: L.rtn_ternary_conv2d(
        fake, 1, C, 8, 8, fake, fake, nthr, fake, fake, 4, k, k, stride, pad, mode,
        ctypes.c_float(1.0), ctypes.c_float(0.0), fake, fake, 1, fake, None, 0, None)
    assert conv(0, 3, 1, 1, 0) == 2
    assert conv(4, 3, 0, 1, 0) == 2
    assert conv(4, 11, 1, 0, 0) == 2          # filter larger than the image
    assert conv(4, 3, 1, 1, 0, nthr=3) == 2
    assert conv(4, 3, 1, 1, 7) == 4
    assert rtn.lib().rtn_status_string(2).startswith(b"RTN_ERR_SHAPE")
    assert L.rtn_selftest_wait_timeout(16, None, None) == 1
    assert L.rtn_selftest_wait_timeout(0, fake, None) == 2
    assert L.rtn_selftest_wait_timeout(1 << 20, fake, None) == 2


def test_k_slices_only_for_small_outputs_with_a_long_k():
    assert rtn.rtn_gemm_k_slices(64, 64, 576) == 1            # config 1: one launch
    assert rtn.rtn_gemm_k_slices(4096, 4096, 4096) == 1       # tensor-core kernel
    assert rtn.rtn_gemm_k_slices(16, 256, 9216) > 1
    assert rtn.rtn_gemm_k_slices(64, 4096, 9216) == 1         # enough output tiles without slicing
    assert rtn.rtn_gemm_k_slices(0, 4, 4) == 0


def test_gemm_kernel_launches_follow_the_operand_expansion():
    assert rtn.rtn_gemm_kernel_launches(0, 4, 4) == 0
    assert rtn.rtn_gemm_kernel_launches(64, 64, 576) == 1         # bit-plane kernel, one launch
    assert rtn.rtn_gemm_kernel_launches(16, 256, 9216) == 2       # K in slices: contraction + epilogue in place
    if rtn.rtn_choose_gemm_variant(4096, 4096, 4096) == rtn.VARIANT_I8:
        assert rtn.rtn_gemm_kernel_launches(4096, 4096, 4096) == 2    # operands expanded ahead, then the contraction
        assert rtn.rtn_gemm_kernel_launches(128, 4096, 4096) == 1     # one row tile: everything inside the kernel


def test_probe_argument_errors_without_a_gpu():
    # RTN_ERR_NULL = 1, RTN_ERR_SHAPE = 2, RTN_ERR_ALIGN = 3 (rtn.h)
    L = ctypes.CDLL(rtn.lib_path())
    for f in (L.rtn_probe_peak_i8, L.rtn_probe_i8_rate, L.rtn_probe_peak_popc, L.rtn_probe_copy):
        f.restype = ctypes.c_int
    buf = ctypes.create_string_buffer(64)
    ok = ctypes.cast(buf, ctypes.c_void_p)
    odd = ctypes.c_void_p(ok.value + 4)
    i64, vp = ctypes.c_int64, ctypes.c_void_p
    assert L.rtn_probe_peak_i8(i64(8), vp(None), vp(None)) == 1
    assert L.rtn_probe_peak_i8(i64(0), ok, vp(None)) == 2
    assert L.rtn_probe_i8_rate(i64(64), i64(8), vp(None), vp(None)) == 1
    for bad_cols in (0, 8, 24, 272):
        assert L.rtn_probe_i8_rate(i64(bad_cols), i64(8), ok, vp(None)) == 2
    assert L.rtn_probe_i8_rate(i64(64), i64(8), odd, vp(None)) == 3
    assert L.rtn_probe_peak_popc(i64(8), vp(None), ok, vp(None)) == 1
    assert L.rtn_probe_peak_popc(i64(0), ok, ok, vp(None)) == 2
    assert L.rtn_probe_copy(vp(None), ok, i64(16), vp(None)) == 1
    assert L.rtn_probe_copy(ok, ok, i64(24), vp(None)) == 2
    assert L.rtn_probe_copy(odd, ok, i64(16), vp(None)) == 3
    assert L.rtn_probe_i8_ops_per_mma() == 2 * 128 * 256 * 32
