"""B200-native forward ternary-by-ternary contraction of the Reparameterized Ternary Network
(arXiv 1912.02057): ternarize + pack, packed ternary GEMM / conv2d, affine epilogue.

The compute lives in the CUDA shared library ``librtn_b200.so`` (C ABI declared in
``include/rtn.h``); :mod:`.binding` marshals torch tensors into it and fails loudly when the
library is missing.  :mod:`.inputs` draws the seeded synthetic workloads.
"""
from .binding import (  # noqa: F401
    RtnError, lib, lib_path,
    rtn_packed_row_bytes, rtn_packed_bytes, rtn_conv_packed_k, rtn_conv_out_dim,
    rtn_pack_weights, rtn_ternarize_pack_act, rtn_ternary_gemm, rtn_ternary_conv2d,
    rtn_pack_quaternary, rtn_quaternary_gemm,
    rtn_ternary_conv2d_noalloc, rtn_ternary_conv2d_fused, rtn_ternary_conv2d_packed,
    rtn_last_device_status, rtn_selftest_wait_timeout, rtn_probe_peak_i8, rtn_probe_i8_rate, rtn_probe_peak_popc, rtn_probe_copy, rtn_choose_gemm_variant, rtn_gemm_k_slices, rtn_gemm_kernel_launches, rtn_choose_conv_variant, rtn_conv_kernel_launches, rtn_conv_next_kernel_launches,
    PAD_CODE_ZERO, PAD_VALUE_ZERO, VARIANT_AUTO, VARIANT_POPC, VARIANT_I8,
)
