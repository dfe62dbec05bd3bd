"""GPU parity: every entry point of the C ABI against the CPU oracle on the same seeded inputs.
Integer accumulators bit-exact; fp32 outputs within |err| <= 1e-5 |ref| or
|err| <= 1e-6 max(1, sum |term_i|)."""
import numpy as np
import pytest
import torch

import oracle
import paper_1912_02057_b200 as rtn
from paper_1912_02057_b200 import inputs
from helpers import (conv_parity, conv_parity_sampled, conv_through_abi, dev, gemm_parity,
                     gemm_parity_sampled, gemm_through_abi)

pytestmark = pytest.mark.gpu

VARIANTS = [pytest.param(rtn.VARIANT_POPC, id="popc"), pytest.param(rtn.VARIANT_I8, id="i8")]


def run_or_skip_unsupported(fn, variant):
    try:
        return fn()
    except rtn.RtnError as e:
        if e.code == 5 and variant == rtn.VARIANT_I8:
            pytest.skip("shape not supported by the tensor-core variant")
        raise


# ------------------------------------------------------------------------------------ packing
@pytest.mark.parametrize("M,K,per_k", [(1, 1, False), (3, 31, False), (7, 128, True), (9, 129, False),
                                       (64, 576, False), (33, 1000, True), (300, 4097, False),
                                       # rows of a multiple of 8 values take the vector kernel; teams of 1..8 warps
                                       (5, 8, False), (5, 136, True), (21, 1000, False), (19, 2056, True),
                                       (11, 4096, False), (3, 9216, True), (2, 9224, False),
                                       # pixel rows of 32..256 channels: several rows share a warp
                                       (5, 32, False), (7, 64, True), (1001, 64, False), (3, 128, True), (9, 256, False),
                                       (33, 256, True), (1, 32, True)])
def test_ternarize_pack_act(M, K, per_k):
    case = inputs.gemm_case("pack", M, 2, K, seed=M * 1000 + K, p_zero=0.4, thresholds=(0.3, 1.0),
                            per_k_thresholds=per_k)
    a = case.a.copy()
    if a.size >= 4:                                    # ties and specials code to 0 / +-1
        a.flat[0] = case.t_hi.flat[0]
        a.flat[1] = case.t_lo.flat[min(1, case.t_lo.size - 1)] if per_k else case.t_lo.flat[0]
        a.flat[2] = np.nan
        a.flat[3] = np.inf
    packed, s = rtn.rtn_ternarize_pack_act(dev(a), dev(case.t_lo), dev(case.t_hi))
    codes = oracle.ternarize(a, case.t_lo, case.t_hi, channel_axis=1)
    assert np.array_equal(packed.cpu().numpy(), oracle.pack_rows(codes))
    assert np.array_equal(s.cpu().numpy(), codes.astype(np.int64).sum(1))
    # without the sum output
    packed2, none = rtn.rtn_ternarize_pack_act(dev(a), dev(case.t_lo), dev(case.t_hi), want_sum=False)
    assert none is None and torch.equal(packed, packed2)


@pytest.mark.parametrize("shape", [(1, 1), (5, 33), (64, 576), (70, 1000), (4, 3, 3, 3), (64, 64, 3, 3),
                                   (10, 40, 1, 1), (6, 100, 5, 5), (256, 128, 1, 1)])
def test_pack_weights(shape):
    g = inputs.rng(sum(shape))
    w = inputs.weight_codes(g, shape, 0.4)
    packed, sums = rtn.rtn_pack_weights(dev(w))
    w4 = w if w.ndim == 4 else w[:, :, None, None]
    assert np.array_equal(packed.cpu().numpy(), oracle.pack_rows(oracle.conv_weight_rows(w4)))
    assert np.array_equal(sums.cpu().numpy(), oracle.conv_weight_sums(w4))


def test_pack_weights_rejects_a_non_ternary_code():
    w = np.zeros((4, 64), np.int8)
    w[2, 17] = 2
    with pytest.raises(rtn.RtnError) as e:
        rtn.rtn_pack_weights(dev(w))
    assert e.value.code == 4
    w[2, 17] = -1                                       # the flag does not stick
    rtn.rtn_pack_weights(dev(w))


# ------------------------------------------------------------------------------------ GEMM
@pytest.mark.parametrize("variant", VARIANTS)
def test_gemm_config1(variant):
    run_or_skip_unsupported(lambda: gemm_parity(inputs.config1(), variant), variant)


@pytest.mark.parametrize("variant", VARIANTS)
@pytest.mark.parametrize("M,N,K", [(1, 1, 1), (3, 5, 31), (17, 33, 129), (65, 63, 577), (130, 70, 1000),
                                   (128, 128, 128), (129, 257, 384), (300, 200, 2500), (1000, 96, 64)])
def test_gemm_ragged_shapes(M, N, K, variant):
    case = inputs.gemm_case(f"gemm_{M}x{N}x{K}", M, N, K, seed=M + N + K, p_zero=0.35,
                            act="uniform3", thresholds=(-0.5, 0.5), per_row_act_params=(M % 2 == 1),
                            per_k_thresholds=(K % 2 == 1))
    run_or_skip_unsupported(lambda: gemm_parity(case, variant), variant)


@pytest.mark.parametrize("M,N,K", [(1, 1000, 4608), (8, 40, 9000), (64, 64, 16384), (16, 256, 9216), (33, 17, 1025)])
def test_linear_layer_with_few_rows_is_cut_along_k(M, N, K):
    """A batch of a few samples through a wide linear layer: AUTO resolves to the bit-plane kernel with K
    cut into slices (integer parts added atomically into the output buffer, affine form in place); the
    integers and the fp32 outputs meet the same bar as everywhere."""
    assert rtn.rtn_choose_gemm_variant(M, N, K) == rtn.VARIANT_POPC
    assert rtn.rtn_gemm_k_slices(M, N, K) > 1
    case = inputs.gemm_case(f"linear_{M}x{N}x{K}", M, N, K, seed=M + N + K, p_zero=0.35, act="uniform3",
                            thresholds=(-0.5, 0.5), per_row_act_params=(M % 2 == 1))
    gemm_parity(case, rtn.VARIANT_AUTO)
    gemm_parity(case, rtn.VARIANT_AUTO)          # a second call starts from a used output buffer


@pytest.mark.parametrize("variant", VARIANTS)
def test_gemm_degenerate_codes(variant):
    # all-zero codes -> K*a_o*w_o; all +1 against all -1 -> S_xw = -K
    M, N, K = 70, 40, 300
    case = inputs.gemm_case("zeros", M, N, K, seed=1, p_zero=1.0, thresholds=(-1e30, 1e30))
    acc, out = run_or_skip_unsupported(lambda: gemm_through_abi(case, variant), variant)
    assert (acc == 0).all()
    want = K * case.a_offset.astype(np.float64) * case.w_offset.astype(np.float64)[None, :]
    assert np.allclose(out, np.broadcast_to(want, out.shape), rtol=1e-5, atol=1e-6)
    case = inputs.gemm_case("ones", M, N, K, seed=1, p_zero=0.0, thresholds=(-1e30, -1e29))
    case.w_codes[:] = -1
    acc, _ = gemm_through_abi(case, variant)
    assert (acc == -K).all()


@pytest.mark.parametrize("variant", VARIANTS)
def test_gemm_accepts_noncanonical_zero(variant):
    # 01 (plane 1 clear, plane 2 set) is a zero too (Table 1); consumers must mask with plane 1
    case = inputs.gemm_case("nc", 40, 24, 200, seed=3, p_zero=0.5, act="uniform3", thresholds=(-0.5, 0.5))
    M, N, K = case.M, case.N, case.K
    w_packed, w_sum = rtn.rtn_pack_weights(dev(case.w_codes))
    a_packed, a_sum = rtn.rtn_ternarize_pack_act(dev(case.a), dev(case.t_lo), dev(case.t_hi))
    ap = a_packed.cpu().numpy().reshape(M, -1, 2, 16)
    wp = w_packed.cpu().numpy().reshape(N, -1, 2, 16)
    g = np.random.default_rng(0)
    ap[:, :, 1, :] |= (~ap[:, :, 0, :]) & g.integers(0, 256, ap[:, :, 1, :].shape, dtype=np.uint8)
    wp[:, :, 1, :] |= (~wp[:, :, 0, :]) & g.integers(0, 256, wp[:, :, 1, :].shape, dtype=np.uint8)
    # keep the K padding canonical-or-not as well: plane 1 is still 0 there
    acc = torch.empty((M, N), dtype=torch.int32, device="cuda")
    try:
        rtn.rtn_ternary_gemm(dev(ap.reshape(M, -1)), a_sum, dev(wp.reshape(N, -1)), w_sum[0], M, N, K,
                             dev(case.a_scale), dev(case.a_offset), dev(case.w_scale),
                             dev(case.w_offset), dbg_acc=acc, variant=variant)
    except rtn.RtnError as e:
        if e.code == 5:
            pytest.skip("unsupported")
        raise
    codes = oracle.ternarize(case.a, case.t_lo, case.t_hi)
    S, _, _ = oracle.gemm_sums(codes, case.w_codes)
    assert np.array_equal(acc.cpu().numpy().astype(np.int64), S)


@pytest.mark.parametrize("variant", VARIANTS)
def test_gemm_config5_2048(variant):
    run_or_skip_unsupported(lambda: gemm_parity(inputs.config5(2048), variant), variant)


@pytest.mark.parametrize("variant", VARIANTS)
@pytest.mark.parametrize("n,n_rows", [(4096, 384), (8192, 256), (16384, 160)])
def test_gemm_config5_large_sampled(n, n_rows, variant):
    """The sweep's larger sizes (Eq. 9 at M = N = K = n): sampled rows x all columns against the plain oracle."""
    case = inputs.config5(n)
    rows = run_or_skip_unsupported(lambda: gemm_parity_sampled(case, variant, n_rows, seed=n), variant)
    assert rows[0] == 0 and rows[-1] == n - 1 and {127, 128, 255, 256, n - 128, n - 129}.issubset(set(rows.tolist()))


def test_gemm_is_deterministic():
    case = inputs.gemm_case("det", 257, 129, 640, seed=9, p_zero=0.3, act="uniform3", thresholds=(-0.5, 0.5))
    for variant in (rtn.VARIANT_POPC, rtn.VARIANT_I8):
        try:
            a1, o1 = gemm_through_abi(case, variant, check_pack=False)
            a2, o2 = gemm_through_abi(case, variant, check_pack=False)
        except rtn.RtnError as e:
            assert e.code == 5
            continue
        assert np.array_equal(a1, a2) and np.array_equal(o1.view(np.int32), o2.view(np.int32))


# ------------------------------------------------------------------------------------ conv
SMALL_CONVS = [
    # B, C, H, W, N, k, stride, pad
    (2, 5, 9, 8, 4, 3, 1, 1),
    (1, 40, 7, 7, 70, 3, 1, 1),
    (2, 64, 12, 20, 64, 3, 1, 1),
    (2, 64, 13, 11, 32, 3, 2, 1),
    (2, 128, 10, 10, 96, 1, 2, 0),
    (1, 33, 8, 9, 5, 1, 1, 0),
    (1, 6, 11, 11, 8, 5, 1, 2),
    (1, 300, 6, 6, 16, 3, 1, 1),
    (3, 64, 56, 56, 64, 3, 1, 1),
    # 256 filters and many channels: the streamed-filter kernel
    (3, 128, 9, 7, 256, 3, 1, 1),
    (2, 100, 10, 14, 250, 3, 1, 1),
    (2, 64, 8, 8, 256, 5, 1, 2),
    # more than 256 filters: two passes of the streamed-filter kernel over the tile's codes (3x3, 5x5), the
    # two-kernel variant with the filter bank split over CTAs where the filter stream is short (1x1)
    (1, 129, 6, 5, 260, 3, 1, 1),
    (2, 512, 7, 7, 512, 3, 1, 1),
    (5, 256, 14, 14, 400, 3, 1, 1),
    (2, 96, 9, 12, 300, 5, 1, 2),
    (3, 64, 10, 10, 272, 1, 1, 0),
    # strided filters: phase images of the two-kernel variant
    (2, 256, 14, 14, 512, 3, 2, 1),
    (2, 256, 14, 14, 512, 1, 2, 0),
    (1, 16, 11, 11, 8, 5, 2, 2),
    (2, 64, 15, 9, 40, 3, 2, 0),
    # channel counts that are not multiples of 32 with per-layer thresholds that code 0.0 as -1
    (2, 40, 8, 12, 24, 3, 1, 1),
    (2, 100, 8, 8, 256, 1, 1, 0),
]


@pytest.mark.parametrize("variant", VARIANTS)
@pytest.mark.parametrize("pad_mode", [oracle.PAD_CODE_ZERO, oracle.PAD_VALUE_ZERO], ids=["codezero", "valuezero"])
@pytest.mark.parametrize("shape", SMALL_CONVS, ids=lambda s: "x".join(map(str, s)))
def test_conv_small_shapes(shape, pad_mode, variant):
    B, C, H, W, N, k, stride, pad = shape
    case = inputs.conv_case("conv_" + "x".join(map(str, shape)), B, C, H, W, N, k, stride, pad,
                            seed=sum(shape), p_zero=0.4, thresholds=(0.3, 1.0),
                            per_channel_thresholds=(C % 2 == 1))
    run_or_skip_unsupported(lambda: conv_parity(case, variant, pad_mode), variant)


@pytest.mark.parametrize("variant", VARIANTS)
def test_conv_config2_thresholds_around_offset(variant):
    # the thresholds the workload names: +-0.5 around the activation offset; on ReLU input no code
    # is -1 (the degenerate case the paper's BN-after-ReLU remark describes)
    case = inputs.config2(batch=4)
    codes = run_or_skip_unsupported(lambda: conv_parity(case, variant), variant)
    assert (codes >= 0).all() and 0.2 < (codes == 1).mean() < 0.4


@pytest.mark.parametrize("variant", VARIANTS)
def test_conv_config2_full_batch_sampled(variant):
    case = inputs.config2(batch=32, thresholds=(0.3, 1.0))
    acc, out, codes = run_or_skip_unsupported(
        lambda: conv_parity_sampled(case, variant, oracle.PAD_CODE_ZERO, 20000, seed=1), variant)
    assert {-1, 0, 1} == set(np.unique(codes).tolist())
    # a property that holds at any size: with unit scales and zero offsets the output IS the integer
    # accumulator; here instead check |S_xw| <= number of non-zero weights of the filter
    nnz = (case.w_codes != 0).sum((1, 2, 3))
    assert (np.abs(acc) <= nnz[None, :, None, None]).all()


@pytest.mark.parametrize("variant", VARIANTS)
@pytest.mark.parametrize("p_zero", [0.2, 0.5, 0.8])
def test_conv_config3_sampled(p_zero, variant):
    a = inputs.config3a(p_zero, batch=128)
    a.t_lo[:], a.t_hi[:] = 0.3, 1.0
    run_or_skip_unsupported(lambda: conv_parity_sampled(a, variant, oracle.PAD_CODE_ZERO, 5000, seed=2), variant)
    b = inputs.config3b(p_zero, batch=128)
    b.t_lo[:], b.t_hi[:] = 0.3, 1.0
    run_or_skip_unsupported(lambda: conv_parity_sampled(b, variant, oracle.PAD_CODE_ZERO, 5000, seed=3), variant)


@pytest.mark.parametrize("variant", VARIANTS)
def test_conv_thresholds_out_of_order(variant):
    # t_lo > t_hi on some channels: "+1 is tested first" still decides (Eq. 3 lists the +1 case first)
    case = inputs.conv_case("conv_lo_gt_hi", 2, 64, 12, 12, 48, 3, 1, 1, seed=77, p_zero=0.4,
                            thresholds=(0.3, 1.0), per_channel_thresholds=True)
    case.t_lo[::3] = 1.2          # above t_hi (about 1.0) on every third channel
    case.x[0, 0, 0, :4] = case.t_hi[0]      # ties with t_hi on such a channel: not > t_hi, but < t_lo -> -1
    codes = run_or_skip_unsupported(lambda: conv_parity(case, variant), variant)
    assert (codes[:, 0] == 0).sum() == 0    # a channel with t_lo > t_hi has no zero codes


@pytest.mark.parametrize("variant", VARIANTS)
@pytest.mark.parametrize("shape", [(256, 512, 4096), (384, 272, 1152), (130, 520, 260), (515, 300, 1001), (300, 302, 200)], ids=lambda s: "x".join(map(str, s)))
def test_gemm_multi_tile_shapes(shape, variant):
    M, N, K = shape
    case = inputs.gemm_case(f"gemm_{M}x{N}x{K}", M, N, K, seed=M + K, p_zero=0.3, act="uniform3",
                            thresholds=(-0.5, 0.5), per_row_act_params=True)
    run_or_skip_unsupported(lambda: gemm_parity(case, variant), variant)


def test_conv_variants_agree_bit_for_bit():
    case = inputs.config2(batch=2, thresholds=(0.3, 1.0))
    a1, o1, _, _ = conv_through_abi(case, rtn.VARIANT_POPC, oracle.PAD_CODE_ZERO)
    try:
        a2, o2, _, _ = conv_through_abi(case, rtn.VARIANT_I8, oracle.PAD_CODE_ZERO)
    except rtn.RtnError as e:
        assert e.code == 5
        pytest.skip("tensor-core variant does not take this shape")
    assert np.array_equal(a1, a2)


# ------------------------------------------------------------------------------------ bounded waits
def test_a_wait_that_nothing_ends_gives_up_and_is_reported_once():
    """Every device-side wait of the tensor-core kernels is bounded.  A wait on an mbarrier nothing arrives on
    must return (the self-test kernel uses the kernels' own wait routine with a short limit), the status word
    must say RTN_ERR_DEVICE_TIMEOUT exactly once, and the context must stay usable."""
    assert rtn.rtn_last_device_status() == 0
    gave_up = rtn.rtn_selftest_wait_timeout(1024)
    torch.cuda.synchronize()
    assert int(gave_up.item()) == 1
    assert rtn.rtn_last_device_status() == 7          # RTN_ERR_DEVICE_TIMEOUT, read and cleared
    assert rtn.rtn_last_device_status() == 0
    # the device still works: a tensor-core conv right after, checked against the oracle
    case = inputs.config2(batch=2, thresholds=(0.3, 1.0))
    conv_parity(case, rtn.VARIANT_I8)
    assert rtn.rtn_last_device_status() == 0
    with pytest.raises(rtn.RtnError) as e:
        rtn.rtn_selftest_wait_timeout(1 << 20)          # the limit itself is bounded
    assert e.value.code == 2
