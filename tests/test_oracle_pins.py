"""Pins for the CPU oracle: every function is checked against something other than itself --
the paper's printed table, closed forms, brute force in pure Python, or a library routine
(numpy integer matmul, torch fp64 conv2d) on a special case that reduces to it."""
import math

import numpy as np
import pytest
import torch
import torch.nn.functional as F

import oracle
from conftest import read_golden
from paper_1912_02057_b200 import inputs


# ------------------------------------------------------------------ Table 1
def test_table1_decode_matches_paper_rows():
    rows = read_golden("table1_encoding.txt")
    assert len(rows) == 4
    for b1, b2, val in rows:
        got = oracle.decode_bits(np.array([int(b1)], np.uint8), np.array([int(b2)], np.uint8))
        assert int(got[0]) == int(val)


def test_table1_encode_is_canonical_and_round_trips():
    codes = np.array([-1, 0, 1, 0, 1, -1], np.int8)
    b1, b2 = oracle.encode_bits(codes)
    assert b1.tolist() == [1, 0, 1, 0, 1, 1]
    assert b2.tolist() == [0, 0, 1, 0, 1, 0]          # zero is emitted as 00, never 01
    assert oracle.decode_bits(b1, b2).tolist() == codes.tolist()


# ------------------------------------------------------------------ Eq. 9
def test_eq9_exhaustive_on_all_two_bit_pairs():
    val = {(0, 0): 0, (0, 1): 0, (1, 0): -1, (1, 1): 1}     # Table 1
    for w1 in (0, 1):
        for w2 in (0, 1):
            for a1 in (0, 1):
                for a2 in (0, 1):
                    got = oracle.dot_eq9([w1], [w2], [a1], [a2])
                    assert got == val[(w1, w2)] * val[(a1, a2)], (w1, w2, a1, a2)


@pytest.mark.parametrize("n", [1, 2, 7, 31, 32, 33, 127, 128, 129, 200])
def test_eq9_brute_force_with_noncanonical_zeros(n):
    g = np.random.default_rng(100 + n)
    w1, w2, a1, a2 = (g.integers(0, 2, n).astype(np.uint8) for _ in range(4))  # 01 zeros occur
    w, a = oracle.decode_bits(w1, w2), oracle.decode_bits(a1, a2)
    want = sum(int(p) * int(q) for p, q in zip(w.tolist(), a.tolist()))
    assert oracle.dot_eq9(w1, w2, a1, a2) == want


def test_eq9_equals_plain_sum_of_gemm_oracle():
    g = np.random.default_rng(7)
    x = inputs.weight_codes(g, (5, 77), 0.4)
    w = inputs.weight_codes(g, (3, 77), 0.2)
    S, _, _ = oracle.gemm_sums(x, w)
    for m in range(5):
        for n in range(3):
            a1, a2 = oracle.encode_bits(x[m])
            w1, w2 = oracle.encode_bits(w[n])
            assert oracle.dot_eq9(w1, w2, a1, a2) == S[m, n]


# ------------------------------------------------------------------ Eq. 1-3
def test_eq3_equals_eq1_of_eq2_for_positive_k():
    g = np.random.default_rng(11)
    for _ in range(200):
        k = float(g.uniform(0.05, 4.0))
        b = float(g.uniform(-2.0, 2.0))
        a = g.normal(0, 2.0, 257).astype(np.float32)
        t_hi = (0.5 - b) / k
        t_lo = -(0.5 + b) / k
        want = oracle.ternarize_eq1_of_eq2(a.astype(np.float64), k, b)
        got = oracle.ternarize(a, np.float32(t_lo), np.float32(t_hi))
        # the fp32 rounding of the thresholds can move a value sitting within one ulp of one
        near = (np.abs(a - t_hi) < 1e-5 * max(1, abs(t_hi))) | (np.abs(a - t_lo) < 1e-5 * max(1, abs(t_lo)))
        assert np.array_equal(got[~near], want[~near])
        assert (~near).sum() > 200


def test_eq1_plain_thresholds_and_ties():
    a = np.array([0.5, -0.5, 0.50001, -0.50001, 0.0, -0.0, 3.0, -3.0,
                  np.nan, np.inf, -np.inf], np.float32)
    got = oracle.ternarize(a, np.float32(-0.5), np.float32(0.5))
    assert got.tolist() == [0, 0, 1, -1, 0, 0, 1, -1, 0, 1, -1]


def test_eq3_both_thresholds_positive_after_relu():
    # BN after ReLU: both thresholds may be positive, so a ReLU output can still code -1
    a = np.array([0.0, 0.29, 0.3, 0.31, 1.0, 1.01], np.float32)
    got = oracle.ternarize(a, np.float32(0.3), np.float32(1.0))
    assert got.tolist() == [-1, -1, 0, 0, 0, 1]


def test_ternarize_per_channel_thresholds_index_the_channel_axis():
    a = np.zeros((2, 3, 4), np.float32)
    a[:, 0, :] = 0.6
    a[:, 1, :] = 0.6
    a[:, 2, :] = -0.6
    lo = np.array([-0.5, -0.5, -0.7], np.float32)
    hi = np.array([0.5, 0.7, 0.5], np.float32)
    got = oracle.ternarize(a, lo, hi, channel_axis=1)
    assert (got[:, 0, :] == 1).all() and (got[:, 1, :] == 0).all() and (got[:, 2, :] == 0).all()
    # GEMM form: thresholds along the last axis
    b = np.array([[0.6, 0.6, -0.6]], np.float32)
    assert oracle.ternarize(b, lo, hi, channel_axis=1).tolist() == [[1, 0, 0]]


def test_config1_code_fractions_follow_the_normal_cdf():
    case = inputs.config1()
    codes = oracle.ternarize(case.a, case.t_lo, case.t_hi)
    n = codes.size
    phi = lambda z: 0.5 * (1 + math.erf(z / math.sqrt(2)))
    for code, p in ((-1, phi(0.3)), (1, 1 - phi(1.0)), (0, phi(1.0) - phi(0.3))):
        frac = float((codes == code).mean())
        assert abs(frac - p) < 4 * math.sqrt(p * (1 - p) / n), (code, frac, p)


# ------------------------------------------------------------------ S_xw, S_x, S_w
def test_gemm_sums_hand_cases():
    x = np.array([[1, 1, 1, 1]], np.int8)
    S, Sx, Sw = oracle.gemm_sums(x, x)
    assert S.tolist() == [[4]] and Sx.tolist() == [4] and Sw.tolist() == [4]
    x = np.array([[1, -1, 0, 1, 0]], np.int8)
    S, Sx, Sw = oracle.gemm_sums(x, -x)
    assert S.tolist() == [[-3]] and Sx.tolist() == [1] and Sw.tolist() == [-1]
    x = np.array([[1, 0], [0, -1]], np.int8)
    w = np.array([[1, 1], [-1, 1], [0, 0]], np.int8)
    S, Sx, Sw = oracle.gemm_sums(x, w)
    assert S.tolist() == [[1, -1, 0], [-1, -1, 0]]      # [m][n]: not transposed
    assert Sx.tolist() == [1, -1] and Sw.tolist() == [2, 0, 0]


def test_gemm_sums_against_numpy_integer_matmul():
    g = np.random.default_rng(3)
    x = inputs.weight_codes(g, (37, 301), 0.3)
    w = inputs.weight_codes(g, (19, 301), 0.5)
    S, Sx, Sw = oracle.gemm_sums(x, w)
    assert np.array_equal(S, x.astype(np.int64) @ w.astype(np.int64).T)
    assert np.array_equal(Sx, x.astype(np.int64).sum(1))
    assert np.array_equal(Sw, w.astype(np.int64).sum(1))


# ------------------------------------------------------------------ epilogue
def _py_direct(x, w, a_s, a_o, w_s, w_o):
    return math.fsum((a_s * int(p) + a_o) * (w_s * int(q) + w_o) for p, q in zip(x, w))


def test_epilogue_equals_direct_evaluation_on_tiny_inputs():
    g = np.random.default_rng(5)
    for K in (1, 2, 3, 9, 40):
        x = inputs.weight_codes(g, (4, K), 0.3)
        w = inputs.weight_codes(g, (3, K), 0.3)
        a_s, a_o = inputs.uniform(g, 0.5, 1.5, (4,)), inputs.uniform(g, -0.5, 0.5, (4,))
        w_s, w_o = inputs.uniform(g, 0.5, 1.5, (3,)), inputs.uniform(g, -0.5, 0.5, (3,))
        _, out, mag = oracle.gemm(x, w, a_s, a_o, w_s, w_o)
        for m in range(4):
            for n in range(3):
                args = (float(a_s[m]), float(a_o[m]), float(w_s[n]), float(w_o[n]))
                want = _py_direct(x[m].tolist(), w[n].tolist(), *args)
                assert abs(out[m, n] - want) <= 1e-12 * max(1.0, mag[m, n])
                assert abs(oracle.direct_dot(x[m], w[n], *args) - want) <= 1e-12 * max(1.0, mag[m, n])


def test_epilogue_all_zero_codes_closed_form():
    K = 37
    x = np.zeros((2, K), np.int8)
    w = np.zeros((3, K), np.int8)
    w_o = np.array([0.25, -0.5, 0.125], np.float32)
    _, out, _ = oracle.gemm(x, w, 1.5, 0.75, np.array([2.0, 3.0, 4.0], np.float32), w_o)
    assert np.array_equal(out, np.broadcast_to(K * 0.75 * w_o.astype(np.float64), (2, 3)))


def test_epilogue_reduces_to_eq10_and_eq11():
    g = np.random.default_rng(9)
    K = 64
    x = inputs.weight_codes(g, (6, K), 0.3)
    w = inputs.weight_codes(g, (5, K), 0.4)
    gamma, beta = 1.3083, 0.5152                       # layer2.0.conv1 in the appendix table
    alpha = inputs.uniform(g, 0.5, 3.0, (5,))
    S, Sx, Sw = oracle.gemm_sums(x, w)
    _, out, _ = oracle.gemm(x, w, gamma, beta, alpha, np.zeros(5, np.float32))
    g32, b32 = float(np.float32(gamma)), float(np.float32(beta))
    eq10 = alpha.astype(np.float64) * g32 * S + alpha.astype(np.float64) * b32 * Sw[None, :]
    assert np.allclose(out, eq10, rtol=1e-14, atol=1e-12)
    # Eq. 11: relu(alpha*gamma*S + C) == alpha * max(0, gamma*S + T), T = beta*S_w, for alpha > 0
    T = b32 * Sw[None, :]
    eq11 = alpha.astype(np.float64) * np.maximum(0.0, g32 * S + T)
    assert np.allclose(np.maximum(out, 0.0), eq11, rtol=1e-14, atol=1e-12)


def test_epilogue_unit_scale_zero_offset_is_the_integer_dot():
    g = np.random.default_rng(10)
    x = inputs.weight_codes(g, (4, 50), 0.3)
    w = inputs.weight_codes(g, (4, 50), 0.3)
    S, out, _ = oracle.gemm(x, w, 1.0, 0.0, 1.0, 0.0)
    assert np.array_equal(out, S.astype(np.float64))


def test_epilogue_each_term_has_its_own_factor():
    # one term at a time: a mistake that swaps S_x and S_w, or drops K, shows here
    x = np.array([[1, 1, 0]], np.int8)      # S_x = 2
    w = np.array([[-1, 0, 0]], np.int8)     # S_w = -1, S_xw = -1
    K = 3
    assert oracle.gemm(x, w, 2.0, 0.0, 3.0, 0.0)[1][0, 0] == 2 * 3 * -1
    assert oracle.gemm(x, w, 2.0, 0.0, 0.0, 5.0)[1][0, 0] == 2 * 5 * 2
    assert oracle.gemm(x, w, 0.0, 7.0, 3.0, 0.0)[1][0, 0] == 7 * 3 * -1
    assert oracle.gemm(x, w, 0.0, 7.0, 0.0, 5.0)[1][0, 0] == K * 7 * 5


def test_epilogue_mag_is_the_sum_of_absolute_terms():
    # mag scales every fp32 tolerance: pin it to a hand-written sum of |term_i| (dyadic values, exact)
    x = np.array([[1, 1, 0]], np.int8)      # S_x = 2
    w = np.array([[-1, 0, 0]], np.int8)     # S_w = -1, S_xw = -1
    K = 3
    a_s, a_o, w_s, w_o = 2.0, -0.5, 3.0, 0.25
    _, out, mag = oracle.gemm(x, w, a_s, a_o, w_s, w_o)
    terms = [a_s * w_s * -1, a_s * w_o * 2, a_o * w_s * -1, K * a_o * w_o]      # -6, 1, 1.5, -0.375
    assert out[0, 0] == sum(terms) == -3.875
    assert mag[0, 0] == sum(abs(t) for t in terms) == 8.875
    # one term at a time: each |term| arrives in mag with its own factor
    assert oracle.gemm(x, w, 2.0, 0.0, 3.0, 0.0)[2][0, 0] == 6.0
    assert oracle.gemm(x, w, 2.0, 0.0, 0.0, 5.0)[2][0, 0] == 20.0
    assert oracle.gemm(x, w, 0.0, 7.0, 3.0, 0.0)[2][0, 0] == 21.0
    assert oracle.gemm(x, w, 0.0, 7.0, 0.0, 5.0)[2][0, 0] == 105.0
    # random small cases against a pure-Python sum, per-row and per-column parameters
    g = np.random.default_rng(12)
    x = inputs.weight_codes(g, (4, 23), 0.3)
    w = inputs.weight_codes(g, (3, 23), 0.3)
    a_s, a_o = inputs.uniform(g, 0.5, 1.5, (4,)), inputs.uniform(g, -0.5, 0.5, (4,))
    w_s, w_o = inputs.uniform(g, 0.5, 1.5, (3,)), inputs.uniform(g, -0.5, 0.5, (3,))
    _, _, mag = oracle.gemm(x, w, a_s, a_o, w_s, w_o)
    for m in range(4):
        for n in range(3):
            sxw = sum(int(p) * int(q) for p, q in zip(x[m], w[n]))
            sx, sw = int(x[m].sum()), int(w[n].sum())
            As, Ao, Ws, Wo = float(a_s[m]), float(a_o[m]), float(w_s[n]), float(w_o[n])
            want = abs(As * Ws * sxw) + abs(As * Wo * sx) + abs(Ao * Ws * sw) + abs(23 * Ao * Wo)
            assert abs(mag[m, n] - want) <= 1e-13 * want
            assert mag[m, n] >= abs(oracle.gemm(x, w, a_s, a_o, w_s, w_o)[1][m, n])


def test_conv_mag_both_pad_modes_hand_case():
    # 1 channel, 2x2 image of all +1, one 3x3 filter of all -1, pad 1: the output at (0, 0) sees 4 inside taps
    x = np.ones((1, 1, 2, 2), np.int8)
    w = -np.ones((1, 1, 3, 3), np.int8)
    a_s, a_o, w_s, w_o = 2.0, 0.5, 4.0, 0.25
    # code-zero padding: S_xw = -4, S_x = 4, S_w = -9, K = 9
    terms0 = [a_s * w_s * -4, a_s * w_o * 4, a_o * w_s * -9, 9 * a_o * w_o]     # -32, 2, -18, 1.125
    S, out, mag = oracle.conv2d(x, w, 1, 1, oracle.PAD_CODE_ZERO, a_s, a_o, np.float32(w_s), np.float32(w_o))
    assert S[0, 0, 0, 0] == -4 and out[0, 0, 0, 0] == sum(terms0) and mag[0, 0, 0, 0] == 53.125
    # value-zero padding: S_w and K over the 4 inside taps only
    terms1 = [a_s * w_s * -4, a_s * w_o * 4, a_o * w_s * -4, 4 * a_o * w_o]     # -32, 2, -8, 0.5
    S, out, mag = oracle.conv2d(x, w, 1, 1, oracle.PAD_VALUE_ZERO, a_s, a_o, np.float32(w_s), np.float32(w_o))
    assert S[0, 0, 0, 0] == -4 and out[0, 0, 0, 0] == sum(terms1) and mag[0, 0, 0, 0] == 42.5
    pts = np.array([[0, 0, 0, 0], [0, 0, 1, 1]], np.int64)
    _, op, mp = oracle.conv2d_points(x, w, 1, 1, oracle.PAD_VALUE_ZERO, a_s, a_o, np.float32(w_s), np.float32(w_o), pts)
    assert list(op) == [sum(terms1)] * 2 and list(mp) == [42.5, 42.5]


def test_within_tolerance_branches_on_hand_made_triples():
    T = oracle.within_tolerance
    one = lambda got, ref, mag: bool(T(np.array([got]), np.array([ref]), np.array([mag]))[0])
    # relative branch alone decides (mag tiny): 1e-5 |ref| with |ref| = 1000 -> 0.01
    assert one(1000.0 + 0.0099, 1000.0, 0.0)
    assert not one(1000.0 + 0.0101, 1000.0, 0.0)
    assert one(-1000.0 - 0.0099, -1000.0, 0.0)
    assert not one(-1000.0 + 0.0101, -1000.0, 0.0)
    # absolute branch with mag < 1: the floor max(1, mag) = 1 -> 1e-6
    assert one(0.9e-6, 0.0, 0.25)
    assert not one(1.1e-6, 0.0, 0.25)
    assert one(-0.9e-6, 0.0, 0.0)
    # absolute branch scaled by mag > 1 (terms cancel: ref near 0, mag = 400 -> 4e-4)
    assert one(0.01 + 3.9e-4, 0.01, 400.0)
    assert not one(0.01 + 4.1e-4, 0.01, 400.0)
    # the two branches are alternatives (or), not both required (and)
    assert one(1000.0 + 0.009, 1000.0, 1.0)         # relative holds, absolute (1e-6) does not
    assert one(1e-3 + 3e-4, 1e-3, 400.0)            # absolute holds, relative (1e-8) does not
    # a mag a thousand times too large would accept this one
    assert not one(0.5, 0.0, 400.0)
    # shapes broadcast elementwise
    got = np.array([[0.0, 2e-6], [1.0, 1.0 + 2e-5]])
    ref = np.array([[0.0, 0.0], [1.0, 1.0]])
    assert T(got, ref, np.ones((2, 2))).tolist() == [[True, False], [True, False]]
    assert (oracle.REL_TOL, oracle.ABS_TOL) == (1e-5, 1e-6)


def test_strict_miss_counts_the_outputs_outside_the_unrelaxed_rule():
    # the unrelaxed rule: |err| <= 1e-5 |ref| or |err| <= 1e-6
    got = np.array([0.0, 2e-6, 1.0 + 2e-5, 1000.0 + 0.009])
    ref = np.array([0.0, 0.0, 1.0, 1000.0])
    n, worst = oracle.strict_miss(got, ref)
    assert n == 2 and abs(worst - 2e-5) < 1e-9


# ------------------------------------------------------------------ convolution
def _deq(codes, s, o):
    return s * torch.from_numpy(codes.astype(np.float64)) + o


@pytest.mark.parametrize("k,stride,pad", [(3, 1, 1), (3, 2, 1), (1, 2, 0), (1, 1, 0), (3, 1, 0), (5, 1, 2)])
def test_conv2d_against_torch_fp64_on_dequantized_values(k, stride, pad):
    g = np.random.default_rng(20 + k + stride)
    B, C, H, W, N = 2, 5, 9, 8, 4
    x = inputs.weight_codes(g, (B, C, H, W), 0.3)
    w = inputs.weight_codes(g, (N, C, k, k), 0.4)
    a_s, a_o = 1.25, -0.375
    w_s, w_o = inputs.uniform(g, 0.5, 1.5, (N,)), inputs.uniform(g, -0.5, 0.5, (N,))
    xd = _deq(x, a_s, a_o)
    wd = torch.from_numpy(w_s.astype(np.float64))[:, None, None, None] * torch.from_numpy(
        w.astype(np.float64)) + torch.from_numpy(w_o.astype(np.float64))[:, None, None, None]
    # value-zero padding is what conv2d's own padding does
    _, out1, _ = oracle.conv2d(x, w, stride, pad, oracle.PAD_VALUE_ZERO, a_s, a_o, w_s, w_o)
    ref1 = F.conv2d(xd, wd, stride=stride, padding=pad).numpy()
    assert np.allclose(out1, ref1, rtol=1e-12, atol=1e-10)
    # code-zero padding: the border holds code 0, whose real value is a_o
    _, out0, _ = oracle.conv2d(x, w, stride, pad, oracle.PAD_CODE_ZERO, a_s, a_o, w_s, w_o)
    ref0 = F.conv2d(F.pad(xd, (pad,) * 4, value=a_o), wd, stride=stride, padding=0).numpy()
    assert np.allclose(out0, ref0, rtol=1e-12, atol=1e-10)
    if pad > 0:
        assert not np.allclose(out0, out1)


def test_conv2d_integer_sums_against_torch_integer_conv():
    g = np.random.default_rng(33)
    x = inputs.weight_codes(g, (2, 6, 7, 7), 0.3)
    w = inputs.weight_codes(g, (3, 6, 3, 3), 0.4)
    S, _, _ = oracle.conv2d(x, w, 1, 1, oracle.PAD_CODE_ZERO, 1.0, 0.0, 1.0, 0.0)
    ref = F.conv2d(torch.from_numpy(x.astype(np.float64)), torch.from_numpy(w.astype(np.float64)),
                   padding=1).numpy()
    assert np.array_equal(S, ref.astype(np.int64))


def test_conv2d_code_zero_equals_gemm_on_materialised_patches():
    g = np.random.default_rng(41)
    B, C, H, W, N, k, stride, pad = 2, 7, 6, 5, 3, 3, 2, 1
    x = inputs.weight_codes(g, (B, C, H, W), 0.3)
    w = inputs.weight_codes(g, (N, C, k, k), 0.4)
    w_s, w_o = inputs.uniform(g, 0.5, 1.5, (N,)), inputs.uniform(g, -0.5, 0.5, (N,))
    S, out, _ = oracle.conv2d(x, w, stride, pad, oracle.PAD_CODE_ZERO, 0.75, 0.125, w_s, w_o)
    cols = oracle.im2col(x, k, k, stride, pad)
    Sg, outg, _ = oracle.gemm(cols, w.reshape(N, -1), 0.75, 0.125, w_s, w_o)
    Ho, Wo = S.shape[2:]
    assert np.array_equal(S, Sg.reshape(B, Ho, Wo, N).transpose(0, 3, 1, 2))
    assert np.allclose(out, outg.reshape(B, Ho, Wo, N).transpose(0, 3, 1, 2), rtol=1e-14, atol=1e-12)


def test_conv1x1_stride1_is_a_gemm():
    g = np.random.default_rng(42)
    B, C, H, W, N = 2, 9, 4, 3, 5
    x = inputs.weight_codes(g, (B, C, H, W), 0.3)
    w = inputs.weight_codes(g, (N, C, 1, 1), 0.4)
    S, _, _ = oracle.conv2d(x, w, 1, 0, oracle.PAD_CODE_ZERO, 1.0, 0.0, 1.0, 0.0)
    ref = np.einsum("bchw,nc->bnhw", x.astype(np.int64), w[:, :, 0, 0].astype(np.int64))
    assert np.array_equal(S, ref)


def test_conv2d_points_match_full():
    g = np.random.default_rng(43)
    x = inputs.weight_codes(g, (2, 4, 6, 6), 0.3)
    w = inputs.weight_codes(g, (3, 4, 3, 3), 0.4)
    w_s, w_o = inputs.uniform(g, 0.5, 1.5, (3,)), inputs.uniform(g, -0.5, 0.5, (3,))
    for mode in (oracle.PAD_CODE_ZERO, oracle.PAD_VALUE_ZERO):
        S, out, mag = oracle.conv2d(x, w, 1, 1, mode, 1.1, 0.2, w_s, w_o)
        pts = np.array([[0, 0, 0, 0], [1, 2, 5, 5], [0, 1, 3, 0], [1, 0, 0, 4]], np.int64)
        Sp, op, mp = oracle.conv2d_points(x, w, 1, 1, mode, 1.1, 0.2, w_s, w_o, pts)
        for i, (b, n, h, v) in enumerate(pts):
            assert Sp[i] == S[b, n, h, v] and op[i] == out[b, n, h, v] and mp[i] == mag[b, n, h, v]


def test_conv_weight_sums_per_tap():
    g = np.random.default_rng(44)
    w = inputs.weight_codes(g, (4, 6, 3, 3), 0.4)
    sums = oracle.conv_weight_sums(w)
    assert np.array_equal(sums[0], w.astype(np.int64).sum((1, 2, 3)))
    assert np.array_equal(sums[1:], w.astype(np.int64).sum(1).reshape(4, 9).T)


# ------------------------------------------------------------------ packed format
def test_pack_rows_golden_bytes():
    # K = 130: two blocks.  codes: k=0 -> +1, k=1 -> -1, k=9 -> +1, k=127 -> -1, k=128 -> +1, k=129 -> -1
    codes = np.zeros((1, 130), np.int8)
    codes[0, [0, 9, 128]] = 1
    codes[0, [1, 127, 129]] = -1
    p = oracle.pack_rows(codes)
    assert p.shape == (1, 64)
    want = np.zeros(64, np.uint8)
    want[0] = 0b11          # first-bit plane: k=0, k=1
    want[1] = 0b10          # k=9
    want[15] = 0x80         # k=127
    want[16] = 0b01         # second-bit plane: k=0 positive
    want[17] = 0b10         # k=9 positive
    want[32] = 0b11         # block 1, first-bit plane: k=128, 129
    want[48] = 0b01         # block 1, second-bit plane: k=128 positive
    assert p[0].tolist() == want.tolist()


@pytest.mark.parametrize("K", [1, 31, 32, 127, 128, 129, 576, 1000])
def test_pack_round_trip(K):
    g = np.random.default_rng(K)
    codes = inputs.weight_codes(g, (5, K), 0.4)
    p = oracle.pack_rows(codes)
    assert p.shape[1] == (K + 127) // 128 * 32 == oracle.packed_row_bytes(K)
    assert np.array_equal(oracle.unpack_rows(p, K), codes)
    # a non-canonical zero (01) decodes to 0 and re-packs to the canonical 00
    q = p.copy()
    zero_at = np.argwhere(codes[0] == 0)
    if len(zero_at):
        k = int(zero_at[0, 0])
        q[0, (k // 128) * 32 + 16 + (k % 128) // 8] |= 1 << (k % 8)
        assert np.array_equal(oracle.unpack_rows(q, K), codes)
        assert np.array_equal(oracle.pack_rows(oracle.unpack_rows(q, K)), p)


def test_conv_weight_rows_order_is_tap_major_channel_minor():
    w = np.zeros((1, 3, 2, 2), np.int8)
    w[0, 2, 1, 0] = -1           # channel 2, tap (1,0) -> index (1*2+0)*32 + 2
    w[0, 0, 0, 1] = 1            # channel 0, tap (0,1) -> index (0*2+1)*32 + 0
    rows = oracle.conv_weight_rows(w)
    assert rows.shape == (1, 2 * 2 * 32)
    nz = {int(i): int(rows[0, i]) for i in np.flatnonzero(rows[0])}
    assert nz == {2 * 32 + 2: -1, 1 * 32 + 0: 1}


# ------------------------------------------------------------------ layer list
def test_resnet18_layer_list_matches_the_appendix_table():
    names = [r[0] for r in read_golden("table4_layers.txt")]
    layers = inputs.resnet18_ternary_layers()
    assert sorted(names) == sorted(l[0] for l in layers) and len(layers) == 19
    assert sum(1 for l in layers if l[3] == 3) == 16 and sum(1 for l in layers if l[3] == 1) == 3


# ------------------------------------------------------------------ what a layer hands to the next one
def test_next_layer_hand_case_order_and_ties():
    # phi acts on the conv output BEFORE the skip connection is added; strict comparisons
    pre = np.array([[[-1.0, 0.2, 3.0, 0.25, -4.0]]])           # [B=1][N=1][5]
    skip = np.array([[[0.5, 0.5, -2.0, 0.5, -1.0]]], np.float32)
    y, codes, margin = oracle.next_layer(pre, True, skip, 0.6, 0.75)
    assert y.ravel().tolist() == [0.5, 0.7, 1.0, 0.75, -1.0]    # relu(-1)+0.5, ..., relu(-4)-1
    assert codes.ravel().tolist() == [-1, 0, 1, 0, -1]          # y == t_hi codes to 0
    assert margin.ravel()[3] == 0.0
    y2, codes2, _ = oracle.next_layer(pre, False, None, 0.6, 0.75)
    assert y2.ravel().tolist() == pre.ravel().tolist()
    assert codes2.ravel().tolist() == [-1, -1, 1, -1, -1]


def test_next_layer_relu_is_eq11_folded_form():
    # Eq. 11: phi(alpha gamma S + C) = alpha * max(0, gamma S + T), T = beta * (1 (x) W^t), alpha > 0
    g = np.random.default_rng(41)
    x = inputs.weight_codes(g, (2, 6, 7, 7), 0.3)
    w = inputs.weight_codes(g, (5, 6, 3, 3), 0.4)
    gamma, beta = 1.25, -0.375
    alpha = inputs.uniform(g, 0.5, 1.5, (5,))
    S, pre, _ = oracle.conv2d(x, w, 1, 1, oracle.PAD_CODE_ZERO, gamma, beta, alpha, np.zeros(5, np.float32))
    y, _, _ = oracle.next_layer(pre, True, None, 0.0, 0.0)
    T = beta * w.astype(np.int64).sum(axis=(1, 2, 3))
    a64 = alpha.astype(np.float64)[None, :, None, None]
    want = a64 * np.maximum(0.0, gamma * S + T[None, :, None, None])
    assert np.allclose(y, want, rtol=1e-12, atol=1e-12)
    assert (y >= 0).all() and (y == 0).any() and (y > 0).any()


@pytest.mark.parametrize("relu,with_skip", [(True, True), (True, False), (False, True)])
def test_next_layer_against_torch_fp64_block(relu, with_skip):
    # conv on de-quantised values -> ReLU -> + skip -> BN transform (Eq. 2) -> Q of Eq. 1, all in torch fp64
    g = np.random.default_rng(43)
    B, C, H, W, N = 2, 5, 8, 8, 6
    x = inputs.weight_codes(g, (B, C, H, W), 0.3)
    w = inputs.weight_codes(g, (N, C, 3, 3), 0.4)
    a_s, a_o = 0.75, 0.125
    w_s, w_o = inputs.uniform(g, 0.5, 1.5, (N,)), inputs.uniform(g, -0.1, 0.1, (N,))
    skip = g.standard_normal((B, N, H, W)).astype(np.float32) if with_skip else None
    k = inputs.uniform(g, 0.2, 0.6, (N,)).astype(np.float64)      # BN scale (k > 0) and shift per channel
    b = inputs.uniform(g, -1.2, -0.7, (N,)).astype(np.float64)    # t_lo > 0: -1 occurs after a ReLU too
    t_hi = ((0.5 - b) / k).astype(np.float32)
    t_lo = (-(0.5 + b) / k).astype(np.float32)
    _, pre, _ = oracle.conv2d(x, w, 1, 1, oracle.PAD_VALUE_ZERO, a_s, a_o, w_s, w_o)
    y, codes, margin = oracle.next_layer(pre, relu, skip, t_lo, t_hi)

    xd = _deq(x, a_s, a_o)
    wd = torch.from_numpy(w_s.astype(np.float64))[:, None, None, None] * torch.from_numpy(
        w.astype(np.float64)) + torch.from_numpy(w_o.astype(np.float64))[:, None, None, None]
    ref = F.conv2d(xd, wd, padding=1)
    if relu:
        ref = F.relu(ref)
    if with_skip:
        ref = ref + torch.from_numpy(skip.astype(np.float64))
    assert np.allclose(y, ref.numpy(), rtol=1e-12, atol=1e-10)
    bn = torch.from_numpy(k)[None, :, None, None] * ref + torch.from_numpy(b)[None, :, None, None]
    q = torch.where(bn.abs() > 0.5, torch.sign(bn), torch.zeros_like(bn)).numpy().astype(np.int8)
    clear = margin > 1e-5            # fp32 thresholds and fp32(y) move a decision only this close to a threshold
    assert clear.mean() > 0.99
    assert np.array_equal(codes[clear], q[clear])
    assert set(np.unique(codes).tolist()) == {-1, 0, 1}


def test_next_layer_per_channel_thresholds_index_axis_1():
    pre = np.zeros((2, 3, 4))
    pre[:, 1] = 1.0
    _, codes, _ = oracle.next_layer(pre, False, None, np.array([-1, 2, -1], np.float32),
                                    np.array([-0.5, 3, 0.5], np.float32))
    assert (codes[:, 0] == 1).all() and (codes[:, 1] == -1).all() and (codes[:, 2] == 0).all()


def test_pack_nhwc_is_one_packed_row_per_pixel():
    g = np.random.default_rng(47)
    B, C, H, W = 2, 70, 3, 5
    codes = inputs.weight_codes(g, (B, C, H, W), 0.3)
    packed = oracle.pack_nhwc(codes)
    assert packed.shape == (B * H * W, 32)
    # pixel (b=1, h=2, w=3): its row is the pack of its C channel codes
    row = (1 * H + 2) * W + 3
    assert np.array_equal(packed[row], oracle.pack_rows(codes[1, :, 2, 3][None, :])[0])
    # channel 9 of that pixel: bit 1 of byte 1 of plane 1 (non-zero) and of plane 2 (positive)
    c = int(codes[1, 9, 2, 3])
    assert (packed[row, 1] >> 1) & 1 == (1 if c != 0 else 0)
    assert (packed[row, 17] >> 1) & 1 == (1 if c > 0 else 0)
    assert np.array_equal(oracle.unpack_nhwc(packed, B, C, H, W), codes)


def test_two_layer_chain_against_torch_fp64():
    # layer 1 -> phi -> ternarize -> layer 2: the codes the first layer hands over are the second's input
    g = np.random.default_rng(53)
    B, C, H, W, N1, N2 = 1, 4, 6, 6, 5, 3
    x = inputs.weight_codes(g, (B, C, H, W), 0.3)
    w1 = inputs.weight_codes(g, (N1, C, 3, 3), 0.4)
    w2 = inputs.weight_codes(g, (N2, N1, 3, 3), 0.4)
    ws1, ws2 = inputs.uniform(g, 0.5, 1.5, (N1,)), inputs.uniform(g, 0.5, 1.5, (N2,))
    zero1, zero2 = np.zeros(N1, np.float32), np.zeros(N2, np.float32)
    _, pre1, _ = oracle.conv2d(x, w1, 1, 1, oracle.PAD_VALUE_ZERO, 1.0, 0.25, ws1, zero1)
    _, codes1, margin = oracle.next_layer(pre1, True, None, 0.5, 2.0)
    assert margin.min() > 1e-6
    _, pre2, _ = oracle.conv2d(codes1, w2, 1, 1, oracle.PAD_VALUE_ZERO, 0.5, -0.125, ws2, zero2)

    def deq_w(w, s):
        return torch.from_numpy(s.astype(np.float64))[:, None, None, None] * torch.from_numpy(w.astype(np.float64))
    h = F.relu(F.conv2d(_deq(x, 1.0, 0.25), deq_w(w1, ws1), padding=1))
    c = torch.where(h > 2.0, 1.0, torch.where(h < 0.5, -1.0, 0.0)).to(torch.float64)
    ref = F.conv2d(0.5 * c - 0.125, deq_w(w2, ws2), padding=1).numpy()
    assert np.allclose(pre2, ref, rtol=1e-12, atol=1e-10)


# ------------------------------------------------------------------ the 2-bit comparison workload
def test_table1_quaternary_column_matches_paper_rows():
    rows = read_golden("table1_quaternary.txt")
    assert len(rows) == 4
    for b1, b2, val in rows:
        assert int(oracle.quaternary_decode([int(b1)], [int(b2)])[0]) == int(val)
    v = np.arange(4, dtype=np.uint8)
    b1, b2 = oracle.quaternary_encode(v)
    assert b1.tolist() == [0, 0, 1, 1] and b2.tolist() == [0, 1, 0, 1]
    assert oracle.quaternary_decode(b1, b2).tolist() == [0, 1, 2, 3]


def test_quaternary_bit_formula_exhaustive_and_brute_force():
    for x in range(4):
        for w in range(4):
            x1, x2 = oracle.quaternary_encode([x])
            w1, w2 = oracle.quaternary_encode([w])
            assert oracle.dot_quaternary_bits(x1, x2, w1, w2) == x * w
    g = np.random.default_rng(61)
    for n in (1, 31, 32, 33, 129, 300):
        x, w = g.integers(0, 4, n).astype(np.uint8), g.integers(0, 4, n).astype(np.uint8)
        want = sum(int(a) * int(b) for a, b in zip(x.tolist(), w.tolist()))
        assert oracle.dot_quaternary_bits(*oracle.quaternary_encode(x), *oracle.quaternary_encode(w)) == want


def test_quaternary_gemm_against_numpy_and_hand_cases():
    g = np.random.default_rng(67)
    x, w = g.integers(0, 4, (7, 45)).astype(np.uint8), g.integers(0, 4, (5, 45)).astype(np.uint8)
    assert np.array_equal(oracle.quaternary_gemm(x, w), x.astype(np.int64) @ w.astype(np.int64).T)
    assert oracle.quaternary_gemm(np.full((1, 10), 3, np.uint8), np.full((1, 10), 3, np.uint8))[0, 0] == 90
    # a transposed operand changes the result
    sq = g.integers(0, 4, (6, 6)).astype(np.uint8)
    y = g.integers(0, 4, (6, 6)).astype(np.uint8)
    assert not np.array_equal(oracle.quaternary_gemm(sq, y), oracle.quaternary_gemm(sq, y.T.copy()))


def test_pack_quaternary_rows_planes():
    v = np.zeros((1, 130), np.uint8)
    v[0, 0], v[0, 9], v[0, 129] = 3, 2, 1
    p = oracle.pack_quaternary_rows(v)
    assert p.shape == (1, 64)
    assert p[0, 0] == 1 and p[0, 16] == 1              # value 3 at position 0: both planes
    assert p[0, 1] == 2 and p[0, 17] == 0              # value 2 at position 9: first-bit plane only
    assert p[0, 32] == 0 and p[0, 48] == 2             # value 1 at position 129: second-bit plane of block 1
    assert p.sum() == 1 + 1 + 2 + 2


# ------------------------------------------------------------------ the chain's recipe (host logic, no arithmetic of the method)
@pytest.mark.parametrize("hin", [56, 28, 16])
def test_resnet18_body_recipe_is_a_consistent_chain(hin):
    layers = inputs.resnet18_body(seed=4, hin=hin)
    assert [l.name for l in layers] == [l[0] for l in inputs.resnet18_ternary_layers()]
    blocks = inputs.resnet18_body_blocks(layers)
    assert len(blocks) == 8 and sum(b["down"] is not None for b in blocks) == 3
    size, chans = hin, 64
    for blk in blocks:
        c1, c2, down = blk["conv1"], blk["conv2"], blk["down"]
        assert c1.cin == chans and c1.hin == size
        out = oracle.conv_out_dim(c1.hin, c1.k, c1.stride, c1.pad)
        assert c2.cin == c1.cout and c2.hin == out and c2.stride == 1
        assert oracle.conv_out_dim(c2.hin, c2.k, 1, c2.pad) == out
        if down is not None:
            assert (down.cin, down.cout, down.hin) == (c1.cin, c2.cout, c1.hin)
            assert oracle.conv_out_dim(down.hin, down.k, down.stride, down.pad) == out
        else:
            assert c1.stride == 1 and c1.cin == c2.cout      # the skip is the block's input itself
        for l in (c1, c2, down):
            if l is not None:
                assert 0 < float(l.t_lo[0]) < float(l.t_hi[0])
        size, chans = out, c2.cout
    if hin == 56:
        assert (size, chans) == (7, 512)
