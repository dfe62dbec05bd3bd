"""GPU parity of the entry points that hand a layer's result to the next layer
(rtn_ternary_conv2d_fused: fp32 input, rtn_ternary_conv2d_packed: packed pixel rows) against the
CPU oracle.  Integer accumulators bit-exact; fp32 y within the library's tolerance (the skip
connection adds one term to sum |term_i|); packed codes bit-exact wherever the oracle's double y is
farther from both thresholds than that tolerance, and one of the two neighbouring codes elsewhere.
With dyadic parameters every intermediate is exact in fp32, and the codes are bit-exact everywhere."""
import numpy as np
import pytest
import torch

import oracle
import paper_1912_02057_b200 as rtn
from paper_1912_02057_b200 import inputs
from helpers import check_fp32, dev

pytestmark = pytest.mark.gpu


def next_thresholds(g, N, per_channel, lo=0.2, hi=1.5):
    if per_channel:
        return inputs.uniform(g, lo - 0.1, lo + 0.1, (N,)), inputs.uniform(g, hi - 0.3, hi + 0.3, (N,))
    return np.array([lo], np.float32), np.array([hi], np.float32)


def run_layer(case, codes_in, packed_in, pad_mode, relu, skip, want_out, nlo, nhi):
    """One layer through the C ABI.  Returns (acc, y or None, packed rows or None) as numpy."""
    B, C, H, W, N, Ho, Wo = case.B, case.C, case.H, case.W, case.N, case.Ho, case.Wo
    w_packed, w_sum = rtn.rtn_pack_weights(dev(case.w_codes))
    acc = torch.full((B, N, Ho, Wo), -12345, dtype=torch.int32, device="cuda")
    out = torch.full((B, N, Ho, Wo), float("nan"), dtype=torch.float32, device="cuda") if want_out else None
    outp = None
    if nlo is not None:
        outp = torch.full((B * Ho * Wo, rtn.rtn_packed_row_bytes(N)), 0xA5, dtype=torch.uint8, device="cuda")
    common = dict(relu=relu, skip=None if skip is None else dev(skip), out=out,
                  next_t_lo=None if nlo is None else dev(nlo), next_t_hi=None if nhi is None else dev(nhi),
                  out_packed=outp, dbg_acc=acc)
    if packed_in:
        rtn.rtn_ternary_conv2d_packed(dev(oracle.pack_nhwc(codes_in)), B, C, H, W, w_packed, w_sum, N,
                                      case.kh, case.kw, case.stride, case.pad, pad_mode, case.a_scale,
                                      case.a_offset, dev(case.w_scale), dev(case.w_offset), **common)
    else:
        rtn.rtn_ternary_conv2d_fused(dev(case.x), dev(case.t_lo), dev(case.t_hi), w_packed, w_sum, N,
                                     case.kh, case.kw, case.stride, case.pad, pad_mode, case.a_scale,
                                     case.a_offset, dev(case.w_scale), dev(case.w_offset), **common)
    torch.cuda.synchronize()
    assert rtn.rtn_last_device_status() == 0
    return (acc.cpu().numpy(), None if out is None else out.cpu().numpy(),
            None if outp is None else outp.cpu().numpy())


def check_layer(case, packed_in, pad_mode, relu, with_skip, want_out, want_packed, per_channel_next, seed,
                exact=False):
    g = inputs.rng(seed)
    codes_in = oracle.ternarize(case.x, case.t_lo, case.t_hi, channel_axis=1)
    skip = None
    if with_skip:
        skip = g.standard_normal((case.B, case.N, case.Ho, case.Wo)).astype(np.float32)
        if exact:
            skip = np.round(skip * 8) / 8
    nlo = nhi = None
    if want_packed:
        nlo, nhi = next_thresholds(g, case.N, per_channel_next)
    acc, y, packed = run_layer(case, codes_in, packed_in, pad_mode, relu, skip, want_out, nlo, nhi)
    S, pre, mag = oracle.conv2d(codes_in, case.w_codes, case.stride, case.pad, pad_mode, case.a_scale,
                                case.a_offset, case.w_scale, case.w_offset)
    assert np.array_equal(acc.astype(np.int64), S), f"{case.name}: integer accumulators differ"
    lo_ref = np.float32(-np.inf) if nlo is None else nlo
    hi_ref = np.float32(np.inf) if nhi is None else nhi
    y_ref, codes_ref, margin = oracle.next_layer(pre, relu, skip, lo_ref, hi_ref)
    mag_y = mag if skip is None else mag + np.abs(skip.astype(np.float64))
    if want_out:
        check_fp32(y, y_ref, mag_y, case.name + " y")
        if exact:
            assert np.array_equal(y.astype(np.float64), y_ref)
    if want_packed:
        got = oracle.unpack_nhwc(packed, case.B, case.N, case.Ho, case.Wo)
        # the packed rows are canonical: re-packing the decoded codes gives the same bytes (00 zeros, zero fill)
        assert np.array_equal(packed, oracle.pack_nhwc(got)), "packed rows not canonical / not zero-filled"
        tol = np.maximum(oracle.REL_TOL * np.abs(y_ref), oracle.ABS_TOL * np.maximum(1.0, mag_y))
        clear = margin > tol
        if exact:
            clear[:] = True
        assert clear.mean() > 0.999
        assert np.array_equal(got[clear], codes_ref[clear]), f"{case.name}: codes differ away from the thresholds"
        # inside the band a code may fall on either side of the threshold it is near, never further
        assert (np.abs(got.astype(np.int32) - codes_ref.astype(np.int32))[~clear] <= 1).all()
        assert set(np.unique(got).tolist()) == {-1, 0, 1}
    return codes_ref


SHAPES = [
    # name, B, C, H, W, N, k, stride, pad
    ("c64_3x3", 2, 64, 12, 12, 64, 3, 1, 1),
    ("ragged", 3, 40, 9, 11, 70, 3, 1, 1),
    ("s2_3x3", 2, 64, 14, 14, 128, 3, 2, 1),
    ("s2_1x1", 2, 64, 14, 14, 128, 1, 2, 0),
    ("n512", 1, 96, 7, 7, 512, 3, 1, 1),
    ("n16_c200", 2, 200, 6, 6, 16, 3, 1, 1),
    ("n257", 1, 32, 5, 5, 257, 1, 1, 0),
]


@pytest.mark.parametrize("packed_in", [False, True], ids=["fp32_in", "packed_in"])
@pytest.mark.parametrize("shape", SHAPES, ids=[s[0] for s in SHAPES])
def test_next_layer_shapes(shape, packed_in):
    name, B, C, H, W, N, k, stride, pad = shape
    case = inputs.conv_case(name, B, C, H, W, N, k, stride, pad, seed=len(name) + C + N, p_zero=0.4,
                            thresholds=(0.3, 1.0), per_channel_thresholds=True)
    check_layer(case, packed_in, oracle.PAD_CODE_ZERO, relu=True, with_skip=True, want_out=True,
                want_packed=True, per_channel_next=True, seed=7)


@pytest.mark.parametrize("relu,with_skip,want_out,want_packed,per_ch", [
    (True, False, False, True, False),       # conv1 of a block: packed codes only
    (False, True, True, False, False),       # fp32 only, no phi
    (True, True, True, True, True),          # conv2 of a block: skip, fp32 for the next skip, codes
    (False, False, True, True, True),
])
@pytest.mark.parametrize("pad_mode", [oracle.PAD_CODE_ZERO, oracle.PAD_VALUE_ZERO], ids=["code0", "value0"])
def test_next_layer_options(relu, with_skip, want_out, want_packed, per_ch, pad_mode):
    case = inputs.conv_case("opts", 2, 64, 10, 10, 96, 3, 1, 1, seed=11, p_zero=0.4, thresholds=(0.3, 1.0))
    for packed_in in (False, True):
        check_layer(case, packed_in, pad_mode, relu, with_skip, want_out, want_packed, per_ch, seed=13)


def dyadic_case(name, B, C, H, W, N, k, stride, pad, seed):
    """Parameters that are small multiples of powers of two: every product and sum of the epilogue is
    exact in fp32 and in double, so both sides hold the same y and decide the same codes."""
    case = inputs.conv_case(name, B, C, H, W, N, k, stride, pad, seed=seed, p_zero=0.4, thresholds=(0.3, 1.0))
    g = inputs.rng(seed + 1)
    case.w_scale = (g.integers(2, 7, N) / 4.0).astype(np.float32)
    case.w_offset = (g.integers(-2, 3, N) / 16.0).astype(np.float32)
    case.a_scale, case.a_offset = 0.75, 0.125
    return case


@pytest.mark.parametrize("packed_in", [False, True], ids=["fp32_in", "packed_in"])
def test_next_layer_dyadic_parameters_give_bit_exact_codes(packed_in):
    case = dyadic_case("dyadic", 2, 64, 12, 12, 64, 3, 1, 1, seed=17)
    check_layer(case, packed_in, oracle.PAD_CODE_ZERO, relu=True, with_skip=True, want_out=True,
                want_packed=True, per_channel_next=False, seed=19, exact=True)


def test_two_blocks_chained_through_packed_rows():
    """conv1 (fp32 in -> codes) -> conv2 (codes in, + skip -> fp32 and codes) -> conv1' (codes in): each
    layer consumes the packed rows the one before wrote; the oracle runs the same chain on its own
    codes.  Dyadic parameters keep every threshold decision exact, so the chains cannot drift apart."""
    B, C, H = 2, 64, 12
    c1 = dyadic_case("chain1", B, C, H, H, C, 3, 1, 1, seed=23)
    c2 = dyadic_case("chain2", B, C, H, H, C, 3, 1, 1, seed=29)
    c3 = dyadic_case("chain3", B, C, H, H, 128, 3, 2, 1, seed=31)
    c1.x = (np.round(c1.x * 8) / 8).astype(np.float32)       # it is also conv2's skip: keep that sum exact
    n12 = (np.array([0.5], np.float32), np.array([2.0], np.float32))
    n23 = (np.array([0.25], np.float32), np.array([1.75], np.float32))
    D = lambda c: dict(w=rtn.rtn_pack_weights(dev(c.w_codes)), ws=dev(c.w_scale), wo=dev(c.w_offset))
    d1, d2, d3 = D(c1), D(c2), D(c3)
    x = dev(c1.x)
    p1 = torch.empty((B * H * H, rtn.rtn_packed_row_bytes(C)), dtype=torch.uint8, device="cuda")
    p2 = torch.empty_like(p1)
    y2 = torch.empty((B, C, H, H), dtype=torch.float32, device="cuda")
    y3 = torch.empty((B, 128, H // 2, H // 2), dtype=torch.float32, device="cuda")
    rtn.rtn_ternary_conv2d_fused(x, dev(c1.t_lo), dev(c1.t_hi), *d1["w"], C, 3, 3, 1, 1, rtn.PAD_CODE_ZERO,
                                 c1.a_scale, c1.a_offset, d1["ws"], d1["wo"], relu=True,
                                 next_t_lo=dev(n12[0]), next_t_hi=dev(n12[1]), out_packed=p1)
    rtn.rtn_ternary_conv2d_packed(p1, B, C, H, H, *d2["w"], C, 3, 3, 1, 1, rtn.PAD_CODE_ZERO,
                                  c2.a_scale, c2.a_offset, d2["ws"], d2["wo"], relu=True, skip=x, out=y2,
                                  next_t_lo=dev(n23[0]), next_t_hi=dev(n23[1]), out_packed=p2)
    rtn.rtn_ternary_conv2d_packed(p2, B, C, H, H, *d3["w"], 128, 3, 3, 2, 1, rtn.PAD_CODE_ZERO,
                                  c3.a_scale, c3.a_offset, d3["ws"], d3["wo"], relu=True, out=y3)
    torch.cuda.synchronize()
    assert rtn.rtn_last_device_status() == 0

    k0 = oracle.ternarize(c1.x, c1.t_lo, c1.t_hi)
    _, pre1, _ = oracle.conv2d(k0, c1.w_codes, 1, 1, oracle.PAD_CODE_ZERO, c1.a_scale, c1.a_offset, c1.w_scale, c1.w_offset)
    _, k1, _ = oracle.next_layer(pre1, True, None, *n12)
    _, pre2, _ = oracle.conv2d(k1, c2.w_codes, 1, 1, oracle.PAD_CODE_ZERO, c2.a_scale, c2.a_offset, c2.w_scale, c2.w_offset)
    r2, k2, _ = oracle.next_layer(pre2, True, c1.x, *n23)
    _, pre3, mag3 = oracle.conv2d(k2, c3.w_codes, 2, 1, oracle.PAD_CODE_ZERO, c3.a_scale, c3.a_offset, c3.w_scale, c3.w_offset)
    r3, _, _ = oracle.next_layer(pre3, True, None, np.float32(-np.inf), np.float32(np.inf))
    assert np.array_equal(oracle.unpack_nhwc(p1.cpu().numpy(), B, C, H, H), k1)
    assert np.array_equal(oracle.unpack_nhwc(p2.cpu().numpy(), B, C, H, H), k2)
    check_fp32(y2.cpu().numpy(), r2, np.abs(r2) + 1.0, "chain y2")
    check_fp32(y3.cpu().numpy(), r3, mag3, "chain y3")


def test_packed_input_accepts_rows_written_by_ternarize_pack_act():
    """rtn_ternarize_pack_act on the NHWC view of the input gives the x_packed of the packed entry."""
    case = inputs.conv_case("nhwc", 2, 64, 10, 10, 64, 3, 1, 1, seed=37, p_zero=0.4, thresholds=(0.3, 1.0),
                            per_channel_thresholds=True)
    B, C, H, W, N = case.B, case.C, case.H, case.W, case.N
    nhwc = dev(np.ascontiguousarray(case.x.transpose(0, 2, 3, 1)).reshape(B * H * W, C))
    xp, _ = rtn.rtn_ternarize_pack_act(nhwc, dev(case.t_lo), dev(case.t_hi), want_sum=False)
    w_packed, w_sum = rtn.rtn_pack_weights(dev(case.w_codes))
    out = torch.empty((B, N, H, W), dtype=torch.float32, device="cuda")
    rtn.rtn_ternary_conv2d_packed(xp, B, C, H, W, w_packed, w_sum, N, 3, 3, 1, 1, rtn.PAD_CODE_ZERO,
                                  case.a_scale, case.a_offset, dev(case.w_scale), dev(case.w_offset), out=out)
    ref = rtn.rtn_ternary_conv2d(dev(case.x), dev(case.t_lo), dev(case.t_hi), w_packed, w_sum, N, 3, 3, 1, 1,
                                 rtn.PAD_CODE_ZERO, case.a_scale, case.a_offset, dev(case.w_scale),
                                 dev(case.w_offset))
    codes = oracle.ternarize(case.x, case.t_lo, case.t_hi, channel_axis=1)
    _, want, mag = oracle.conv2d(codes, case.w_codes, 1, 1, oracle.PAD_CODE_ZERO, case.a_scale, case.a_offset,
                                 case.w_scale, case.w_offset)
    check_fp32(out.cpu().numpy(), want, mag, "packed input from ternarize_pack_act")
    check_fp32(ref.cpu().numpy(), want, mag, "fp32 entry")


def test_packed_input_treats_01_as_zero_and_ignores_bits_past_C():
    g = inputs.rng(41)
    B, C, H, W, N = 1, 40, 6, 6, 32
    codes = inputs.weight_codes(g, (B, C, H, W), 0.4)
    case = inputs.conv_case("nc", B, C, H, W, N, 3, 1, 1, seed=43, p_zero=0.4)
    packed = oracle.pack_nhwc(codes).copy()
    nzp, sgp = packed[:, 0:16], packed[:, 16:32]
    sgp |= (~nzp) & g.integers(0, 256, sgp.shape).astype(np.uint8)      # second zero of Table 1 (01), and junk
    nzp[:, 5:] |= g.integers(0, 256, nzp[:, 5:].shape).astype(np.uint8)  # positions 40.. of the non-zero plane
    w_packed, w_sum = rtn.rtn_pack_weights(dev(case.w_codes))
    out = torch.empty((B, N, H, W), dtype=torch.float32, device="cuda")
    acc = torch.empty((B, N, H, W), dtype=torch.int32, device="cuda")
    rtn.rtn_ternary_conv2d_packed(dev(packed), B, C, H, W, w_packed, w_sum, N, 3, 3, 1, 1, rtn.PAD_CODE_ZERO,
                                  case.a_scale, case.a_offset, dev(case.w_scale), dev(case.w_offset), out=out,
                                  dbg_acc=acc)
    S, want, mag = oracle.conv2d(codes, case.w_codes, 1, 1, oracle.PAD_CODE_ZERO, case.a_scale, case.a_offset,
                                 case.w_scale, case.w_offset)
    assert np.array_equal(acc.cpu().numpy().astype(np.int64), S)
    check_fp32(out.cpu().numpy(), want, mag, "non-canonical packed input")


def test_next_layer_argument_errors():
    case = inputs.conv_case("err", 1, 32, 6, 6, 32, 3, 1, 1, seed=47, p_zero=0.4)
    w_packed, w_sum = rtn.rtn_pack_weights(dev(case.w_codes))
    args = (dev(case.x), dev(case.t_lo), dev(case.t_hi), w_packed, w_sum, 32, 3, 3, 1, 1, rtn.PAD_CODE_ZERO,
            case.a_scale, case.a_offset, dev(case.w_scale), dev(case.w_offset))
    with pytest.raises(rtn.RtnError) as e:                      # neither output requested
        rtn.rtn_ternary_conv2d_fused(*args)
    assert e.value.code == 1
    outp = torch.empty((36, 32), dtype=torch.uint8, device="cuda")
    with pytest.raises(rtn.RtnError) as e:                      # packed output without thresholds
        rtn.rtn_ternary_conv2d_fused(*args, out_packed=outp)
    assert e.value.code == 1
    with pytest.raises(rtn.RtnError) as e:                      # 3 thresholds for 32 channels
        rtn.rtn_ternary_conv2d_fused(*args, out_packed=outp, next_t_lo=dev(np.zeros(3, np.float32)),
                                     next_t_hi=dev(np.ones(3, np.float32)))
    assert e.value.code == 2


@pytest.mark.parametrize("name,maker", [
    ("cfg2", lambda: inputs.config2(batch=32, thresholds=(0.3, 1.0))),          # one-kernel variant
    ("cfg3a", lambda: inputs.config3a(0.5, batch=128)),                          # two-kernel variant
])
def test_next_layer_full_size_sampled(name, maker):
    """The benchmark's shapes at full batch, in the launch configuration bench.py times (packed rows in, ReLU,
    skip, fp32 and packed rows out): sampled outputs against the oracle point by point, the four image corners
    and the last channel included."""
    case = maker()
    g = inputs.rng(91)
    B, C, H, W, N, Ho, Wo = case.B, case.C, case.H, case.W, case.N, case.Ho, case.Wo
    codes_in = oracle.ternarize(case.x, case.t_lo, case.t_hi, channel_axis=1)
    skip = g.standard_normal((B, N, Ho, Wo)).astype(np.float32)
    nlo, nhi = next_thresholds(g, N, True, lo=2.0, hi=12.0)
    acc, y, packed = run_layer(case, codes_in, True, oracle.PAD_CODE_ZERO, True, skip, True, nlo, nhi)
    n_pts = 6000
    pts = np.stack([g.integers(0, B, n_pts), g.integers(0, N, n_pts), g.integers(0, Ho, n_pts),
                    g.integers(0, Wo, n_pts)], 1)
    corners = [(b, n, h, v) for b in (0, B - 1) for n in (0, N - 1) for h in (0, Ho - 1) for v in (0, Wo - 1)]
    pts = np.concatenate([pts, np.array(corners, np.int64)], 0)
    S, pre, mag = oracle.conv2d_points(codes_in, case.w_codes, case.stride, case.pad, oracle.PAD_CODE_ZERO,
                                       case.a_scale, case.a_offset, case.w_scale, case.w_offset, pts)
    ix = tuple(pts.T)
    assert np.array_equal(acc[ix].astype(np.int64), S), f"{name}: sampled accumulators differ"
    # the hand-over step at the sampled points: one "image" of len(pts) channels-by-1 values, thresholds per point
    sk = skip[ix]
    y_ref, codes_ref, margin = oracle.next_layer(pre.reshape(1, -1, 1), True, sk.reshape(1, -1, 1),
                                                 nlo[pts[:, 1]], nhi[pts[:, 1]])
    y_ref, codes_ref, margin = y_ref.ravel(), codes_ref.ravel(), margin.ravel()
    mag_y = mag + np.abs(sk.astype(np.float64))
    check_fp32(y[ix], y_ref, mag_y, name + " y (sampled)")
    got = oracle.unpack_nhwc(packed, B, N, Ho, Wo)[ix]
    clear = margin > np.maximum(oracle.REL_TOL * np.abs(y_ref), oracle.ABS_TOL * np.maximum(1.0, mag_y))
    assert clear.mean() > 0.999
    assert np.array_equal(got[clear], codes_ref[clear]), f"{name}: sampled codes differ away from the thresholds"
    assert set(np.unique(got).tolist()) == {-1, 0, 1}
    # every packed row is canonical (00 zeros, zero fill past N)
    assert np.array_equal(packed, oracle.pack_nhwc(oracle.unpack_nhwc(packed, B, N, Ho, Wo)))
