"""Shared by the GPU parity tests: run a case through the C ABI and through the CPU oracle."""
import numpy as np
import torch

import oracle
import paper_1912_02057_b200 as rtn


def dev(a):
    return torch.from_numpy(np.ascontiguousarray(a)).cuda()


# per case: outputs compared, outputs outside the rule WITHOUT the sum-of-terms relaxation, largest such error
STRICT_REPORT = {}


def check_fp32(got, ref, mag, what):
    """fp32 outputs: |err| <= 1e-5 |ref|  or  |err| <= 1e-6 max(1, sum |term_i|).  Also counts, for the report
    at the end of the run, the outputs that miss the unrelaxed rule (1e-5 relative or 1e-6 absolute)."""
    n_miss, worst = oracle.strict_miss(got, ref)
    n, m, w = STRICT_REPORT.get(what, (0, 0, 0.0))
    STRICT_REPORT[what] = (n + int(np.size(ref)), m + n_miss, max(w, worst))
    ok = oracle.within_tolerance(got, ref, mag)
    if not ok.all():
        bad = np.argwhere(~ok)[0]
        i = tuple(bad)
        raise AssertionError(f"{what}: {int((~ok).sum())} outputs out of tolerance; first at {i}: "
                             f"got {got[i]!r} want {ref[i]!r} (sum|terms| {mag[i]!r})")


def gemm_through_abi(case, variant, check_pack=True):
    """Returns (acc int32 [M,N], out fp32 [M,N]) as numpy, after checking the packed operands."""
    M, N, K = case.M, case.N, case.K
    w_packed, w_sum = rtn.rtn_pack_weights(dev(case.w_codes))
    a_packed, a_sum = rtn.rtn_ternarize_pack_act(dev(case.a), dev(case.t_lo), dev(case.t_hi))
    acc = torch.full((M, N), -12345, dtype=torch.int32, device="cuda")
    out = rtn.rtn_ternary_gemm(a_packed, a_sum, w_packed, w_sum[0], M, N, K, dev(case.a_scale),
                               dev(case.a_offset), dev(case.w_scale), dev(case.w_offset),
                               dbg_acc=acc, variant=variant)
    torch.cuda.synchronize()
    assert rtn.rtn_last_device_status() == 0
    if check_pack:
        codes = oracle.ternarize(case.a, case.t_lo, case.t_hi, channel_axis=1)
        assert np.array_equal(a_packed.cpu().numpy(), oracle.pack_rows(codes)), "activation planes"
        assert np.array_equal(w_packed.cpu().numpy(), oracle.pack_rows(case.w_codes)), "weight planes"
        assert np.array_equal(a_sum.cpu().numpy(), codes.astype(np.int64).sum(1)), "S_x"
        assert np.array_equal(w_sum[0].cpu().numpy(), case.w_codes.astype(np.int64).sum(1)), "S_w"
        assert np.array_equal(w_sum[1].cpu().numpy(), w_sum[0].cpu().numpy())
    return acc.cpu().numpy(), out.cpu().numpy()


def gemm_without_dbg(case, variant, unaligned_out=False):
    """The call a user makes: dbg_acc = NULL, which is what lets the kernels take their fast store paths.
    unaligned_out: the output starts 4 bytes past a 16-byte boundary."""
    M, N, K = case.M, case.N, case.K
    w_packed, w_sum = rtn.rtn_pack_weights(dev(case.w_codes))
    a_packed, a_sum = rtn.rtn_ternarize_pack_act(dev(case.a), dev(case.t_lo), dev(case.t_hi))
    out = None
    if unaligned_out:
        out = torch.full((M * N + 4,), float("nan"), dtype=torch.float32, device="cuda")[1:1 + M * N].view(M, N)
        assert out.data_ptr() % 16 == 4
    out = rtn.rtn_ternary_gemm(a_packed, a_sum, w_packed, w_sum[0], M, N, K, dev(case.a_scale),
                               dev(case.a_offset), dev(case.w_scale), dev(case.w_offset), out=out, variant=variant)
    torch.cuda.synchronize()
    assert rtn.rtn_last_device_status() == 0
    return out.cpu().numpy()


def gemm_parity(case, variant):
    acc, out = gemm_through_abi(case, variant)
    codes = oracle.ternarize(case.a, case.t_lo, case.t_hi, channel_axis=1)
    S, ref, mag = oracle.gemm(codes, case.w_codes, case.a_scale, case.a_offset, case.w_scale,
                              case.w_offset)
    assert np.array_equal(acc.astype(np.int64), S), f"{case.name}: integer accumulators differ"
    check_fp32(out, ref, mag, case.name)
    # the production call (no debug output) runs other store paths: against the oracle and bit-equal to the first
    for unaligned in (False, True):
        out2 = gemm_without_dbg(case, variant, unaligned)
        check_fp32(out2, ref, mag, case.name)
        assert np.array_equal(out2.view(np.int32), out.view(np.int32)), f"{case.name}: the call without dbg_acc differs"


def edge_rows(M, n_rows, seed, tile=128):
    """Sampled row indices of an M-row problem: the first and last row of the first three and the last two
    128-row tiles (every tile-edge class of 128- and 256-row tiles), both edges of a few random tiles,
    and random rows up to n_rows in all."""
    g = np.random.default_rng(seed)
    rows = set()
    for t in list(range(min(3, (M + tile - 1) // tile))) + [max(0, (M - 1) // tile - 1), (M - 1) // tile]:
        rows.update({min(M - 1, t * tile), min(M - 1, t * tile + tile - 1)})
    for t in g.integers(0, (M + tile - 1) // tile, 8):
        rows.update({min(M - 1, int(t) * tile), min(M - 1, int(t) * tile + tile - 1)})
    while len(rows) < min(n_rows, M):
        rows.add(int(g.integers(0, M)))
    return np.array(sorted(rows), np.int64)


def gemm_parity_sampled(case, variant, n_rows, seed):
    """Full-size GEMM: sampled rows x ALL columns against the plain oracle (so every column-tile edge is
    covered, and the row sample holds both edges of every row-tile class), integers bit-exact with and fp32
    within tolerance both with the debug output and in the call a user makes (dbg_acc = NULL)."""
    acc, out = gemm_through_abi(case, variant, check_pack=False)
    rows = edge_rows(case.M, n_rows, seed)
    codes = oracle.ternarize(case.a[rows], case.t_lo, case.t_hi, channel_axis=1)
    per_row = case.a_scale.size > 1
    S, ref, mag = oracle.gemm(codes, case.w_codes, case.a_scale[rows] if per_row else case.a_scale,
                              case.a_offset[rows] if per_row else case.a_offset, case.w_scale, case.w_offset)
    assert np.array_equal(acc[rows].astype(np.int64), S), f"{case.name}: sampled accumulators differ"
    check_fp32(out[rows], ref, mag, case.name)
    del acc
    out2 = gemm_without_dbg(case, variant)
    check_fp32(out2[rows], ref, mag, case.name)
    assert np.array_equal(out2.view(np.int32), out.view(np.int32)), f"{case.name}: the call without dbg_acc differs"
    # a property that holds at any size: |S_xw| <= K, and the whole output is finite
    assert np.isfinite(out2).all()
    return rows


def conv_through_abi(case, variant, pad_mode):
    w_packed, w_sum = rtn.rtn_pack_weights(dev(case.w_codes))
    acc = torch.full((case.B, case.N, case.Ho, case.Wo), -12345, dtype=torch.int32, device="cuda")
    out = rtn.rtn_ternary_conv2d(dev(case.x), dev(case.t_lo), dev(case.t_hi), w_packed, w_sum,
                                 case.N, case.kh, case.kw, case.stride, case.pad, pad_mode,
                                 case.a_scale, case.a_offset, dev(case.w_scale), dev(case.w_offset),
                                 dbg_acc=acc, variant=variant)
    torch.cuda.synchronize()
    assert rtn.rtn_last_device_status() == 0
    # the production call (dbg_acc = NULL) takes the kernels' fast epilogues: same bits required
    out2 = rtn.rtn_ternary_conv2d(dev(case.x), dev(case.t_lo), dev(case.t_hi), w_packed, w_sum,
                                  case.N, case.kh, case.kw, case.stride, case.pad, pad_mode,
                                  case.a_scale, case.a_offset, dev(case.w_scale), dev(case.w_offset),
                                  variant=variant)
    torch.cuda.synchronize()
    assert rtn.rtn_last_device_status() == 0
    assert torch.equal(out2.view(torch.int32), out.view(torch.int32)), f"{case.name}: the call without dbg_acc differs"
    return acc.cpu().numpy(), out.cpu().numpy(), w_packed, w_sum


def conv_parity(case, variant, pad_mode=oracle.PAD_CODE_ZERO):
    acc, out, w_packed, w_sum = conv_through_abi(case, variant, pad_mode)
    assert np.array_equal(w_packed.cpu().numpy(), oracle.pack_rows(oracle.conv_weight_rows(case.w_codes)))
    assert np.array_equal(w_sum.cpu().numpy(), oracle.conv_weight_sums(case.w_codes))
    codes = oracle.ternarize(case.x, case.t_lo, case.t_hi, channel_axis=1)
    S, ref, mag = oracle.conv2d(codes, case.w_codes, case.stride, case.pad, pad_mode, case.a_scale,
                                case.a_offset, case.w_scale, case.w_offset)
    assert np.array_equal(acc.astype(np.int64), S), f"{case.name}: integer accumulators differ"
    check_fp32(out, ref, mag, case.name)
    return codes


def conv_parity_sampled(case, variant, pad_mode, n_pts, seed):
    """Full-size case: compare sampled outputs (every tile-edge class included by the random draw
    plus the four image corners and the last channel) with the oracle point by point."""
    acc, out, _, _ = conv_through_abi(case, variant, pad_mode)
    codes = oracle.ternarize(case.x, case.t_lo, case.t_hi, channel_axis=1)
    g = np.random.default_rng(seed)
    pts = np.stack([g.integers(0, case.B, n_pts), g.integers(0, case.N, n_pts),
                    g.integers(0, case.Ho, n_pts), g.integers(0, case.Wo, n_pts)], 1)
    corners = [(b, n, h, v) for b in (0, case.B - 1) for n in (0, case.N - 1)
               for h in (0, case.Ho - 1) for v in (0, case.Wo - 1)]
    pts = np.concatenate([pts, np.array(corners, np.int64)], 0)
    S, ref, mag = oracle.conv2d_points(codes, case.w_codes, case.stride, case.pad, pad_mode,
                                       case.a_scale, case.a_offset, case.w_scale, case.w_offset, pts)
    ix = tuple(pts.T)
    assert np.array_equal(acc[ix].astype(np.int64), S), f"{case.name}: sampled accumulators differ"
    check_fp32(out[ix], ref, mag, case.name)
    return acc, out, codes
