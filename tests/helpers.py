"""Shared by the GPU parity tests: run a case through the C ABI and through the CPU oracle."""
import numpy as np
import torch

import oracle
import paper_1912_02057_b200 as rtn


def dev(a):
    return torch.from_numpy(np.ascontiguousarray(a)).cuda()


def check_fp32(got, ref, mag, what):
    """fp32 outputs: |err| <= 1e-5 |ref|  or  |err| <= 1e-6 max(1, sum |term_i|)."""
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


def gemm_parity(case, variant):
    acc, out = gemm_through_abi(case, variant)
    codes = oracle.ternarize(case.a, case.t_lo, case.t_hi, channel_axis=1)
    S, ref, mag = oracle.gemm(codes, case.w_codes, case.a_scale, case.a_offset, case.w_scale,
                              case.w_offset)
    assert np.array_equal(acc.astype(np.int64), S), f"{case.name}: integer accumulators differ"
    check_fp32(out, ref, mag, case.name)


def conv_through_abi(case, variant, pad_mode):
    w_packed, w_sum = rtn.rtn_pack_weights(dev(case.w_codes))
    acc = torch.full((case.B, case.N, case.Ho, case.Wo), -12345, dtype=torch.int32, device="cuda")
    out = rtn.rtn_ternary_conv2d(dev(case.x), dev(case.t_lo), dev(case.t_hi), w_packed, w_sum,
                                 case.N, case.kh, case.kw, case.stride, case.pad, pad_mode,
                                 case.a_scale, case.a_offset, dev(case.w_scale), dev(case.w_offset),
                                 dbg_acc=acc, variant=variant)
    torch.cuda.synchronize()
    assert rtn.rtn_last_device_status() == 0
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
