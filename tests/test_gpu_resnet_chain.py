"""The ternary body of ResNet-18 as a chain through the C ABI (packed hand-over between layers)
against the same chain in the CPU oracle, at a reduced image size.  Dyadic parameters make every
epilogue exact in fp32 and in double, so both sides decide the same codes along all 19 layers and
every packed row must match bit for bit."""
import numpy as np
import pytest
import torch

import oracle
from paper_1912_02057_b200 import chain, inputs
import paper_1912_02057_b200 as rtn
from helpers import check_fp32, dev

pytestmark = pytest.mark.gpu


def oracle_chain(blocks, s, pad_mode):
    """The chain of chain.Body.forward, written out with the oracle's functions."""
    def conv(l, codes):
        return oracle.conv2d(codes, l.w_codes, l.stride, l.pad, pad_mode, l.a_scale, l.a_offset, l.w_scale, l.w_offset)
    streams, packed = [], []
    p = oracle.ternarize(s, blocks[0]["conv1"].t_lo, blocks[0]["conv1"].t_hi)
    for i, blk in enumerate(blocks):
        c1, c2, down = blk["conv1"], blk["conv2"], blk["down"]
        _, pre1, _ = conv(c1, p)
        _, q, _ = oracle.next_layer(pre1, True, None, c2.t_lo, c2.t_hi)
        skip = s
        if down is not None:
            _, pre_d, _ = conv(down, oracle.ternarize(s, down.t_lo, down.t_hi))
            skip, _, _ = oracle.next_layer(pre_d, True, None, np.float32(-np.inf), np.float32(np.inf))
            assert np.array_equal(skip, skip.astype(np.float32))          # exact in fp32 (dyadic parameters)
            skip = skip.astype(np.float32)
        nxt = blocks[i + 1]["conv1"] if i + 1 < len(blocks) else c1
        _, pre2, _ = conv(c2, q)
        y, p, margin = oracle.next_layer(pre2, True, skip, nxt.t_lo, nxt.t_hi)
        assert np.array_equal(y, y.astype(np.float32))
        s = y.astype(np.float32)
        streams.append(s)
        packed.append(p)
    return streams, packed


@pytest.mark.parametrize("pad_mode", [oracle.PAD_CODE_ZERO, oracle.PAD_VALUE_ZERO], ids=["code0", "value0"])
def test_resnet18_body_chain_matches_the_oracle_chain(pad_mode):
    B, hin = 3, 28
    layers = inputs.resnet18_body(seed=4, dyadic=True, hin=hin)
    blocks = inputs.resnet18_body_blocks(layers, sigma_in=1.0, dyadic=True)
    g = inputs.rng(77)
    s0 = (np.round(inputs.relu_normal(g, (B, 64, hin, hin)) * 8) / 8).astype(np.float32)
    body = chain.Body(blocks, B, pad_mode)
    out, packed = body.forward(dev(s0))
    torch.cuda.synchronize()
    assert rtn.rtn_last_device_status() == 0
    streams, codes = oracle_chain(blocks, s0, pad_mode)
    for i, (e, k) in enumerate(zip(body.bufs, codes)):
        Bk, Nk, Hk, Wk = k.shape
        got = oracle.unpack_nhwc(e["p_next"].cpu().numpy(), Bk, Nk, Hk, Wk)
        assert np.array_equal(got, k), f"block {i}: packed codes differ"
        assert set(np.unique(k).tolist()) == {-1, 0, 1}, f"block {i}: degenerate codes"
        assert np.array_equal(e["s_next"].cpu().numpy(), streams[i]), f"block {i}: residual stream differs"
    assert np.array_equal(out.cpu().numpy(), streams[-1])


def _points(g, shape, n_pts):
    B, N, H, W = shape
    pts = np.stack([g.integers(0, B, n_pts), g.integers(0, N, n_pts), g.integers(0, H, n_pts),
                    g.integers(0, W, n_pts)], 1)
    corners = [(b, n, h, v) for b in (0, B - 1) for n in (0, N - 1) for h in (0, H - 1) for v in (0, W - 1)]
    return np.concatenate([pts, np.array(corners, np.int64)], 0)


def _check_layer_at_points(l, codes_in, pts, acc, skip, y_got, codes_got, t_next, what):
    """One layer of the chain at sampled output points: the oracle gets the layer's input codes (the GPU's own
    packed input, decoded) and must reproduce the integers bit for bit, the fp32 stream within tolerance and
    the packed codes wherever y is clear of the next layer's thresholds."""
    S, pre, mag = oracle.conv2d_points(codes_in, l.w_codes, l.stride, l.pad, oracle.PAD_CODE_ZERO, l.a_scale,
                                       l.a_offset, l.w_scale, l.w_offset, pts)
    ix = tuple(pts.T)
    assert np.array_equal(acc[ix].astype(np.int64), S), f"{what}: integer accumulators differ"
    sk = None if skip is None else skip[ix].reshape(-1, 1)
    lo, hi = (np.float32(-np.inf), np.float32(np.inf)) if t_next is None else t_next
    y_ref, codes_ref, margin = oracle.next_layer(pre.reshape(-1, 1), True, sk, lo, hi)
    y_ref, codes_ref, margin = y_ref.ravel(), codes_ref.ravel(), margin.ravel()
    mag_y = mag if skip is None else mag + np.abs(skip[ix].astype(np.float64))
    if y_got is not None:
        check_fp32(y_got[ix], y_ref, mag_y, what)
    if codes_got is not None:
        got = codes_got[ix]
        clear = margin > np.maximum(oracle.REL_TOL * np.abs(y_ref), oracle.ABS_TOL * np.maximum(1.0, mag_y))
        assert clear.mean() > 0.99, what
        assert np.array_equal(got[clear], codes_ref[clear]), f"{what}: codes differ away from the thresholds"
        assert (np.abs(got.astype(np.int32) - codes_ref.astype(np.int32))[~clear] <= 1).all(), what


def test_resnet18_body_chain_at_the_benchmark_size_sampled():
    """The configuration the benchmark times (batch 64, 56x56 input, U(0.5,1.5) / U(-0.1,0.1) parameters, the
    kernel each layer takes at that batch): the production pass (no debug output) must equal a pass with
    debug accumulators bit for bit, and every layer is compared with the oracle at sampled points, the
    oracle reading the layer's input as the GPU wrote it."""
    B = 64
    layers = inputs.resnet18_body(seed=4)
    blocks = inputs.resnet18_body_blocks(layers, sigma_in=1.0)
    s0 = inputs.relu_normal(inputs.rng(44), (B, 64, 56, 56))
    body = chain.Body(blocks, B)
    x = dev(s0)
    out, _ = body.forward(x)
    torch.cuda.synchronize()
    keep = [{k: (None if v is None else v.clone()) for k, v in e.items()} for e in body.bufs]
    dbg = {}
    for l in body.layers():
        ho = rtn.rtn_conv_out_dim(l.hin, l.k, l.stride, l.pad)
        dbg[l.name] = torch.full((B, l.cout, ho, ho), -12345, dtype=torch.int32, device="cuda")
    body.forward(x, dbg=dbg)
    torch.cuda.synchronize()
    assert rtn.rtn_last_device_status() == 0
    for i, (e, k) in enumerate(zip(body.bufs, keep)):
        for name in ("q", "s_next", "p_next", "skip"):
            if e[name] is not None:
                assert torch.equal(e[name].view(torch.uint8), k[name].view(torch.uint8)), f"block {i} {name}: passes differ"
    g = np.random.default_rng(5)
    s, p_codes = s0, None
    for i, (blk, e) in enumerate(zip(blocks, body.bufs)):
        c1, c2, down = blk["conv1"], blk["conv2"], blk["down"]
        nxt = blocks[i + 1]["conv1"] if i + 1 < len(blocks) else c1
        ho = rtn.rtn_conv_out_dim(c1.hin, c1.k, c1.stride, c1.pad)
        in1 = p_codes if p_codes is not None else oracle.ternarize(s, c1.t_lo, c1.t_hi)
        q = oracle.unpack_nhwc(e["q"].cpu().numpy(), B, c1.cout, ho, ho)
        pts = _points(g, (B, c1.cout, ho, ho), 3000)
        _check_layer_at_points(c1, in1, pts, dbg[c1.name].cpu().numpy(), None, None, q, (c2.t_lo, c2.t_hi), c1.name)
        skip = s
        if down is not None:
            skip = e["skip"].cpu().numpy()
            _check_layer_at_points(down, oracle.ternarize(s, down.t_lo, down.t_hi), pts, dbg[down.name].cpu().numpy(),
                                   None, skip, None, None, down.name)
        s_next = e["s_next"].cpu().numpy()
        p_next = oracle.unpack_nhwc(e["p_next"].cpu().numpy(), B, c2.cout, ho, ho)
        _check_layer_at_points(c2, q, pts, dbg[c2.name].cpu().numpy(), skip, s_next, p_next, (nxt.t_lo, nxt.t_hi), c2.name)
        for codes in (q, p_next):
            frac = [(codes == v).mean() for v in (-1, 0, 1)]
            assert min(frac) > 0.02, f"block {i}: degenerate codes {frac}"
        s, p_codes = s_next, p_next
    assert np.array_equal(out.cpu().numpy(), s)
