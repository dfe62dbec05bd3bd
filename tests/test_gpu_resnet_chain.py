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
