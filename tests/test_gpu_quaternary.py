"""GPU parity of the paper's 2-bit quaternary comparison workload (rtn_pack_quaternary,
rtn_quaternary_gemm) against the CPU oracle: packed bytes and integer dot products bit-exact."""
import numpy as np
import pytest

import oracle
import paper_1912_02057_b200 as rtn
from paper_1912_02057_b200 import inputs
from helpers import dev

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("M,N,K", [(1, 1, 1), (3, 5, 31), (17, 33, 129), (64, 64, 576), (130, 70, 1000),
                                   (300, 257, 2500), (1000, 96, 64)])
def test_quaternary_gemm_matches_the_plain_sum(M, N, K):
    g = inputs.rng(M + 7 * N + 13 * K)
    x = g.integers(0, 4, (M, K)).astype(np.uint8)
    w = g.integers(0, 4, (N, K)).astype(np.uint8)
    xp, wp = rtn.rtn_pack_quaternary(dev(x)), rtn.rtn_pack_quaternary(dev(w))
    assert np.array_equal(xp.cpu().numpy(), oracle.pack_quaternary_rows(x))
    assert np.array_equal(wp.cpu().numpy(), oracle.pack_quaternary_rows(w))
    out = rtn.rtn_quaternary_gemm(xp, wp, M, N, K).cpu().numpy()
    assert np.array_equal(out.astype(np.int64), oracle.quaternary_gemm(x, w))


def test_quaternary_extremes_and_bad_value():
    K = 4100
    x = np.full((2, K), 3, np.uint8)
    xp = rtn.rtn_pack_quaternary(dev(x))
    out = rtn.rtn_quaternary_gemm(xp, xp, 2, 2, K).cpu().numpy()
    assert (out == 9 * K).all()
    x[1, 77] = 4
    with pytest.raises(rtn.RtnError) as e:
        rtn.rtn_pack_quaternary(dev(x))
    assert e.value.code == 4
    x[1, 77] = 0
    rtn.rtn_pack_quaternary(dev(x))                      # the flag does not stick
