"""The peak probes run and report rates of the right order (they are the denominators of the roofline fractions)."""
import numpy as np
import pytest

pytestmark = pytest.mark.gpu


def test_i8_probe_rate_and_width_sweep():
    import torch
    import paper_1912_02057_b200 as rtn
    cycles, ops = rtn.rtn_probe_peak_i8(2048)
    torch.cuda.synchronize()
    per_clk = ops / float(np.median(cycles.cpu().numpy()))
    assert 8000 < per_clk < 17000, per_clk                  # 16384 = 128 x 256 x 32 x 2 / 128 cycles at best
    cost = {}
    for n_cols in (64, 128, 256):
        cyc, ops_n = rtn.rtn_probe_i8_rate(n_cols, 2048)
        torch.cuda.synchronize()
        assert ops_n == 2048 * 2 * 128 * n_cols * 32
        cost[n_cols] = float(np.median(cyc.cpu().numpy())) / 2048
    # a narrower instruction is never dearer, and never cheaper than a quarter of the widest
    assert cost[64] <= cost[128] * 1.05 <= cost[256] * 1.1025
    assert cost[64] >= cost[256] / 4
    assert rtn.rtn_last_device_status() == 0


def test_popc_probe_rate():
    import torch
    import paper_1912_02057_b200 as rtn
    cycles, ops = rtn.rtn_probe_peak_popc(256)
    torch.cuda.synchronize()
    lanes = ops / float(np.median(cycles.cpu().numpy())) / 32.0
    assert 4.0 < lanes < 17.0, lanes                        # 16 popcount lanes per clock and SM at best


def test_copy_probe_copies():
    import torch
    import paper_1912_02057_b200 as rtn
    src = torch.randint(0, 255, (1 << 20,), dtype=torch.uint8, device="cuda")
    dst = torch.zeros_like(src)
    rtn.rtn_probe_copy(src, dst)
    torch.cuda.synchronize()
    assert torch.equal(src, dst)
