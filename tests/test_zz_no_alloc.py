"""The conv entry point that allocates nothing (collected last: its first call does the per-device
set-up of the static scratch array)."""
import ctypes

import numpy as np
import pytest
import torch

import oracle
import paper_1912_02057_b200 as rtn
from paper_1912_02057_b200 import inputs
from helpers import check_fp32

pytestmark = pytest.mark.gpu

# cudaMemPoolAttr values of the CUDA runtime API
_RESERVED_HIGH, _USED_HIGH = 6, 8


class DefaultPool:
    """High-water marks of the device's default stream-ordered memory pool: the pool cudaMallocAsync draws
    from.  (Free-memory readings miss an allocation that is given back before the next synchronize.)"""

    def __init__(self):
        self.rt = ctypes.CDLL("libcudart.so.12")
        self.pool = ctypes.c_void_p()
        assert self.rt.cudaDeviceGetDefaultMemPool(ctypes.byref(self.pool), torch.cuda.current_device()) == 0

    def reset(self):
        zero = ctypes.c_uint64(0)
        for attr in (_RESERVED_HIGH, _USED_HIGH):
            assert self.rt.cudaMemPoolSetAttribute(self.pool, attr, ctypes.byref(zero)) == 0

    def high(self):
        v = ctypes.c_uint64(0)
        out = []
        for attr in (_RESERVED_HIGH, _USED_HIGH):
            assert self.rt.cudaMemPoolGetAttribute(self.pool, attr, ctypes.byref(v)) == 0
            out.append(int(v.value))
        return tuple(out)


def _dev(a):
    return torch.from_numpy(np.ascontiguousarray(a)).cuda()


def _args(case):
    w_packed, w_sum = rtn.rtn_pack_weights(_dev(case.w_codes))
    return dict(x=_dev(case.x), t_lo=_dev(case.t_lo), t_hi=_dev(case.t_hi), w_packed=w_packed, w_sum=w_sum,
                N=case.N, kh=case.kh, kw=case.kw, stride=case.stride, pad=case.pad,
                a_scale=case.a_scale, a_offset=case.a_offset, w_scale=_dev(case.w_scale),
                w_offset=_dev(case.w_offset))


@pytest.mark.parametrize("pad_mode", [rtn.PAD_CODE_ZERO, rtn.PAD_VALUE_ZERO], ids=["codezero", "valuezero"])
@pytest.mark.parametrize("shape", [(2, 512, 7, 7, 512, 3, 1, 1), (3, 96, 9, 12, 300, 5, 1, 2), (2, 40, 8, 12, 24, 3, 1, 1),
                                   (2, 128, 14, 14, 256, 3, 2, 1)],
                         ids=lambda s: "x".join(map(str, s)))
def test_noalloc_matches_the_allocating_entry_point_twice_in_a_row(shape, pad_mode):
    B, C, H, W, N, k, stride, pad = shape
    case = inputs.conv_case("noalloc_" + "x".join(map(str, shape)), B, C, H, W, N, k, stride, pad,
                            seed=sum(shape), p_zero=0.4, thresholds=(0.3, 1.0), per_channel_thresholds=(C % 3 == 0))
    a = _args(case)
    ref = rtn.rtn_ternary_conv2d(pad_mode=pad_mode, variant=rtn.VARIANT_AUTO, **a)
    acc_ref = torch.empty(ref.shape, dtype=torch.int32, device="cuda")
    rtn.rtn_ternary_conv2d(pad_mode=pad_mode, variant=rtn.VARIANT_AUTO, dbg_acc=acc_ref, **a)
    out1 = torch.full_like(ref, float("nan"))
    out2 = torch.full_like(ref, float("nan"))
    acc2 = torch.empty_like(acc_ref)
    rtn.rtn_ternary_conv2d_noalloc(pad_mode=pad_mode, out=out1, **a)        # a device's first call does the set-up
    out1.fill_(float("nan"))
    torch.cuda.synchronize()
    free_before = torch.cuda.mem_get_info()[0]
    pool = DefaultPool()
    pool.reset()
    rtn.rtn_ternary_conv2d_noalloc(pad_mode=pad_mode, out=out1, **a)
    rtn.rtn_ternary_conv2d_noalloc(pad_mode=pad_mode, out=out2, dbg_acc=acc2, **a)      # reuses the same scratch
    torch.cuda.synchronize()
    assert torch.cuda.mem_get_info()[0] == free_before, "device memory in use changed across the calls"
    assert pool.high() == (0, 0), "the stream-ordered pool was used during the calls"
    assert rtn.rtn_last_device_status() == 0
    # against the oracle directly: integers bit for bit, fp32 within the library's tolerance
    codes = oracle.ternarize(case.x, case.t_lo, case.t_hi, channel_axis=1)
    S, want, mag = oracle.conv2d(codes, case.w_codes, case.stride, case.pad, pad_mode, case.a_scale,
                                 case.a_offset, case.w_scale, case.w_offset)
    assert np.array_equal(acc2.cpu().numpy().astype(np.int64), S), "integer accumulators differ from the oracle"
    check_fp32(out1.cpu().numpy(), want, mag, case.name)
    check_fp32(out2.cpu().numpy(), want, mag, case.name)
    # same arithmetic as the allocating entry point: integers equal, fp32 equal bit for bit
    assert torch.equal(acc2, acc_ref)
    assert torch.equal(out1.view(torch.int32), ref.view(torch.int32))
    assert torch.equal(out2.view(torch.int32), ref.view(torch.int32))


def test_pool_high_water_marks_see_an_allocating_call():
    """The instrument of the test above works: the allocating entry point on the same two-kernel path does
    raise the pool's high-water marks."""
    case = inputs.conv_case("alloc_3x3s2", 2, 128, 14, 14, 256, 3, 2, 1, seed=3, p_zero=0.4, thresholds=(0.3, 1.0))
    assert rtn.rtn_conv_kernel_launches(2, 128, 14, 14, 256, 3, 3, 2, 1) == 2
    a = _args(case)
    rtn.rtn_ternary_conv2d(pad_mode=rtn.PAD_CODE_ZERO, **a)
    torch.cuda.synchronize()
    pool = DefaultPool()
    pool.reset()
    rtn.rtn_ternary_conv2d(pad_mode=rtn.PAD_CODE_ZERO, **a)
    torch.cuda.synchronize()
    assert pool.high()[1] > 0


def test_noalloc_rejects_what_does_not_fit_or_is_not_taken():
    # codes of this layer: 64 * 30 * 30 padded pixels * 512 channels = 29.5 MB > the 16 MiB array
    big = inputs.conv_case("noalloc_big", 64, 512, 28, 28, 16, 3, 1, 1, seed=5, p_zero=0.4, thresholds=(0.3, 1.0))
    a = _args(big)
    out = torch.empty((64, 16, 28, 28), dtype=torch.float32, device="cuda")
    with pytest.raises(rtn.RtnError) as e:
        rtn.rtn_ternary_conv2d_noalloc(pad_mode=rtn.PAD_CODE_ZERO, out=out, **a)
    assert e.value.code == 5          # RTN_ERR_UNSUPPORTED
    strided = inputs.conv_case("noalloc_s3", 2, 64, 12, 12, 32, 3, 3, 1, seed=6, p_zero=0.4, thresholds=(0.3, 1.0))
    a = _args(strided)        # 3x3 with stride 3 reads nine phase images: not taken
    out = torch.empty((2, 32, 4, 4), dtype=torch.float32, device="cuda")
    with pytest.raises(rtn.RtnError) as e:
        rtn.rtn_ternary_conv2d_noalloc(pad_mode=rtn.PAD_CODE_ZERO, out=out, **a)
    assert e.value.code == 5
