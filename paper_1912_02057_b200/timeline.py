"""Role timelines of the tensor-core kernels from in-kernel clock stamps.

    python -m paper_1912_02057_b200.timeline [--workload cfg2|layer2|layer3|layer4|cfg3a|cfg3b|gemm2048|gemm4096|gemm8192] [--batch B] [--io fp32|packed]

Builds librtn_b200_timeline.so (the library with -DRTN_TIMELINE, see csrc/rtn_timeline.cuh), runs the workload's
layer (conv_i8_kernel for cfg2 / layer2, conv_i8s_kernel for cfg3a and cfg3b, gemm_i8_kernel for the square GEMMs) on it a few
times (the last run is reported; earlier ones warm the caches and overlap each launch's
set-up with the previous kernel's tail as in a stream of layers) and prints, for four CTAs spread over the grid,
the microseconds after the CTA's entry at which each role began and ended each tile.  The stamps are SM cycle
counts; microseconds use the SM clock nvidia-smi reports right after the run.  The product library carries no
stamps, and nothing here is timed for a benchmark figure.
"""
import argparse
import ctypes
import os
import subprocess
import sys

HERE = os.path.dirname(os.path.abspath(__file__))

SLOTS = {"conv_i8": {"entry": 0, "set-up done": 1, "filters expanded": 2, "epilogue ready": 3, "end": 4,
                     "roles": {"producer": 8, "converters": 24, "mma": 40, "epilogue": 56}, "tiles": 8},
         "conv_i8s": {"entry": 0, "set-up done": 1, "end": 4,
                      "roles": {"ternarizers": 24, "mma": 40, "epilogue": 56}, "tiles": 8},
         "conv_i8r": {"entry": 0, "filters expanded": 2, "code kernel done": 1, "end": 4,
                      "roles": {"mma": 40, "epilogue": 56}, "tiles": 8},
         "gemm_i8": {"entry": 0, "set-up done": 1, "end": 4, "roles": {"mma": 40, "epilogue": 56}, "tiles": 8}}
# workload -> (instrumented kernel, how to build the case)
WORKLOADS = {"layer3": "conv_i8r", "layer4": "conv_i8r", "cfg2": "conv_i8", "layer2": "conv_i8", "cfg3a": "conv_i8s", "cfg3b": "conv_i8s",
             "gemm4096": "gemm_i8", "gemm2048": "gemm_i8", "gemm8192": "gemm_i8"}


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--workload", default="cfg2", choices=sorted(WORKLOADS))
    ap.add_argument("--batch", type=int, default=None, help="conv workloads: batch size (default: the workload's own)")
    ap.add_argument("--io", default="fp32", choices=["fp32", "packed", "packed_skip"],
                    help="conv workloads: fp32 in and out; packed rows in and out (a block's first layer); or packed rows in, "
                         "fp32 skip connection in, fp32 and packed rows out (a block's second layer)")
    ap.add_argument("--runs", type=int, default=4)
    a = ap.parse_args()
    from . import build
    os.environ["RTN_B200_LIBRARY"] = build.build(timeline=True)
    import numpy as np
    import torch
    from . import binding as rtn, inputs
    tag = WORKLOADS[a.workload]
    dev = lambda t: torch.from_numpy(np.ascontiguousarray(t)).cuda()
    L = rtn.lib()
    reader = getattr(L, f"rtn_timeline_read_{tag}")
    reader.argtypes = [ctypes.c_void_p, ctypes.c_int]
    if a.workload.startswith("gemm"):
        case = inputs.config5(int(a.workload[4:]))
        M, N, K = case.M, case.N, case.K
        w_packed, w_sum = rtn.rtn_pack_weights(dev(case.w_codes))
        a_packed, a_sum = rtn.rtn_ternarize_pack_act(dev(case.a), dev(case.t_lo), dev(case.t_hi))
        par = [dev(v) for v in (case.a_scale, case.a_offset, case.w_scale, case.w_offset)]
        outs = [torch.empty((M, N), dtype=torch.float32, device="cuda") for _ in range(2)]
        torch.cuda.synchronize()
        assert reader(None, 1) == 0
        for j in range(a.runs):
            rtn.rtn_ternary_gemm(a_packed, a_sum, w_packed, w_sum[0], M, N, K, *par, out=outs[j % 2], variant=rtn.VARIANT_I8)
        name = case.name
    else:
        if a.workload == "cfg2":
            case = inputs.config2(batch=a.batch or 32)
        elif a.workload == "cfg3a":
            case = inputs.config3a(0.5, batch=a.batch or 128)
        elif a.workload in ("layer3", "layer4"):      # stride-1 3x3 layers of stages 3 and 4 (split-bank pair at batch 64)
            case = inputs.resnet18_layer("layer3.1.conv1" if a.workload == "layer3" else "layer4.1.conv1", batch=a.batch or 64)
        elif a.workload == "cfg3b":
            case = inputs.config3b(0.5, batch=a.batch or 128)
        else:
            case = inputs.resnet18_layer("layer2.0.conv2", batch=a.batch or 64)
        w_packed, w_sum = rtn.rtn_pack_weights(dev(case.w_codes))
        t_lo, t_hi, w_s, w_o = dev(case.t_lo), dev(case.t_hi), dev(case.w_scale), dev(case.w_offset)
        if a.io != "fp32":
            nhwc = dev(np.ascontiguousarray(case.x.transpose(0, 2, 3, 1)).reshape(-1, case.C))
            xp, _ = rtn.rtn_ternarize_pack_act(nhwc, t_lo, t_hi, want_sum=False)
            rows = [torch.empty((case.B * case.Ho * case.Wo, rtn.rtn_packed_row_bytes(case.N)), dtype=torch.uint8, device="cuda")
                    for _ in range(a.runs)]
            n_lo, n_hi = dev(np.array([0.5], np.float32)), dev(np.array([2.0], np.float32))
            extra = {}
            if a.io == "packed_skip":
                skip = torch.randn((case.B, case.N, case.Ho, case.Wo), dtype=torch.float32, device="cuda")
                ys = [torch.empty_like(skip) for _ in range(a.runs)]
        else:
            xs = [dev(case.x) for _ in range(a.runs)]
            outs = [torch.empty((case.B, case.N, case.Ho, case.Wo), dtype=torch.float32, device="cuda") for _ in range(a.runs)]
        torch.cuda.synchronize()
        assert reader(None, 1) == 0
        for j in range(a.runs):
            if a.io != "fp32":
                if a.io == "packed_skip":
                    extra = dict(skip=skip, out=ys[j])
                rtn.rtn_ternary_conv2d_packed(xp, case.B, case.C, case.H, case.W, w_packed, w_sum, case.N, case.kh, case.kw,
                                              case.stride, case.pad, rtn.PAD_CODE_ZERO, case.a_scale, case.a_offset, w_s, w_o,
                                              relu=True, next_t_lo=n_lo, next_t_hi=n_hi, out_packed=rows[j], **extra)
            else:
                rtn.rtn_ternary_conv2d(xs[j], t_lo, t_hi, w_packed, w_sum, case.N, case.kh, case.kw, case.stride, case.pad,
                                       rtn.PAD_CODE_ZERO, case.a_scale, case.a_offset, w_s, w_o, out=outs[j])
        name = f"{case.name}, io {a.io}"
    torch.cuda.synchronize()
    assert rtn.rtn_last_device_status() == 0
    mhz = float(subprocess.run(["nvidia-smi", "--query-gpu=clocks.sm", "--format=csv,noheader,nounits", "--id=0"],
                               capture_output=True, text=True).stdout.strip().splitlines()[0])
    buf = (ctypes.c_longlong * (4 * 96))()
    assert reader(buf, 0) == 0
    st = np.array(buf, dtype=np.int64).reshape(4, 96)
    lay = SLOTS[tag]
    print(f"{name} ({tag} kernel): stamps of the last of {a.runs} launches, SM clock {mhz:.0f} MHz; microseconds after the CTA's entry")
    for c in range(4):
        t0 = st[c, lay["entry"]]
        if t0 == 0:
            continue
        us = lambda v: (v - t0) / mhz
        head = ", ".join(f"{k} {us(st[c, v]):.2f}" for k, v in lay.items() if isinstance(v, int) and k not in ("entry", "tiles"))
        print(f"CTA {c} of 4 recorded: {head}")
        for role, base in lay["roles"].items():
            cells = []
            for i in range(lay["tiles"]):
                b, e = st[c, base + 2 * i], st[c, base + 2 * i + 1]
                if b == 0 and e == 0:
                    break
                cells.append(f"{us(b):.2f}-{us(e):.2f}")
            print(f"    {role:<10} " + "  ".join(cells))
        cells = []
        for i in range(6):
            v = st[c, 72 + 4 * i: 76 + 4 * i]
            if not v.any():
                break
            cells.append("/".join(f"{us(x):.2f}" if x else "-" for x in v))
        if cells:
            print("    staged rows landed / converted, per channel group: " + "  ".join(cells))
    return 0


if __name__ == "__main__":
    sys.exit(main())
