#!/usr/bin/env python
"""Benchmark of the ternary hot path: effective ternary TOPS (2*M*N*K / s).

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference] [--workload NAME]

One step = one pass of the whole hot path over one batch of seeded synthetic input: for a conv
workload a single rtn_ternary_conv2d call (ternarize in-kernel -> implicit-GEMM contraction ->
affine epilogue); for a GEMM workload rtn_ternarize_pack_act followed by rtn_ternary_gemm.  Weight
packing is the offline step and happens before the timed region.

Prints ONE JSON line (rank 0).  With N > 1 (torchrun) every rank runs an independent replica on
its own GPU -- the path has no exchange step -- and `value` is the work of all ranks divided by
the slowest rank's time.
"""
import argparse
import json
import os
import subprocess
import sys
import threading
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

from paper_1912_02057_b200 import inputs  # noqa: E402

L2_BYTES = 126 * 1024 * 1024
FALLBACK_HBM_GBS = 6650.0
GRAPH_STEPS = 200

WORKLOADS = {
    "cfg2_conv3x3_c64_56x56_b32": lambda: inputs.config2(batch=32),
    "cfg3a_conv3x3_c256_14x14_b128": lambda: inputs.config3a(0.5, batch=128),
    "cfg3b_conv1x1s2_c128_28x28_b128": lambda: inputs.config3b(0.5, batch=128),
    "cfg1_gemm_64x64x576": inputs.config1,
    # a batch of 16 samples through a wide linear layer (K cut into slices by the bit-plane kernel)
    "linear_m16_n256_k9216": lambda: inputs.gemm_case("linear_m16_n256_k9216", 16, 256, 9216, seed=9, p_zero=0.5,
                                                      thresholds=(0.3, 1.0)),
    "cfg5_gemm_2048": lambda: inputs.config5(2048),
    "cfg5_gemm_4096": lambda: inputs.config5(4096),
    "cfg5_gemm_8192": lambda: inputs.config5(8192),
}
# every ternary conv layer of ResNet-18 at batch 128 (the layer table of the paper's appendix)
for _l in inputs.resnet18_ternary_layers():
    WORKLOADS[f"r18_{_l[0]}_b128"] = (lambda n=_l[0]: inputs.resnet18_layer(n, batch=128))
# the 19 ternary layers chained (packed hand-over between layers), batch 64 of 224x224 images (56x56 after the stem)
WORKLOADS["r18_body_b64"] = lambda: BodyCase(64)
# the paper's comparison: 2-bit quaternary against ternary, both with the bit-plane (AND / popcount) pattern
WORKLOADS["quaternary_vs_ternary_popc_gemm_2048"] = lambda: QuaternaryCase(2048)
DEFAULT_WORKLOAD = "cfg2_conv3x3_c64_56x56_b32"
# --io packed: thresholds of the next layer's ternarizer (per layer), applied to phi(conv output)
NEXT_THRESHOLDS = (0.5, 2.0)


class BodyCase:
    """The ternary body of ResNet-18 as one workload: random-init layers, thresholds by the recipe of
    inputs.resnet18_body_blocks, input = max(0, N(0,1)) standing in for the stem's max-pooled output."""

    def __init__(self, batch):
        self.B = batch
        self.layers = inputs.resnet18_body(seed=4)
        self.blocks = inputs.resnet18_body_blocks(self.layers, sigma_in=1.0)
        self.x = inputs.relu_normal(inputs.rng(44), (batch, 64, 56, 56))


class QuaternaryCase:
    """Square GEMM on 2-bit quaternary values (uniform over {0,1,2,3}) and, for the ratio the paper's
    hardware section argues about, the same-size ternary GEMM on the bit-plane kernel."""

    def __init__(self, n):
        self.n = n
        g = inputs.rng(6)
        self.x = g.integers(0, 4, (n, n)).astype(np.uint8)
        self.w = g.integers(0, 4, (n, n)).astype(np.uint8)
        self.ternary = inputs.gemm_case(f"ternary_{n}", n, n, n, seed=6, p_zero=1.0 / 3.0, act="uniform3",
                                        thresholds=(-0.5, 0.5))


FALLBACK_BF16_TFLOPS = 1590.0
FALLBACK_BF16_TFLOPS_SUSTAINED = 1400.0
INT8_OVER_BF16 = 2.0            # nominal dense ratio 4.5 / 2.25 PFLOP/s
# Traffic counters of the dominant kernel, per launch, from the ncu captures summarised under
# profiles/ (None once the kernel has changed since the capture).
NCU_TRAFFIC_BYTES = {
    # dram__bytes_read.sum + dram__bytes_write.sum of one launch; a kernel's fp32 output is still in L2
    # when the kernel ends, so the write-back of most of it falls outside the capture window
    "cfg2_conv3x3_c64_56x56_b32": 25_799_424 + 11_008,
    "cfg2_conv3x3_c64_56x56_b32/packed": 3_311_872 + 0,
    "cfg3a_conv3x3_c256_14x14_b128": 26_533_888 + 196_096,
    "cfg3b_conv1x1s2_c128_28x28_b128": 51_397_888 + 51_456 + 3_419_648 + 256,    # both kernels of a step
    "cfg5_gemm_4096": 36_865_280 + 20_435_200,
}


def measured_peaks():
    """(HBM GB/s, INT8 dense TOPS for a kernel timed alone, the same under a sustained load, source)."""
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            p = json.load(f)
        return (float(p["hbm_gbs"]), INT8_OVER_BF16 * float(p["bf16_tflops"]),
                INT8_OVER_BF16 * float(p.get("bf16_tflops_sustained", p["bf16_tflops"])),
                "of measured (MEASURED_PEAKS.json; int8 = bf16 x 2 nominal ratio)")
    return (FALLBACK_HBM_GBS, INT8_OVER_BF16 * FALLBACK_BF16_TFLOPS,
            INT8_OVER_BF16 * FALLBACK_BF16_TFLOPS_SUSTAINED, "of fallback (no MEASURED_PEAKS.json)")


def roofline_of(workload, kernel_bytes, kernel_ops, kernel_ms):
    """Roofline object of the dominant kernel: the slower of its HBM time and its tensor time binds."""
    hbm, i8_burst, i8_sust, src = measured_peaks()
    # a kernel that runs for milliseconds sits under the power cap: sustained figure
    i8 = i8_sust if kernel_ms > 0.5 else i8_burst
    t_hbm = kernel_bytes / (hbm * 1e9)
    t_tensor = kernel_ops / (i8 * 1e12)
    traffic = NCU_TRAFFIC_BYTES.get(workload)
    if t_hbm >= t_tensor:
        achieved = kernel_bytes / (kernel_ms * 1e-3) / 1e9
        return {"bound": "hbm", "achieved": achieved, "peak": hbm, "unit": "GB/s", "frac": achieved / hbm,
                "traffic": traffic, "peak_source": src, "bytes_per_launch": int(kernel_bytes),
                "kernel_ms": kernel_ms}
    achieved = kernel_ops / (kernel_ms * 1e-3) / 1e12
    return {"bound": "tensor", "achieved": achieved, "peak": i8, "unit": "TOP/s", "frac": achieved / i8,
            "traffic": traffic, "peak_source": src, "ops_per_launch": kernel_ops, "kernel_ms": kernel_ms}


def time_e2e(torch, step, xs, host_in, host_out, n_sets, n_steps, barrier):
    """Milliseconds per step of: pinned host input -> device, step(j) (the C-ABI calls), result -> pinned host.

    Consecutive steps overlap as a caller with a queue of batches would run them: the upload of step i + 1, the
    kernels of step i and the download of step i - 1 on three streams (the two copy directions use different
    engines), each buffer set guarded by events.  With one buffer set the steps run back to back.  Returns
    (ms per step, whether steps overlapped)."""
    pipelined = n_sets >= 2
    host_outs = [host_out, torch.empty_like(host_out).pin_memory()] if pipelined else [host_out]
    main = torch.cuda.current_stream()
    s_in, s_c, s_out = (torch.cuda.Stream(), torch.cuda.Stream(), torch.cuda.Stream()) if pipelined else (main, main, main)
    ev_in = [torch.cuda.Event() for _ in range(n_sets)]
    ev_c = [torch.cuda.Event() for _ in range(n_sets)]
    ev_out = [torch.cuda.Event() for _ in range(n_sets)]

    def run(n):
        for st in (s_in, s_c, s_out):
            if st is not main:
                st.wait_stream(main)
        for i in range(n):
            j = i % n_sets
            with torch.cuda.stream(s_in):
                s_in.wait_event(ev_c[j])                 # the step that last read xs[j] is done
                xs[j].copy_(host_in, non_blocking=True)
                ev_in[j].record(s_in)
            with torch.cuda.stream(s_c):
                s_c.wait_event(ev_in[j])
                s_c.wait_event(ev_out[j])                # the download that last read this set's output is done
                res = step(j)
                ev_c[j].record(s_c)
            with torch.cuda.stream(s_out):
                s_out.wait_event(ev_c[j])
                host_outs[i % len(host_outs)].copy_(res, non_blocking=True)
                ev_out[j].record(s_out)
        for st in (s_in, s_c, s_out):
            if st is not main:
                main.wait_stream(st)

    run(2)
    barrier()
    e_begin, e_end = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e_begin.record()
    run(n_steps)
    e_end.record()
    barrier()
    return e_begin.elapsed_time(e_end) / n_steps, pipelined


E2E_OVERLAP = "upload, kernels and download of consecutive steps on three streams"


class ClockSampler:
    """Samples SM clock and throttle reasons with nvidia-smi while the timed region runs."""
    Q = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
         "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
         "clocks_event_reasons.sw_power_cap")

    def __init__(self, index):
        self.index, self.proc, self.lines = index, None, []

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", f"--id={self.index}", f"--query-gpu={self.Q}",
                 "--format=csv,noheader,nounits", "-lms", "100"],
                stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=self._read, daemon=True)
            self.thread.start()
        except OSError:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.lines.append(line.strip())

    def stop(self):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        time.sleep(0.15)
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except subprocess.TimeoutExpired:
            self.proc.kill()
        sm, mx, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for ln in self.lines:
            parts = [p.strip() for p in ln.split(",")]
            if len(parts) < 7:
                continue
            try:
                sm.append(float(parts[0]))
                mx.append(float(parts[1]))
            except ValueError:
                continue
            for nm, val in zip(names, parts[3:7]):
                if val.lower().startswith("active"):
                    reasons.add(nm)
        return {"sm_mhz": float(np.median(sm)) if sm else None,
                "sm_max_mhz": float(max(mx)) if mx else None,
                "samples": len(sm), "reasons": sorted(reasons)}


def algorithmic_bytes(case, io="fp32"):
    """Bytes the method must move per step: the fp32 input it touches once, fp32 output once, packed weights once.
    io == "packed": input and output are packed pixel rows (2 bits per value, rows of whole 32-byte blocks)."""
    if isinstance(case, inputs.ConvCase) and io == "packed":
        M, N, K = case.gemm_mnk
        kc = case.kh * case.kw * ((case.C + 31) // 32 * 32)
        rows = {ho * case.stride - case.pad + i for ho in range(case.Ho) for i in range(case.kh)}
        cols = {wo * case.stride - case.pad + j for wo in range(case.Wo) for j in range(case.kw)}
        touched = len([r for r in rows if 0 <= r < case.H]) * len([c for c in cols if 0 <= c < case.W])
        row_bytes = lambda k: (k + 127) // 128 * 32
        return case.B * touched * row_bytes(case.C) + M * row_bytes(N) + N * row_bytes(kc)
    if isinstance(case, inputs.ConvCase):
        M, N, K = case.gemm_mnk
        kc = case.kh * case.kw * ((case.C + 31) // 32 * 32)
        # input pixels some filter tap lands on (a strided 1x1 layer touches a fraction of them)
        rows = {ho * case.stride - case.pad + i for ho in range(case.Ho) for i in range(case.kh)}
        cols = {wo * case.stride - case.pad + j for wo in range(case.Wo) for j in range(case.kw)}
        touched = len([r for r in rows if 0 <= r < case.H]) * len([c for c in cols if 0 <= c < case.W])
        return 4 * case.B * case.C * touched + 4 * M * N + N * ((kc + 127) // 128) * 32
    M, N, K = case.M, case.N, case.K
    packed = lambda r: r * ((K + 127) // 128) * 32
    # ternarize+pack: read fp32, write planes; GEMM: read both packed operands, write fp32
    return case.a.nbytes + packed(M) + packed(M) + packed(N) + 4 * M * N


def ops_of(case):
    M, N, K = case.gemm_mnk if isinstance(case, inputs.ConvCase) else (case.M, case.N, case.K)
    return 2.0 * M * N * K


# ------------------------------------------------------------------------------------------------
# CPU oracle leg (reference arm and cpu_baseline)
# ------------------------------------------------------------------------------------------------
def oracle_sample(case, budget_s=12.0, io="fp32", fill_budget=False):
    """Times the CPU oracle, as it stands, on a bounded sample of the workload.
    Returns (ops per second, seconds, description).  fill_budget: when the whole batch takes a small part
    of the budget, run it several times in a row so that the figure rests on about budget_s of CPU work."""
    import oracle
    if isinstance(case, inputs.ConvCase):
        def run(nb):
            x = case.x[:nb]
            t0 = time.perf_counter()
            codes = oracle.ternarize(x, case.t_lo, case.t_hi, channel_axis=1)
            _, pre, _ = oracle.conv2d(codes, case.w_codes, case.stride, case.pad, oracle.PAD_CODE_ZERO,
                                      case.a_scale, case.a_offset, case.w_scale, case.w_offset)
            if io == "packed":
                _, nxt, _ = oracle.next_layer(pre, True, None, *NEXT_THRESHOLDS)
                oracle.pack_nhwc(nxt)
            dt = time.perf_counter() - t0
            M, N, K = case.gemm_mnk
            return 2.0 * (M // case.B * nb) * N * K, dt
        ops, dt = run(1)
        nb = int(max(1, min(case.B, budget_s / max(dt, 1e-6))))
        if nb > 1:
            ops, dt = run(nb)
        what = f"first {nb} of {case.B} images, all output channels (ternarize + conv2d + epilogue)"
        if fill_budget and nb == case.B and dt < budget_s / 3:
            reps = int(min(40, budget_s / max(dt, 1e-6)))
            tot_ops, tot_dt = 0.0, 0.0
            for _ in range(reps):
                o, d = run(nb)
                tot_ops, tot_dt = tot_ops + o, tot_dt + d
            ops, dt = tot_ops, tot_dt
            what = f"the whole batch of {case.B} images {reps} times in a row, all output channels (ternarize + conv2d + epilogue)"
        return ops / dt, dt, what

    def run(rows):
        a = case.a[:rows]
        t0 = time.perf_counter()
        codes = oracle.ternarize(a, case.t_lo, case.t_hi, channel_axis=1)
        n_ap = case.a_scale.size
        oracle.gemm(codes, case.w_codes, case.a_scale[:rows] if n_ap > 1 else case.a_scale,
                    case.a_offset[:rows] if n_ap > 1 else case.a_offset, case.w_scale, case.w_offset)
        dt = time.perf_counter() - t0
        return 2.0 * rows * case.N * case.K, dt
    rows = min(case.M, 16)
    ops, dt = run(rows)
    rows2 = int(max(rows, min(case.M, rows * budget_s / max(dt, 1e-6))))
    if rows2 > rows:
        ops, dt = run(rows2)
        rows = rows2
    return ops / dt, dt, f"first {rows} of {case.M} rows, all columns (ternarize + gemm + epilogue)"


def run_reference(args, case, name):
    import oracle
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    per_step_budget = max(0.2, min(12.0, 60.0 / max(1, args.steps + args.warmup)))
    sample = ""
    for _ in range(args.warmup):
        _, _, sample = oracle_sample(case, per_step_budget, args.io)
    rates, secs = [], []
    for _ in range(args.steps):
        r, dt, sample = oracle_sample(case, per_step_budget, args.io)
        rates.append(r)
        secs.append(dt)
    value = float(np.mean(rates)) / 1e12
    line = {
        "impl": "reference", "metric": "effective ternary TOPS (2MNK/s)", "value": value,
        "unit": "TOPS", "n_gpus": args.gpus, "steps": args.steps, "warmup": args.warmup,
        "ms_per_step": 1e3 * float(np.mean(secs)), "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "int64", "data": "synthetic",
        "config": {"workload": name, "io": args.io, "note": "CPU oracle on a bounded sample per step"},
        "cpu_baseline": {"value": value, "unit": "TOPS", "cores": oracle.threads(), "kind": "oracle",
                         "sample": sample},
        "e2e": {"value": value, "unit": "TOPS", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line))


# ------------------------------------------------------------------------------------------------
# GPU leg
# ------------------------------------------------------------------------------------------------
def max_over_ranks(values, world, device):
    """Each rank's device-timed milliseconds -> the slowest rank's (the job ends when it does)."""
    if world <= 1:
        return [float(v) for v in values]
    import torch
    import torch.distributed as dist
    t = torch.tensor(values, dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return [float(v) for v in t]


def whole_job_tops(ops_per_replica, world, ms):
    """Replicas only: every rank does the same work, so the job's rate is world * ops / slowest time."""
    return world * ops_per_replica / (ms * 1e-3) / 1e12


def oracle_body_sample(case, budget_s=12.0):
    """The CPU oracle on the body's first residual block (two 3x3 layers with the hand-over between
    them) for as many images as fit the time budget.  Returns (ops per second, seconds, description)."""
    import oracle
    c1, c2 = case.blocks[0]["conv1"], case.blocks[0]["conv2"]
    nxt = case.blocks[1]["conv1"]

    def run(nb):
        s = case.x[:nb]
        t0 = time.perf_counter()
        p = oracle.ternarize(s, c1.t_lo, c1.t_hi)
        _, pre1, _ = oracle.conv2d(p, c1.w_codes, 1, 1, oracle.PAD_CODE_ZERO, c1.a_scale, c1.a_offset, c1.w_scale, c1.w_offset)
        _, q, _ = oracle.next_layer(pre1, True, None, c2.t_lo, c2.t_hi)
        _, pre2, _ = oracle.conv2d(q, c2.w_codes, 1, 1, oracle.PAD_CODE_ZERO, c2.a_scale, c2.a_offset, c2.w_scale, c2.w_offset)
        oracle.next_layer(pre2, True, s, nxt.t_lo, nxt.t_hi)
        dt = time.perf_counter() - t0
        return 2 * 2.0 * nb * 56 * 56 * 64 * 64 * 9, dt
    ops, dt = run(1)
    nb = int(max(1, min(case.B, budget_s / max(dt, 1e-6))))
    if nb > 1:
        ops, dt = run(nb)
    return ops / dt, dt, f"first residual block (layer1.0.conv1, conv2 and their hand-over) on {nb} of {case.B} images"


def run_body(args, case, name):
    """Whole-chain workload: a step = the 19 ternary layers of ResNet-18 on one batch."""
    import torch
    import torch.distributed as dist
    import paper_1912_02057_b200 as rtn
    from paper_1912_02057_b200 import chain

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    torch.cuda.set_device(local)
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))
    n_sets = 2          # two complete sets of activations (input, every intermediate), used in turn
    bodies = [chain.Body(case.blocks, case.B) for _ in range(n_sets)]
    xs = [torch.from_numpy(case.x).cuda() for _ in range(n_sets)]
    host_in = torch.from_numpy(case.x).pin_memory()
    outs = [None] * n_sets

    def step(i):
        j = i % n_sets
        outs[j], _ = bodies[j].forward(xs[j])
        return outs[j]

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    for i in range(max(args.warmup, 3)):
        step(i)
    barrier()
    host_out = torch.empty(outs[0].shape, dtype=torch.float32).pin_memory()
    steps = args.steps
    chunk = min(steps, 20)
    n_full, tail = divmod(steps, chunk)

    class Eager:
        def __init__(self, n):
            self.n = n

        def replay(self):
            for i in range(self.n):
                step(i)

    def capture(n):
        if args.eager:
            return Eager(n)
        g = torch.cuda.CUDAGraph()
        with torch.cuda.graph(g):
            for i in range(n):
                step(i)
        return g
    graph = capture(chunk)
    graph_tail = capture(tail) if tail else None
    graph.replay()
    if graph_tail is not None:
        graph_tail.replay()
    barrier()
    sampler = ClockSampler(local)
    if rank == 0:
        sampler.start()
    t0, t1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    t0.record()
    for _ in range(n_full):
        graph.replay()
    if graph_tail is not None:
        graph_tail.replay()
    t1.record()
    barrier()
    total_ms = t0.elapsed_time(t1)
    if rank == 0 and not args.eager:
        w0 = time.perf_counter()
        while time.perf_counter() - w0 < 1.0:
            graph.replay()
            torch.cuda.synchronize()
    clocks = sampler.stop() if rank == 0 else None
    if clocks is not None:
        clocks["window"] = "timed region plus about 1 s of the same launches, untimed"
    barrier()
    if rtn.rtn_last_device_status() != 0:
        raise RuntimeError("device status after the timed region")
    e2e_ms, pipelined = time_e2e(torch, step, xs, host_in, host_out, n_sets, max(3, min(steps, 20)), barrier)
    total_ms, e2e_ms = max_over_ranks([total_ms, e2e_ms], world, "cuda")
    ms_per_step = total_ms / steps
    ops = bodies[0].ops()
    launches = bodies[0].kernel_launches()
    if rank == 0:
        line = {
            "metric": "effective ternary TOPS (2MNK/s)", "value": whole_job_tops(ops, world, ms_per_step),
            "unit": "TOPS", "n_gpus": world, "steps": steps, "warmup": max(args.warmup, 3),
            "ms_per_step": ms_per_step, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
            "dtype": "int32 accumulate (int8 / 1-bit-plane operands), fp32 epilogue", "data": "synthetic",
            "config": {"workload": name, "io": "packed rows between layers, fp32 residual stream",
                       "images_per_s": world * case.B / (ms_per_step * 1e-3),
                       "layers": 19, "launches_per_step": launches,
                       "l2": f"{n_sets} complete sets of activations used in turn; a layer's output may still be in L2 "
                             "when its consumer reads it (part of the chain, not of the timing method)",
                       "weights": "packed before the timed region (offline step)",
                       "launch": "eager" if args.eager else f"CUDA graph, {chunk} steps per replay",
                       "parallelism": "replicas only" if world > 1 else "1 GPU"},
            "clocks": clocks,
            "e2e": {"value": whole_job_tops(ops, world, e2e_ms), "unit": "TOPS", "ms_per_step": e2e_ms,
                    "h2d_bytes_per_step": int(host_in.numel() * 4), "d2h_bytes_per_step": int(host_out.numel() * 4),
                    "overlap": E2E_OVERLAP if pipelined else "none: one buffer set"},
            "gpu_launches": launches * steps,
            "roofline": roofline_of(name, bodies[0].algorithmic_bytes(), ops, ms_per_step),
        }
        line["roofline"]["note"] = "whole chain (19 layers) against the binding bound of its summed bytes and operations"
        if not args.no_cpu_baseline and world == 1:
            import oracle
            rate, dt, sample = oracle_body_sample(case, 12.0)
            line["cpu_baseline"] = {"value": rate / 1e12, "unit": "TOPS", "cores": oracle.threads(),
                                    "kind": "oracle", "sample": sample, "seconds": dt}
        print(json.dumps(line))
    if world > 1:
        dist.destroy_process_group()


def run_body_reference(args, case, name):
    import oracle
    if int(os.environ.get("RANK", "0")) != 0:
        return
    per_step_budget = max(0.2, min(12.0, 60.0 / max(1, args.steps + args.warmup)))
    sample = ""
    for _ in range(args.warmup):
        _, _, sample = oracle_body_sample(case, per_step_budget)
    rates, secs = [], []
    for _ in range(args.steps):
        r, dt, sample = oracle_body_sample(case, per_step_budget)
        rates.append(r)
        secs.append(dt)
    value = float(np.mean(rates)) / 1e12
    print(json.dumps({
        "impl": "reference", "metric": "effective ternary TOPS (2MNK/s)", "value": value, "unit": "TOPS",
        "n_gpus": args.gpus, "steps": args.steps, "warmup": args.warmup, "ms_per_step": 1e3 * float(np.mean(secs)),
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "int64", "data": "synthetic",
        "config": {"workload": name, "note": "CPU oracle on a bounded sample per step"},
        "cpu_baseline": {"value": value, "unit": "TOPS", "cores": oracle.threads(), "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": "TOPS", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0}))


POPC_LANES_PER_CLK_SM = 16      # popcount issue rate per SM and clock (quarter rate)
SMS = 148


def run_quaternary(args, case, name):
    """rtn_quaternary_gemm against rtn_ternary_gemm's bit-plane variant at the same size."""
    import torch
    import paper_1912_02057_b200 as rtn
    if int(os.environ.get("WORLD_SIZE", "1")) > 1 and int(os.environ.get("RANK", "0")) != 0:
        return
    torch.cuda.set_device(int(os.environ.get("LOCAL_RANK", "0")))
    dev = lambda a: torch.from_numpy(np.ascontiguousarray(a)).cuda()
    n = case.n
    n_sets = 8                      # 8 x (2 x 1 MiB packed + 16 MiB out) > L2
    xq = [rtn.rtn_pack_quaternary(dev(case.x)) for _ in range(n_sets)]
    wq = rtn.rtn_pack_quaternary(dev(case.w))
    outs = [torch.empty((n, n), dtype=torch.int32, device="cuda") for _ in range(n_sets)]
    t = case.ternary
    w_packed, w_sum = rtn.rtn_pack_weights(dev(t.w_codes))
    packs = [rtn.rtn_ternarize_pack_act(dev(t.a), dev(t.t_lo), dev(t.t_hi)) for _ in range(n_sets)]
    a_s, a_o, w_s, w_o = dev(t.a_scale), dev(t.a_offset), dev(t.w_scale), dev(t.w_offset)
    fouts = [torch.empty((n, n), dtype=torch.float32, device="cuda") for _ in range(n_sets)]
    steps = min(args.steps, 200)

    def q_step(i):
        j = i % n_sets
        return rtn.rtn_quaternary_gemm(xq[j], wq, n, n, n, out=outs[j])

    def t_step(i):
        j = i % n_sets
        return rtn.rtn_ternary_gemm(packs[j][0], packs[j][1], w_packed, w_sum[0], n, n, n, a_s, a_o, w_s, w_o,
                                    out=fouts[j], variant=rtn.VARIANT_POPC)

    def timed(fn):
        for i in range(max(args.warmup, 3)):
            fn(i)
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for i in range(steps):
            fn(i)
        e1.record()
        torch.cuda.synchronize()
        return e0.elapsed_time(e1) / steps
    sampler = ClockSampler(int(os.environ.get("LOCAL_RANK", "0")))
    sampler.start()
    t_ms = timed(t_step)
    q_ms = timed(q_step)
    clocks = sampler.stop()
    host_in = torch.from_numpy(case.x).pin_memory()
    dx = torch.empty((n, n), dtype=torch.uint8, device="cuda")
    host_out = torch.empty((n, n), dtype=torch.int32).pin_memory()
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e2e_steps = 5
    e0.record()
    for i in range(e2e_steps):
        dx.copy_(host_in, non_blocking=True)
        host_out.copy_(rtn.rtn_quaternary_gemm(rtn.rtn_pack_quaternary(dx), wq, n, n, n, out=outs[0]), non_blocking=True)
    e1.record()
    torch.cuda.synchronize()
    e2e_ms = e0.elapsed_time(e1) / e2e_steps
    ops = 2.0 * n * n * n
    mhz = clocks.get("sm_mhz") or 1965.0
    # four popcounts per 32 multiply-accumulates at 16 lanes per clock and SM
    peak = 2.0 * 32 * POPC_LANES_PER_CLK_SM * SMS * mhz * 1e6 / 4 / 1e12
    achieved = ops / (q_ms * 1e-3) / 1e12
    line = {
        "metric": "effective 2-bit TOPS (2MNK/s)", "value": achieved, "unit": "TOPS", "n_gpus": 1, "steps": steps,
        "warmup": max(args.warmup, 3), "ms_per_step": q_ms, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "int32 accumulate (1-bit-plane operands)", "data": "synthetic",
        "config": {"workload": name, "ternary_popc_ms": t_ms, "ternary_popc_tops": ops / (t_ms * 1e-3) / 1e12,
                   "quaternary_over_ternary_time": q_ms / t_ms,
                   "note": "same tiling for both; per 32 values and output 4 popcounts (quaternary) against 2 (ternary, Eq. 9)",
                   "l2": f"{n_sets} rotating operand/output sets > L2", "launch": "eager", "parallelism": "1 GPU"},
        "clocks": clocks,
        "e2e": {"value": ops / (e2e_ms * 1e-3) / 1e12, "unit": "TOPS", "ms_per_step": e2e_ms,
                "h2d_bytes_per_step": int(host_in.numel()), "d2h_bytes_per_step": int(host_out.numel() * 4)},
        "gpu_launches": steps,
        "roofline": {"bound": "alu", "achieved": achieved, "peak": peak, "unit": "TOP/s", "frac": achieved / peak,
                     "traffic": None,
                     "peak_source": f"derived: 16 popcount lanes per clock and SM x {SMS} SMs x {mhz:.0f} MHz (median sampled), "
                                    "4 popcounts per 32 multiply-accumulates",
                     "kernel_ms": q_ms},
    }
    if not args.no_cpu_baseline:
        import oracle
        rows = 16
        t0 = time.perf_counter()
        oracle.quaternary_gemm(case.x[:rows], case.w)
        dt = time.perf_counter() - t0
        rows2 = int(max(rows, min(n, rows * 12.0 / max(dt, 1e-6))))
        t0 = time.perf_counter()
        oracle.quaternary_gemm(case.x[:rows2], case.w)
        dt = time.perf_counter() - t0
        line["cpu_baseline"] = {"value": 2.0 * rows2 * n * n / dt / 1e12, "unit": "TOPS", "cores": oracle.threads(),
                                "kind": "oracle", "sample": f"first {rows2} of {n} rows, all columns", "seconds": dt}
    print(json.dumps(line))


def run_ours(args, case, name):
    import torch
    import torch.distributed as dist
    import paper_1912_02057_b200 as rtn

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    torch.cuda.set_device(local)
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))
    dev = lambda a: torch.from_numpy(np.ascontiguousarray(a)).cuda()
    is_conv = isinstance(case, inputs.ConvCase)

    # resident inputs: enough rotating copies that consecutive steps never find their data in L2
    packed_io = is_conv and args.io == "packed"
    step_bytes = algorithmic_bytes(case, args.io if is_conv else "fp32")
    n_sets = max(2, int(np.ceil(2.5 * L2_BYTES / step_bytes)))
    n_sets = min(n_sets, 64)
    w_packed, w_sum = rtn.rtn_pack_weights(dev(case.w_codes))
    w_s, w_o = dev(case.w_scale), dev(case.w_offset)
    t_lo, t_hi = dev(case.t_lo), dev(case.t_hi)
    if packed_io:
        # input: packed pixel rows (what the layer before hands over); output: packed rows for the next
        # layer (phi = ReLU, that layer's thresholds), no fp32 tensor at either end
        nhwc = dev(np.ascontiguousarray(case.x.transpose(0, 2, 3, 1)).reshape(-1, case.C))
        x0, _ = rtn.rtn_ternarize_pack_act(nhwc, t_lo, t_hi, want_sum=False)
        del nhwc
        xs = [x0.clone() for _ in range(n_sets)]
        outs = [torch.empty((case.B * case.Ho * case.Wo, rtn.rtn_packed_row_bytes(case.N)), dtype=torch.uint8,
                            device="cuda") for _ in range(n_sets)]
        n_lo, n_hi = (dev(np.array([v], np.float32)) for v in NEXT_THRESHOLDS)
        variant = 2
        launches_per_step = 2

        def step(i):
            j = i % n_sets
            rtn.rtn_ternary_conv2d_packed(xs[j], case.B, case.C, case.H, case.W, w_packed, w_sum, case.N,
                                          case.kh, case.kw, case.stride, case.pad, rtn.PAD_CODE_ZERO,
                                          case.a_scale, case.a_offset, w_s, w_o, relu=True,
                                          next_t_lo=n_lo, next_t_hi=n_hi, out_packed=outs[j])
            return outs[j]
        host_in = x0.cpu().pin_memory()
    elif is_conv:
        xs = [dev(case.x) for _ in range(n_sets)]
        outs = [torch.empty((case.B, case.N, case.Ho, case.Wo), dtype=torch.float32, device="cuda")
                for _ in range(n_sets)]
        variant = rtn.rtn_choose_conv_variant(case.B, case.C, case.H, case.W, case.N, case.kh,
                                              case.kw, case.stride, case.pad)
        launches_per_step = rtn.rtn_conv_kernel_launches(case.B, case.C, case.H, case.W, case.N, case.kh,
                                                         case.kw, case.stride, case.pad)

        def step(i):
            j = i % n_sets
            rtn.rtn_ternary_conv2d(xs[j], t_lo, t_hi, w_packed, w_sum, case.N, case.kh, case.kw,
                                   case.stride, case.pad, rtn.PAD_CODE_ZERO, case.a_scale,
                                   case.a_offset, w_s, w_o, out=outs[j])
            return outs[j]
        host_in = torch.from_numpy(case.x).pin_memory()
    else:
        M, N, K = case.M, case.N, case.K
        xs = [dev(case.a) for _ in range(n_sets)]
        a_s, a_o = dev(case.a_scale), dev(case.a_offset)
        packs = [torch.empty((M, rtn.rtn_packed_row_bytes(K)), dtype=torch.uint8, device="cuda")
                 for _ in range(n_sets)]
        sums = [torch.empty((M,), dtype=torch.int32, device="cuda") for _ in range(n_sets)]
        outs = [torch.empty((M, N), dtype=torch.float32, device="cuda") for _ in range(n_sets)]
        variant = rtn.rtn_choose_gemm_variant(M, N, K)
        # ternarize_pack + the GEMM's kernels (+ the memset of a sliced K)
        launches_per_step = 1 + rtn.rtn_gemm_kernel_launches(M, N, K) + (1 if rtn.rtn_gemm_k_slices(M, N, K) > 1 else 0)

        def step(i):
            j = i % n_sets
            rtn.rtn_ternarize_pack_act(xs[j], t_lo, t_hi, out=packs[j], out_sum=sums[j])
            rtn.rtn_ternary_gemm(packs[j], sums[j], w_packed, w_sum[0], M, N, K, a_s, a_o, w_s, w_o,
                                 out=outs[j])
            return outs[j]
        host_in = torch.from_numpy(case.a).pin_memory()
    host_out = torch.empty(outs[0].shape, dtype=outs[0].dtype).pin_memory()

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    # ---- device-resident timing.  The steps are captured into a CUDA graph (chunks of up to
    # GRAPH_STEPS launches) so that the host's launch overhead does not starve a ~10 us kernel.
    for i in range(args.warmup):
        step(i)
    barrier()
    chunk = min(args.steps, GRAPH_STEPS)
    n_full, tail = divmod(args.steps, chunk)

    class Eager:
        def __init__(self, n):
            self.n = n

        def replay(self):
            for i in range(self.n):
                step(i)

    def capture(n):
        if args.eager:
            return Eager(n)
        g = torch.cuda.CUDAGraph()
        with torch.cuda.graph(g):
            for i in range(n):
                step(i)
        return g
    graph = capture(chunk)
    graph_tail = capture(tail) if tail else None
    graph.replay()                                     # untimed: uploads the graph
    if graph_tail is not None:
        graph_tail.replay()
    barrier()
    sampler = ClockSampler(local)
    if rank == 0:
        sampler.start()
    t_begin, t_end = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    t_begin.record()
    for _ in range(n_full):
        graph.replay()
    if graph_tail is not None:
        graph_tail.replay()
    t_end.record()
    barrier()
    total_ms = t_begin.elapsed_time(t_end)
    # keep the same kernels running, untimed, until the clock sampler has seen about a second of load
    if rank == 0 and not args.eager:
        t0 = time.perf_counter()
        while time.perf_counter() - t0 < 1.0:
            graph.replay()
            torch.cuda.synchronize()
    clocks = sampler.stop() if rank == 0 else None
    if clocks is not None:
        clocks["window"] = "timed region plus about 1 s of the same launches, untimed"
    barrier()
    status = rtn.rtn_last_device_status()
    if status != 0:
        raise RuntimeError(f"device status {status} after the timed region")

    # ---- GEMM workloads: the dominant kernel (rtn_ternary_gemm) timed alone, rotating operand sets
    gemm_kernel_ms = gemm_kernel_bytes = None
    if not is_conv:
        reps = max(5, min(50, args.steps))

        def gemm_only():
            for i in range(reps):
                j = i % n_sets
                rtn.rtn_ternary_gemm(packs[j], sums[j], w_packed, w_sum[0], M, N, K, a_s, a_o, w_s, w_o, out=outs[j])
        if args.eager:
            replay_gemm = gemm_only
        else:               # through a graph, like the steps: the host's launch and allocator calls stay out of the time
            gg = torch.cuda.CUDAGraph()
            with torch.cuda.graph(gg):
                gemm_only()
            replay_gemm = gg.replay
            replay_gemm()
        k0, k1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        barrier()
        k0.record()
        replay_gemm()
        k1.record()
        barrier()
        gemm_kernel_ms = k0.elapsed_time(k1) / reps
        gemm_kernel_bytes = (M + N) * ((K + 127) // 128) * 32 + 4 * M * N

    # ---- end to end: pinned host input -> device, the C-ABI call(s), result -> pinned host, every step
    e2e_ms, pipelined = time_e2e(torch, step, xs, host_in, host_out, n_sets, max(3, min(args.steps, 40)), barrier)

    total_ms, e2e_ms = max_over_ranks([total_ms, e2e_ms], world, "cuda")
    ms_per_step = total_ms / args.steps
    ops = ops_of(case)
    value = whole_job_tops(ops, world, ms_per_step)
    e2e_value = whole_job_tops(ops, world, e2e_ms)

    if rank == 0:
        if is_conv:
            kernel_ms, kernel_bytes = ms_per_step, step_bytes
        else:
            kernel_ms, kernel_bytes = gemm_kernel_ms, gemm_kernel_bytes
        line = {
            "metric": "effective ternary TOPS (2MNK/s)", "value": value, "unit": "TOPS",
            "n_gpus": world, "steps": args.steps, "warmup": args.warmup, "ms_per_step": ms_per_step,
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
            "dtype": "int32 accumulate (int8 / 1-bit-plane operands), fp32 epilogue",
            "data": "synthetic",
            "config": {"workload": name, "io": args.io if is_conv else "fp32",
                       "variant": {1: "popc", 2: "i8"}[variant],
                       "l2": f"{n_sets} rotating input/output sets ({n_sets * step_bytes >> 20} MiB) > L2",
                       "thresholds": "t_lo = a_offset - 0.5, t_hi = a_offset + 0.5" if is_conv else
                                     "per layer, as the workload names them",
                       "weights": "packed before the timed region (offline step)",
                       "launch": "eager" if args.eager else f"CUDA graph, {chunk} steps per replay",
                       "parallelism": "replicas only" if world > 1 else "1 GPU"},
            "clocks": clocks,
            "e2e": {"value": e2e_value, "unit": "TOPS", "ms_per_step": e2e_ms,
                    "h2d_bytes_per_step": int(host_in.numel() * host_in.element_size()),
                    "d2h_bytes_per_step": int(host_out.numel() * host_out.element_size()),
                    "overlap": E2E_OVERLAP if pipelined else "none: one buffer set"},
            "gpu_launches": launches_per_step * args.steps,
            "roofline": roofline_of(name if not packed_io else name + "/packed", kernel_bytes, ops, kernel_ms),
        }
        if not args.no_cpu_baseline and world == 1:
            import oracle
            rate, dt, sample = oracle_sample(case, 12.0, args.io, fill_budget=True)
            line["cpu_baseline"] = {"value": rate / 1e12, "unit": "TOPS", "cores": oracle.threads(),
                                    "kind": "oracle", "sample": sample, "seconds": dt}
        print(json.dumps(line))
    if world > 1:
        dist.destroy_process_group()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=2000)
    ap.add_argument("--warmup", type=int, default=20)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default=DEFAULT_WORKLOAD, choices=sorted(WORKLOADS))
    ap.add_argument("--io", default="fp32", choices=["fp32", "packed"],
                    help="conv workloads: fp32 NCHW in and out (rtn_ternary_conv2d), or packed pixel rows in and "
                         "out with the hand-over to the next layer fused (rtn_ternary_conv2d_packed)")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--eager", action="store_true",
                    help="launch the timed steps one by one instead of through a CUDA graph (for profilers)")
    args = ap.parse_args()
    if args.warmup < 3:
        args.warmup = 3
    case = WORKLOADS[args.workload]()
    if isinstance(case, QuaternaryCase):
        if args.impl == "reference":
            import oracle
            if int(os.environ.get("RANK", "0")) == 0:
                t0 = time.perf_counter()
                rows = 64
                oracle.quaternary_gemm(case.x[:rows], case.w)
                dt = time.perf_counter() - t0
                v = 2.0 * rows * case.n * case.n / dt / 1e12
                print(json.dumps({"impl": "reference", "metric": "effective 2-bit TOPS (2MNK/s)", "value": v, "unit": "TOPS",
                                  "n_gpus": args.gpus, "steps": args.steps, "warmup": args.warmup, "ms_per_step": 1e3 * dt,
                                  "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "int64",
                                  "data": "synthetic", "config": {"workload": args.workload},
                                  "cpu_baseline": {"value": v, "unit": "TOPS", "cores": oracle.threads(), "kind": "oracle",
                                                   "sample": f"first {rows} of {case.n} rows, all columns"},
                                  "e2e": {"value": v, "unit": "TOPS", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
                                  "gpu_launches": 0}))
        else:
            run_quaternary(args, case, args.workload)
        return
    if isinstance(case, BodyCase):
        if args.steps == 2000:          # the default suits 20 us kernels; a chain step is a few milliseconds
            args.steps = 100
        (run_body_reference if args.impl == "reference" else run_body)(args, case, args.workload)
        return
    if args.impl == "reference":
        run_reference(args, case, args.workload)
    else:
        run_ours(args, case, args.workload)


if __name__ == "__main__":
    main()
