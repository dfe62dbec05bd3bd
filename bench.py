#!/usr/bin/env python
"""Benchmark of the ternary hot path: effective ternary TOPS (2*M*N*K / s), fraction of the binding roofline,
ResNet-18 images/s.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference]
                    [--workload NAME] [--variant auto|popc|i8] [--io fp32|packed]

Without --workload the run covers every configuration of the workload list (SUITE) and prints ONE JSON line:
the headline configuration's numbers at the top level and one entry per configuration under `per_config`
(time, TOPS, roofline, end-to-end), plus the measured peaks of the int8 tensor pipe and of the AND / XOR /
popcount pattern (`peaks`).  With --workload the line describes that configuration alone.

One step = one pass of the whole hot path over one batch of seeded synthetic input: for a conv workload a
single rtn_ternary_conv2d call (ternarize in-kernel -> implicit-GEMM contraction -> affine epilogue); for a
GEMM workload rtn_ternarize_pack_act followed by rtn_ternary_gemm; for ResNet-18 the fp32 stem, the 19 ternary
layers with their fused hand-over, and the fp32 classifier.  Weight packing is the offline step and happens
before the timed region.

Timing: whatever --steps says, a timed region is a whole number of K-step repeats long enough to span about
50 ms, five such regions are timed with CUDA events and the median is reported.

With N > 1 (torchrun) every rank runs an independent replica on its own GPU -- the path has no exchange step --
and a configuration's time is the slowest rank's.
"""
import argparse
import hashlib
import json
import math
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
FALLBACK_BF16_TFLOPS = 1590.0
FALLBACK_BF16_TFLOPS_SUSTAINED = 1400.0
INT8_OVER_BF16 = 2.0            # nominal dense ratio 4.5 / 2.25 PFLOP/s
GRAPH_STEPS = 200               # steps per captured graph at most
REGION_MS = 50.0                # a timed region spans at least this long
REGIONS = 5                     # regions timed; the median is reported
NEXT_THRESHOLDS = (0.5, 2.0)    # --io packed: thresholds of the next layer's ternarizer (per layer)
METRIC = "effective ternary TOPS (2MNK/s)"
DTYPE = "int32 accumulate (int8 / 1-bit-plane operands), fp32 epilogue"


class BodyCase:
    """The ternary body of ResNet-18 as one workload: random-init layers, thresholds by the recipe of
    inputs.resnet18_body_blocks, input = max(0, N(0,1)) standing in for the stem's max-pooled output."""

    def __init__(self, batch):
        self.B = batch
        self.layers = inputs.resnet18_body(seed=4)
        self.blocks = inputs.resnet18_body_blocks(self.layers, sigma_in=1.0)
        self.x = inputs.relu_normal(inputs.rng(44), (batch, 64, 56, 56))


class FullCase:
    """The full ResNet-18 topology at 224x224: fp32 stem (7x7 stride-2 conv, BN with its initial statistics,
    ReLU, 3x3 stride-2 max-pool) and fp32 classifier (global average pool, 512 -> 1000 linear layer) in torch
    around the 19 ternary layers; images ~ N(0,1), random-init weights.  The thresholds of the ternary layers
    follow the rule of inputs.resnet18_body_blocks with sigma_in calibrated on the stem's real output: the
    standard deviation of the stem's max-pooled output on this batch divided by 0.584, the ratio between the
    standard deviation of max(0, N(0, s)) and s (the stand-in input max(0, N(0,1)) gives 1.0 by the same rule)."""

    RELU_STD_RATIO = 0.584

    def __init__(self, batch):
        self.B = batch
        self.images = inputs.rng(45).standard_normal((batch, 3, 224, 224), dtype=np.float32)
        self.ends = inputs.resnet18_fp32_ends(seed=46)
        self.layers = inputs.resnet18_body(seed=4)
        self.blocks = None          # set by calibrate()
        self.sigma_in = None

    def stem(self, torch, images, w, out=None):
        """fp32 stem on whatever device the tensors live on; NCHW result (written into `out` when given).
        Max-pool, ReLU and the BN scale are applied in that order: all three are monotone (the scale is positive and
        rounding preserves order), so the result is bit for bit that of scale -> ReLU -> max-pool on the same
        convolution output, and the two elementwise passes run on a quarter of the values."""
        F = torch.nn.functional
        y = torch.relu_(F.max_pool2d(F.conv2d(images, w, stride=2, padding=3), 3, stride=2, padding=1))
        scale = 1.0 / math.sqrt(1.0 + 1e-5)             # BN with its initial statistics (mean 0, variance 1)
        if out is None:
            out = torch.empty(y.shape, dtype=y.dtype, device=y.device)
        return torch.mul(y, scale, out=out)

    def calibrate(self, torch, stem_out):
        self.sigma_in = float(stem_out.float().std().item()) / self.RELU_STD_RATIO
        self.blocks = inputs.resnet18_body_blocks(self.layers, sigma_in=self.sigma_in)


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


WORKLOADS = {
    "cfg1_gemm_64x64x576": inputs.config1,
    "cfg2_conv3x3_c64_56x56_b32": lambda: inputs.config2(batch=32),
    "cfg3a_conv3x3_c256_14x14_b128": lambda: inputs.config3a(0.5, batch=128),
    "cfg3b_conv1x1s2_c128_28x28_b128": lambda: inputs.config3b(0.5, batch=128),
    # a batch of 16 samples through a wide linear layer (K cut into slices by the bit-plane kernel)
    "linear_m16_n256_k9216": lambda: inputs.gemm_case("linear_m16_n256_k9216", 16, 256, 9216, seed=9, p_zero=0.5,
                                                      thresholds=(0.3, 1.0)),
    # the 19 ternary layers chained (packed hand-over between layers), batch 64 of 224x224 images (56x56 after the stem)
    "r18_body_b64": lambda: BodyCase(64),
    # the full topology: fp32 stem and classifier around the chain
    "r18_full_b64": lambda: FullCase(64),
    # the paper's comparison: 2-bit quaternary against ternary, both with the bit-plane (AND / popcount) pattern
    "quaternary_vs_ternary_popc_gemm_2048": lambda: QuaternaryCase(2048),
}
for _z in (0.2, 0.8):           # the weight-zero fraction sweep (the names without a suffix are the 0.5 case)
    WORKLOADS[f"cfg3a_conv3x3_c256_14x14_b128_z{_z}"] = (lambda z=_z: inputs.config3a(z, batch=128))
    WORKLOADS[f"cfg3b_conv1x1s2_c128_28x28_b128_z{_z}"] = (lambda z=_z: inputs.config3b(z, batch=128))
for _n in (2048, 4096, 8192, 16384):
    WORKLOADS[f"cfg5_gemm_{_n}"] = (lambda n=_n: inputs.config5(n))
# every ternary conv layer of ResNet-18 at batch 128 (the layer table of the paper's appendix)
for _l in inputs.resnet18_ternary_layers():
    WORKLOADS[f"r18_{_l[0]}_b128"] = (lambda n=_l[0]: inputs.resnet18_layer(n, batch=128))

# The default run: every configuration of the workload list, the largest one as the headline.
SUITE = [
    "cfg1_gemm_64x64x576",
    "cfg2_conv3x3_c64_56x56_b32",
    "cfg3a_conv3x3_c256_14x14_b128_z0.2", "cfg3a_conv3x3_c256_14x14_b128", "cfg3a_conv3x3_c256_14x14_b128_z0.8",
    "cfg3b_conv1x1s2_c128_28x28_b128_z0.2", "cfg3b_conv1x1s2_c128_28x28_b128", "cfg3b_conv1x1s2_c128_28x28_b128_z0.8",
    "r18_full_b64",
    "cfg5_gemm_2048", "cfg5_gemm_4096", "cfg5_gemm_8192", "cfg5_gemm_16384",
]
HEADLINE = "cfg5_gemm_16384"


# ------------------------------------------------------------------------------------------------
# peaks, roofline, traffic
# ------------------------------------------------------------------------------------------------
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


TRAFFIC_FILE = os.path.join(ROOT, "profiles", "traffic.json")


def file_sha256(path):
    h = hashlib.sha256()
    with open(path, "rb") as f:
        h.update(f.read())
    return h.hexdigest()


def traffic_of(key):
    """DRAM bytes per launch of the workload's dominant kernel from the tracked ncu record, or None when there
    is no record or a source file of the kernel has changed since the counters were taken."""
    import re
    key = re.sub(r"_z0\.\d+", "", key)          # the weight-zero fraction does not change what a kernel moves
    try:
        with open(TRAFFIC_FILE) as f:
            rec = json.load(f).get(key)
    except (OSError, ValueError):
        return None
    if not rec:
        return None
    for rel, sha in rec.get("sources", {}).items():
        path = os.path.join(ROOT, rel)
        if not os.path.exists(path) or file_sha256(path) != sha:
            return None
    return int(rec["bytes_per_launch"])


def roofline_of(key, kernel_bytes, kernel_ops, kernel_ms, variant="i8", peaks=None):
    """Roofline object of the dominant kernel.  Tensor-core variant: the slower of its HBM time and its int8
    tensor time binds.  Bit-plane variant: HBM against the AND / XOR / popcount issue rate (bound "alu")."""
    hbm, i8_burst, i8_sust, src = measured_peaks()
    # a kernel that runs for milliseconds sits under the power cap: sustained figure
    i8 = i8_sust if kernel_ms > 0.5 else i8_burst
    t_hbm = kernel_bytes / (hbm * 1e9)
    common = {"traffic": traffic_of(key), "kernel_ms": kernel_ms}
    if variant == "popc":
        alu = (peaks or {}).get("popc")
        if alu is None:
            return {"bound": "alu", "achieved": kernel_ops / (kernel_ms * 1e-3) / 1e12, "peak": None, "unit": "TOP/s",
                    "frac": None, "peak_source": "the popcount probe did not run", **common}
        t_alu = kernel_ops / (alu["tops"] * 1e12)
        if t_alu >= t_hbm:
            achieved = kernel_ops / (kernel_ms * 1e-3) / 1e12
            return {"bound": "alu", "achieved": achieved, "peak": alu["tops"], "unit": "TOP/s",
                    "frac": achieved / alu["tops"], "peak_source": alu["source"], "ops_per_launch": kernel_ops, **common}
    else:
        t_tensor = kernel_ops / (i8 * 1e12)
        if t_tensor > t_hbm:
            achieved = kernel_ops / (kernel_ms * 1e-3) / 1e12
            r = {"bound": "tensor", "achieved": achieved, "peak": i8, "unit": "TOP/s", "frac": achieved / i8,
                 "peak_source": src, "ops_per_launch": kernel_ops, **common}
            probe = (peaks or {}).get("i8")
            if probe is not None:
                r["peak_probe"] = probe["tops"]
                r["frac_of_probe"] = achieved / probe["tops"]
                r["peak_probe_source"] = probe["source"]
            return r
    achieved = kernel_bytes / (kernel_ms * 1e-3) / 1e9
    r = {"bound": "hbm", "achieved": achieved, "peak": hbm, "unit": "GB/s", "frac": achieved / hbm,
         "peak_source": src, "bytes_per_launch": int(kernel_bytes), **common}
    copy = (peaks or {}).get("copy")
    if copy is not None and 0.5 < kernel_bytes / (copy["bytes_read"] + copy["bytes_written"]) < 2.0:
        # a plain copy of about this many bytes, same launch method: the fraction of the HBM peak it reaches
        r["copy_probe_frac"] = copy["frac_of_hbm_peak"]
        r["frac_of_copy_probe"] = achieved / copy["gbs"]
    return r


def algorithmic_bytes(case, io="fp32"):
    """Bytes the method must move per step: the fp32 input it touches once, fp32 output once, packed weights once.
    io == "packed": input and output are packed pixel rows (2 bits per value, rows of whole 32-byte blocks)."""
    if isinstance(case, inputs.ConvCase):
        M, N, K = case.gemm_mnk
        kc = case.kh * case.kw * ((case.C + 31) // 32 * 32)
        # input pixels some filter tap lands on (a strided 1x1 layer touches a fraction of them)
        rows = {ho * case.stride - case.pad + i for ho in range(case.Ho) for i in range(case.kh)}
        cols = {wo * case.stride - case.pad + j for wo in range(case.Wo) for j in range(case.kw)}
        touched = len([r for r in rows if 0 <= r < case.H]) * len([c for c in cols if 0 <= c < case.W])
        row_bytes = lambda k: (k + 127) // 128 * 32
        if io == "packed":
            return case.B * touched * row_bytes(case.C) + M * row_bytes(N) + N * row_bytes(kc)
        return 4 * case.B * case.C * touched + 4 * M * N + N * row_bytes(kc)
    M, N, K = case.M, case.N, case.K
    packed = lambda r: r * ((K + 127) // 128) * 32
    # ternarize+pack: read fp32, write planes; GEMM: read both packed operands, write fp32
    return case.a.nbytes + packed(M) + packed(M) + packed(N) + 4 * M * N


def ops_of(case):
    M, N, K = case.gemm_mnk if isinstance(case, inputs.ConvCase) else (case.M, case.N, case.K)
    return 2.0 * M * N * K


# ------------------------------------------------------------------------------------------------
# timing helpers
# ------------------------------------------------------------------------------------------------
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
                 "--format=csv,noheader,nounits", "-lms", "50"],
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
        time.sleep(0.1)
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


class Ctx:
    """Per-process state: ranks, the barrier, the max over ranks."""

    def __init__(self, args):
        import torch
        self.torch = torch
        self.args = args
        self.world = int(os.environ.get("WORLD_SIZE", "1"))
        self.rank = int(os.environ.get("RANK", "0"))
        self.local = int(os.environ.get("LOCAL_RANK", "0"))
        torch.cuda.set_device(self.local)
        torch.backends.cudnn.allow_tf32 = False          # the fp32 ends of ResNet-18 stay fp32
        torch.backends.cuda.matmul.allow_tf32 = False
        self.dist = None
        if self.world > 1:
            import torch.distributed as dist
            dist.init_process_group("nccl", device_id=torch.device("cuda", self.local))
            self.dist = dist
        self.launches = 0           # kernels of the library launched inside timed regions

    def barrier(self):
        if self.dist is not None:
            self.dist.barrier()
        self.torch.cuda.synchronize()

    def max_over_ranks(self, values):
        return max_over_ranks(values, self.world, "cuda")

    def close(self):
        if self.dist is not None:
            self.dist.destroy_process_group()

    def dev(self, a):
        return self.torch.from_numpy(np.ascontiguousarray(a)).cuda()


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


def time_steps(ctx, step, k_steps, warmup, launches_per_step, sample_clocks=True):
    """Device time per step of `step(i)`.  K steps are captured in CUDA graphs (chunks of up to GRAPH_STEPS, so
    that the host's launch overhead does not starve a short kernel; with --eager they are launched one by one);
    a timed region repeats the K steps until it spans about REGION_MS; REGIONS regions are timed with CUDA
    events on the launching stream and the median (of the max over ranks) is reported.
    Returns (ms per step, timing dict, clocks dict or None)."""
    torch, args = ctx.torch, ctx.args
    for i in range(max(3, warmup)):
        step(i)
    ctx.barrier()
    chunk = min(k_steps, GRAPH_STEPS)
    n_full, tail = divmod(k_steps, chunk)

    def capture(n):
        if args.eager:
            return lambda: [step(i) for i in range(n)]
        g = torch.cuda.CUDAGraph()
        with torch.cuda.graph(g):
            for i in range(n):
                step(i)
        return g.replay
    replay = capture(chunk)
    replay_tail = capture(tail) if tail else None

    def k_steps_once():
        for _ in range(n_full):
            replay()
        if replay_tail is not None:
            replay_tail()
    k_steps_once()                                      # untimed: uploads the graphs
    ctx.barrier()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    k_steps_once()
    e1.record()
    ctx.barrier()
    once_ms = ctx.max_over_ranks([e0.elapsed_time(e1)])[0]
    repeats = max(1, int(math.ceil(REGION_MS / max(once_ms, 1e-3))))
    sampler = ClockSampler(ctx.local) if (sample_clocks and ctx.rank == 0) else None
    if sampler is not None:
        sampler.start()
    region_ms = []
    for _ in range(REGIONS):
        ctx.barrier()
        e0.record()
        for _ in range(repeats):
            k_steps_once()
        e1.record()
        ctx.barrier()
        region_ms.append(e0.elapsed_time(e1))
    ctx.launches += REGIONS * repeats * k_steps * launches_per_step
    region_ms = ctx.max_over_ranks(region_ms)
    clocks = None
    if sampler is not None:
        # keep the same launches running, untimed, until the sampler has seen about half a second of load
        t0 = time.perf_counter()
        while time.perf_counter() - t0 < 0.5:
            k_steps_once()
            torch.cuda.synchronize()
        clocks = sampler.stop()
        clocks["window"] = "the timed regions plus about 0.5 s of the same launches, untimed"
    ctx.barrier()
    per_step = sorted(r / (repeats * k_steps) for r in region_ms)
    timing = {"regions": REGIONS, "steps_per_region": repeats * k_steps, "statistic": "median over regions",
              "region_ms": [round(r, 4) for r in region_ms],
              "launch": "eager" if args.eager else f"CUDA graph, {chunk} steps per replay"}
    return per_step[len(per_step) // 2], timing, clocks


E2E_OVERLAP = "upload, kernels and download of consecutive steps on three streams"


def time_e2e(ctx, step, xs, host_in, host_out, n_sets, n_steps):
    """Milliseconds per step of: pinned host input -> device, step(j) (the C-ABI calls), result -> pinned host.

    Consecutive steps overlap as a caller with a queue of batches would run them: the upload of step i + 1, the
    kernels of step i and the download of step i - 1 on three streams (the two copy directions use different
    engines), each buffer set guarded by events.  With one buffer set the steps run back to back.  Returns
    (ms per step, whether steps overlapped)."""
    torch = ctx.torch
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
    ctx.barrier()
    e_begin, e_end = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e_begin.record()
    run(n_steps)
    e_end.record()
    ctx.barrier()
    ms = ctx.max_over_ranks([e_begin.elapsed_time(e_end) / n_steps])[0]
    return ms, pipelined


def e2e_steps_for(bytes_per_step, k_steps):
    """Steps of the end-to-end loop: as many as asked for, within about a second of PCIe time."""
    est_ms = max(0.05, bytes_per_step / 20e9 * 1e3)
    return int(max(3, min(k_steps, 40, 1000.0 / est_ms)))


def e2e_dict(ctx, ops, e2e_ms, pipelined, host_in, host_out):
    return {"value": whole_job_tops(ops, ctx.world, e2e_ms), "unit": "TOPS", "ms_per_step": e2e_ms,
            "h2d_bytes_per_step": int(host_in.numel() * host_in.element_size()),
            "d2h_bytes_per_step": int(host_out.numel() * host_out.element_size()),
            "overlap": E2E_OVERLAP if pipelined else "none: one buffer set"}


# ------------------------------------------------------------------------------------------------
# peak probes
# ------------------------------------------------------------------------------------------------
def run_peaks(ctx):
    """The int8 tensor-pipe rate and the AND / XOR / popcount issue rate, measured by the library's probes:
    operations per clock and SM from the in-kernel cycle counts, TOPS from the event-timed launch."""
    import paper_1912_02057_b200 as rtn
    torch = ctx.torch
    out = {}
    for name, fn, work in (("i8", rtn.rtn_probe_peak_i8, 16384), ("popc", rtn.rtn_probe_peak_popc, 1024)):
        fn(work // 8)
        torch.cuda.synchronize()
        sampler = ClockSampler(ctx.local)
        sampler.start()
        best_ms, cycles, ops = None, None, None
        t0 = time.perf_counter()
        while best_ms is None or time.perf_counter() - t0 < 0.4:
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record()
            cyc, ops = fn(work)
            e1.record()
            torch.cuda.synchronize()
            ms = e0.elapsed_time(e1)
            if best_ms is None or ms < best_ms:
                best_ms, cycles = ms, cyc.cpu().numpy()
        clocks = sampler.stop()
        ctas = int(cycles.size)
        per_clk_sm = ops / float(np.median(cycles))
        entry = {"ops_per_clk_sm": per_clk_sm, "ctas": ctas, "kernel_ms": best_ms,
                 "tops": ctas * ops / (best_ms * 1e-3) / 1e12, "sm_mhz": clocks.get("sm_mhz"),
                 "reasons": clocks.get("reasons")}
        if name == "i8":
            entry["source"] = ("measured: rtn_probe_peak_i8, tcgen05.mma kind::i8 M=128 N=256 K=32 back to back on "
                               "shared-memory operands, one CTA per SM, event-timed")
        else:
            entry["popc_lanes_per_clk_sm"] = per_clk_sm / 32.0       # 2 popcounts per 32 pairs = 64 operations
            entry["source"] = ("measured: rtn_probe_peak_popc, AND + XOR-AND + 2 popcounts + 2 adds per 32 code pairs "
                               "on registers, 1024 threads per SM, event-timed")
        out[name] = entry
    # what one tensor-core instruction of a narrower accumulator costs with nothing else in the way (cycles per
    # instruction from the in-kernel counts): the floor under the conv kernels' 64- to 128-column instructions
    widths = {}
    for n_cols in (32, 64, 80, 128, 256):
        cyc, _ = rtn.rtn_probe_i8_rate(n_cols, 4096)
        torch.cuda.synchronize()
        widths[str(n_cols)] = float(np.median(cyc.cpu().numpy())) / 4096.0
    out["i8"]["cycles_per_mma_by_columns"] = widths
    if rtn.rtn_last_device_status() != 0:
        raise RuntimeError("device status after the peak probes")
    # what a plain copy reaches at the size of the HBM-bound conv configurations (25.7 MB in, 25.7 MB out):
    # rotating buffers larger than L2, the launches in a CUDA graph like the timed steps
    nbytes, n_sets, reps = 25_690_112, 8, 40
    srcs = [torch.empty(nbytes, dtype=torch.uint8, device="cuda").fill_(j) for j in range(n_sets)]
    dsts = [torch.empty(nbytes, dtype=torch.uint8, device="cuda") for _ in range(n_sets)]
    for j in range(n_sets):
        rtn.rtn_probe_copy(srcs[j], dsts[j])
    torch.cuda.synchronize()
    g = torch.cuda.CUDAGraph()
    with torch.cuda.graph(g):
        for i in range(reps):
            rtn.rtn_probe_copy(srcs[i % n_sets], dsts[i % n_sets])
    g.replay()
    torch.cuda.synchronize()
    times = []
    for _ in range(5):
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for _ in range(25):
            g.replay()
        e1.record()
        torch.cuda.synchronize()
        times.append(e0.elapsed_time(e1) / (25 * reps))
    ms = sorted(times)[2]
    hbm = measured_peaks()[0]
    out["copy"] = {"bytes_read": nbytes, "bytes_written": nbytes, "kernel_ms": ms, "gbs": 2 * nbytes / (ms * 1e-3) / 1e9,
                   "frac_of_hbm_peak": 2 * nbytes / (ms * 1e-3) / 1e9 / hbm,
                   "source": "measured: rtn_probe_copy, 16 bytes per thread and trip, 2 x 1024 threads per SM, graph replay "
                             "on 8 rotating buffer pairs; the ceiling a pure data mover sets for a 51 MB conv call"}
    del srcs, dsts
    return out


# ------------------------------------------------------------------------------------------------
# GPU legs, one per kind of workload; each returns the configuration's entry
# ------------------------------------------------------------------------------------------------
VARIANT_IDS = {"auto": 0, "popc": 1, "i8": 2}


def bench_conv(ctx, case, name, peaks):
    import paper_1912_02057_b200 as rtn
    torch, args = ctx.torch, ctx.args
    dev = ctx.dev
    packed_io = args.io == "packed"
    step_bytes = algorithmic_bytes(case, args.io)
    n_sets = min(64, max(2, int(np.ceil(2.5 * L2_BYTES / step_bytes))))
    w_packed, w_sum = rtn.rtn_pack_weights(dev(case.w_codes))
    w_s, w_o = dev(case.w_scale), dev(case.w_offset)
    t_lo, t_hi = dev(case.t_lo), dev(case.t_hi)
    shape = (case.B, case.C, case.H, case.W, case.N, case.kh, case.kw, case.stride, case.pad)
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
        variant = "i8"
        launches_per_step = rtn.rtn_conv_next_kernel_launches(*shape)

        def step(i):
            j = i % n_sets
            rtn.rtn_ternary_conv2d_packed(xs[j], case.B, case.C, case.H, case.W, w_packed, w_sum, case.N,
                                          case.kh, case.kw, case.stride, case.pad, rtn.PAD_CODE_ZERO,
                                          case.a_scale, case.a_offset, w_s, w_o, relu=True,
                                          next_t_lo=n_lo, next_t_hi=n_hi, out_packed=outs[j])
            return outs[j]
        host_in = x0.cpu().pin_memory()
    else:
        xs = [dev(case.x) for _ in range(n_sets)]
        outs = [torch.empty((case.B, case.N, case.Ho, case.Wo), dtype=torch.float32, device="cuda")
                for _ in range(n_sets)]
        vid = VARIANT_IDS[args.variant]
        if vid == 0:
            vid = rtn.rtn_choose_conv_variant(*shape)
            launches_per_step = rtn.rtn_conv_kernel_launches(*shape)
        else:
            launches_per_step = 1 if vid == 1 else rtn.rtn_conv_kernel_launches(*shape)
        variant = {1: "popc", 2: "i8"}[vid]

        def step(i):
            j = i % n_sets
            rtn.rtn_ternary_conv2d(xs[j], t_lo, t_hi, w_packed, w_sum, case.N, case.kh, case.kw,
                                   case.stride, case.pad, rtn.PAD_CODE_ZERO, case.a_scale,
                                   case.a_offset, w_s, w_o, out=outs[j], variant=vid)
            return outs[j]
        host_in = torch.from_numpy(case.x).pin_memory()
    host_out = torch.empty(outs[0].shape, dtype=outs[0].dtype).pin_memory()
    ms, timing, clocks = time_steps(ctx, step, args.steps, args.warmup, launches_per_step)
    if rtn.rtn_last_device_status() != 0:
        raise RuntimeError(f"{name}: device status after the timed region")
    ops = ops_of(case)
    e2e_ms, pipelined = time_e2e(ctx, step, xs, host_in, host_out, n_sets,
                                 e2e_steps_for(host_in.numel() * host_in.element_size() + host_out.numel() * host_out.element_size(), args.steps))
    key = name + ("/packed" if packed_io else "") + ("/popc" if variant == "popc" else "")
    return {
        "workload": name, "ms_per_step": ms, "value": whole_job_tops(ops, ctx.world, ms), "unit": "TOPS",
        "io": args.io, "variant": variant, "launches_per_step": int(launches_per_step),
        "l2": f"{n_sets} rotating input/output sets ({n_sets * step_bytes >> 20} MiB) > L2",
        "roofline": roofline_of(key, step_bytes, ops, ms, variant, peaks),
        "e2e": e2e_dict(ctx, ops, e2e_ms, pipelined, host_in, host_out),
        "timing": timing, "clocks": clocks,
    }


def bench_gemm(ctx, case, name, peaks):
    import paper_1912_02057_b200 as rtn
    torch, args = ctx.torch, ctx.args
    dev = ctx.dev
    M, N, K = case.M, case.N, case.K
    step_bytes = algorithmic_bytes(case)
    n_sets = min(64, max(2, int(np.ceil(2.5 * L2_BYTES / step_bytes))))
    w_packed, w_sum = rtn.rtn_pack_weights(dev(case.w_codes))
    w_s, w_o = dev(case.w_scale), dev(case.w_offset)
    t_lo, t_hi = dev(case.t_lo), dev(case.t_hi)
    xs = [dev(case.a) for _ in range(n_sets)]
    a_s, a_o = dev(case.a_scale), dev(case.a_offset)
    packs = [torch.empty((M, rtn.rtn_packed_row_bytes(K)), dtype=torch.uint8, device="cuda") for _ in range(n_sets)]
    sums = [torch.empty((M,), dtype=torch.int32, device="cuda") for _ in range(n_sets)]
    outs = [torch.empty((M, N), dtype=torch.float32, device="cuda") for _ in range(n_sets)]
    vid = VARIANT_IDS[args.variant]
    if vid == 0:
        vid = rtn.rtn_choose_gemm_variant(M, N, K)
        gemm_launches = rtn.rtn_gemm_kernel_launches(M, N, K) + (1 if rtn.rtn_gemm_k_slices(M, N, K) > 1 else 0)
    else:
        gemm_launches = 1 if vid == 1 else 2        # forced: the bit-plane kernel unsliced, or expansion + contraction at most
    variant = {1: "popc", 2: "i8"}[vid]
    launches_per_step = 1 + gemm_launches           # ternarize_pack + the GEMM's kernels (+ the memset of a sliced K)

    def gemm(j):
        rtn.rtn_ternary_gemm(packs[j], sums[j], w_packed, w_sum[0], M, N, K, a_s, a_o, w_s, w_o, out=outs[j],
                             variant=vid if args.variant != "auto" else 0)

    def step(i):
        j = i % n_sets
        rtn.rtn_ternarize_pack_act(xs[j], t_lo, t_hi, out=packs[j], out_sum=sums[j])
        gemm(j)
        return outs[j]
    ms, timing, clocks = time_steps(ctx, step, args.steps, args.warmup, launches_per_step)
    # the dominant kernel (rtn_ternary_gemm) timed alone on the rotating operand sets
    kernel_ms, kernel_timing, _ = time_steps(ctx, lambda i: gemm(i % n_sets), args.steps, 3, gemm_launches, sample_clocks=False)
    if rtn.rtn_last_device_status() != 0:
        raise RuntimeError(f"{name}: device status after the timed region")
    kernel_bytes = (M + N) * ((K + 127) // 128) * 32 + 4 * M * N
    ops = ops_of(case)
    host_in = torch.from_numpy(case.a).pin_memory()
    host_out = torch.empty((M, N), dtype=torch.float32).pin_memory()
    e2e_ms, pipelined = time_e2e(ctx, step, xs, host_in, host_out, n_sets,
                                 e2e_steps_for(host_in.numel() * 4 + host_out.numel() * 4, args.steps))
    launch_bound = ops < 1e8
    if launch_bound:
        roof = {"bound": "launch", "frac": None, "achieved": None, "peak": None, "unit": None, "traffic": None,
                "kernel_ms": kernel_ms,
                "note": "launch-bound: the problem is microseconds of work for one SM wave; a fraction of a memory or "
                        "tensor roofline says nothing here.  kernel_ms is the time per call inside a CUDA graph."}
    else:
        roof = roofline_of(name + ("/popc" if variant == "popc" and args.variant != "auto" else ""), kernel_bytes, ops,
                           kernel_ms, variant, peaks)
    return {
        "workload": name, "ms_per_step": ms, "value": whole_job_tops(ops, ctx.world, ms), "unit": "TOPS",
        "io": "fp32", "variant": variant, "launches_per_step": int(launches_per_step),
        "gemm_kernel_ms": kernel_ms, "gemm_kernel_tops": ops / (kernel_ms * 1e-3) / 1e12,
        "l2": (f"{n_sets} rotating operand/output sets ({n_sets * step_bytes >> 20} MiB)"
               + (" > L2" if n_sets * step_bytes > L2_BYTES else ": fits L2 (launch-bound size)")),
        "roofline": roof,
        "e2e": e2e_dict(ctx, ops, e2e_ms, pipelined, host_in, host_out),
        "timing": timing, "kernel_timing": kernel_timing, "clocks": clocks,
    }


def bench_body(ctx, case, name, peaks):
    """Whole-chain workload: a step = the 19 ternary layers of ResNet-18 on one batch."""
    import paper_1912_02057_b200 as rtn
    from paper_1912_02057_b200 import chain
    torch, args = ctx.torch, ctx.args
    n_sets = 2          # two complete sets of activations (input, every intermediate), used in turn
    bodies = [chain.Body(case.blocks, case.B) for _ in range(n_sets)]
    xs = [torch.from_numpy(case.x).cuda() for _ in range(n_sets)]
    host_in = torch.from_numpy(case.x).pin_memory()
    outs = [None] * n_sets

    def step(i):
        j = i % n_sets
        outs[j], _ = bodies[j].forward(xs[j])
        return outs[j]
    launches = bodies[0].kernel_launches()
    steps = min(args.steps, 100)
    ms, timing, clocks = time_steps(ctx, step, steps, args.warmup, launches)
    if rtn.rtn_last_device_status() != 0:
        raise RuntimeError(f"{name}: device status after the timed region")
    host_out = torch.empty(outs[0].shape, dtype=torch.float32).pin_memory()
    e2e_ms, pipelined = time_e2e(ctx, step, xs, host_in, host_out, n_sets, max(3, min(steps, 20)))
    ops = bodies[0].ops()
    roof = roofline_of(name, bodies[0].algorithmic_bytes(), ops, ms, "i8", peaks)
    roof["note"] = "whole chain (19 layers) against the binding bound of its summed bytes and operations"
    return {
        "workload": name, "ms_per_step": ms, "value": whole_job_tops(ops, ctx.world, ms), "unit": "TOPS",
        "io": "packed rows between layers, fp32 residual stream", "variant": "i8",
        "images_per_s": ctx.world * case.B / (ms * 1e-3), "layers": 19, "launches_per_step": int(launches),
        "l2": f"{n_sets} complete sets of activations used in turn; a layer's output may still be in L2 "
              "when its consumer reads it (part of the chain, not of the timing method)",
        "roofline": roof, "e2e": e2e_dict(ctx, ops, e2e_ms, pipelined, host_in, host_out),
        "timing": timing, "clocks": clocks,
    }


def bench_full(ctx, case, name, peaks):
    """Full ResNet-18 topology: fp32 stem (torch) -> 19 ternary layers (the library) -> fp32 classifier (torch).
    A step = one forward pass of a batch of 224x224 images; the ternary body is also timed alone on the stem's
    output."""
    import paper_1912_02057_b200 as rtn
    from paper_1912_02057_b200 import chain
    torch, args = ctx.torch, ctx.args
    F = torch.nn.functional
    stem_w, fc_w, fc_b = (ctx.dev(t) for t in case.ends)
    n_sets = 2
    imgs = [torch.from_numpy(case.images).cuda() for _ in range(n_sets)]
    with torch.no_grad():
        s0 = case.stem(torch, imgs[0], stem_w)
    case.calibrate(torch, s0)
    bodies = [chain.Body(case.blocks, case.B) for _ in range(n_sets)]
    stems = [torch.empty_like(s0) for _ in range(n_sets)]
    logits = [None] * n_sets

    def body_step(i):
        j = i % n_sets
        out, _ = bodies[j].forward(stems[j])
        return out

    def step(i):
        j = i % n_sets
        with torch.no_grad():
            case.stem(torch, imgs[j], stem_w, out=stems[j])
            out, _ = bodies[j].forward(stems[j])
            logits[j] = F.linear(out.mean((2, 3)), fc_w, fc_b)
        return logits[j]
    launches = bodies[0].kernel_launches()
    steps = min(args.steps, 100)
    ms, timing, clocks = time_steps(ctx, step, steps, args.warmup, launches)
    body_ms, body_timing, _ = time_steps(ctx, body_step, steps, 3, launches, sample_clocks=False)
    if rtn.rtn_last_device_status() != 0:
        raise RuntimeError(f"{name}: device status after the timed region")
    # the codes along the chain stay non-degenerate with the calibrated thresholds
    last = oracle_free_code_fractions(torch, bodies[0].bufs[-1]["p_next"], case.blocks[-1]["conv2"].cout)
    host_in = torch.from_numpy(case.images).pin_memory()
    host_out = torch.empty(logits[0].shape, dtype=torch.float32).pin_memory()
    e2e_ms, pipelined = time_e2e(ctx, step, imgs, host_in, host_out, n_sets, max(3, min(steps, 20)))
    ops = bodies[0].ops()
    stem_flops = 2.0 * case.B * 112 * 112 * 64 * 3 * 49
    roof = roofline_of("r18_body_b64", bodies[0].algorithmic_bytes(), ops, body_ms, "i8", peaks)
    roof["note"] = ("the ternary body (19 layers) against the binding bound of its summed bytes and operations; "
                    "the fp32 ends run in torch (cuDNN / cuBLAS) and are outside the path")
    return {
        "workload": name, "ms_per_step": ms, "value": whole_job_tops(ops, ctx.world, ms), "unit": "TOPS",
        "value_note": "ternary operations of the 19 layers over the time of the whole forward pass",
        "io": "fp32 images in, fp32 logits out; packed rows between ternary layers, fp32 residual stream",
        "variant": "i8", "images_per_s": ctx.world * case.B / (ms * 1e-3),
        "body_ms": body_ms, "body_images_per_s": ctx.world * case.B / (body_ms * 1e-3),
        "body_tops": whole_job_tops(ops, ctx.world, body_ms),
        "fp32_ends_ms": ms - body_ms, "stem_gflop": stem_flops / 1e9,
        "thresholds": f"0.3 / 1.0 x sigma along the chain, sigma_in = std(stem output) / 0.584 = {case.sigma_in:.4f}",
        "code_fractions_last_block": last,
        "layers": "fp32 stem + 19 ternary + fp32 classifier", "launches_per_step": int(launches),
        "l2": f"{n_sets} complete sets of images and activations used in turn",
        "roofline": roof, "e2e": e2e_dict(ctx, ops, e2e_ms, pipelined, host_in, host_out),
        "timing": timing, "body_timing": body_timing, "clocks": clocks,
    }


def oracle_free_code_fractions(torch, packed_rows, n_codes):
    """Fractions of -1 / 0 / +1 in packed pixel rows, counted from the bit planes with torch integer ops (a
    report on the data, no part of the path)."""
    rows = packed_rows.view(packed_rows.shape[0], -1, 2, 16).to(torch.int32)
    bits = lambda t: sum(((t >> k) & 1).sum().item() for k in range(8))
    nz = bits(rows[:, :, 0, :])
    pos = bits(rows[:, :, 0, :] & rows[:, :, 1, :])
    total = float(packed_rows.shape[0] * n_codes)
    return {"-1": (nz - pos) / total, "0": 1.0 - nz / total, "+1": pos / total}


def bench_quaternary(ctx, case, name, peaks):
    """rtn_quaternary_gemm against rtn_ternary_gemm's bit-plane variant at the same size."""
    import paper_1912_02057_b200 as rtn
    torch, args = ctx.torch, ctx.args
    dev = ctx.dev
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

    def q_step(i):
        j = i % n_sets
        return rtn.rtn_quaternary_gemm(xq[j], wq, n, n, n, out=outs[j])

    def t_step(i):
        j = i % n_sets
        return rtn.rtn_ternary_gemm(packs[j][0], packs[j][1], w_packed, w_sum[0], n, n, n, a_s, a_o, w_s, w_o,
                                    out=fouts[j], variant=rtn.VARIANT_POPC)
    steps = min(args.steps, 200)
    t_ms, _, _ = time_steps(ctx, t_step, steps, args.warmup, 1, sample_clocks=False)
    q_ms, timing, clocks = time_steps(ctx, q_step, steps, args.warmup, 1)
    host_in = torch.from_numpy(case.x).pin_memory()
    dx = [torch.empty((n, n), dtype=torch.uint8, device="cuda") for _ in range(2)]
    host_out = torch.empty((n, n), dtype=torch.int32).pin_memory()
    e2e_ms, pipelined = time_e2e(ctx, lambda j: rtn.rtn_quaternary_gemm(rtn.rtn_pack_quaternary(dx[j]), wq, n, n, n, out=outs[j]),
                                 dx, host_in, host_out, 2, 5)
    ops = 2.0 * n * n * n
    achieved = ops / (q_ms * 1e-3) / 1e12
    alu = (peaks or {}).get("popc")
    # four popcounts per 32 multiply-accumulates against the ternary pattern's two
    peak = alu["tops"] / 2.0 if alu else None
    return {
        "workload": name, "metric": "effective 2-bit TOPS (2MNK/s)", "ms_per_step": q_ms, "value": achieved, "unit": "TOPS",
        "io": "packed", "variant": "popc", "launches_per_step": 1,
        "ternary_popc_ms": t_ms, "ternary_popc_tops": ops / (t_ms * 1e-3) / 1e12, "quaternary_over_ternary_time": q_ms / t_ms,
        "note": "same tiling for both; per 32 values and output 4 popcounts (quaternary) against 2 (ternary, Eq. 9)",
        "l2": f"{n_sets} rotating operand/output sets > L2",
        "roofline": {"bound": "alu", "achieved": achieved, "peak": peak, "unit": "TOP/s",
                     "frac": achieved / peak if peak else None, "traffic": None, "kernel_ms": q_ms,
                     "peak_source": (alu["source"] + "; halved: four popcounts per 32 code pairs instead of two") if alu else None},
        "e2e": e2e_dict(ctx, ops, e2e_ms, pipelined, host_in, host_out),
        "timing": timing, "clocks": clocks,
    }


def bench_one(ctx, name, peaks):
    """Builds the workload's inputs, runs its leg, frees its device memory."""
    import gc
    case = WORKLOADS[name]()
    if isinstance(case, QuaternaryCase):
        entry = bench_quaternary(ctx, case, name, peaks)
    elif isinstance(case, FullCase):
        entry = bench_full(ctx, case, name, peaks)
    elif isinstance(case, BodyCase):
        entry = bench_body(ctx, case, name, peaks)
    elif isinstance(case, inputs.ConvCase):
        entry = bench_conv(ctx, case, name, peaks)
    else:
        entry = bench_gemm(ctx, case, name, peaks)
    gc.collect()
    ctx.torch.cuda.empty_cache()
    return entry, case


# ------------------------------------------------------------------------------------------------
# CPU oracle leg (reference arm and cpu_baseline)
# ------------------------------------------------------------------------------------------------
def oracle_sample(case, budget_s=12.0, io="fp32", fill_budget=False):
    """Times the CPU oracle, as it stands, on a bounded sample of the workload.
    Returns (ops per second, seconds, description).  fill_budget: when the whole batch takes a small part
    of the budget, run it several times in a row so that the figure rests on about budget_s of CPU work."""
    import oracle
    if isinstance(case, (BodyCase, FullCase)):
        return oracle_body_sample(case, budget_s)
    if isinstance(case, QuaternaryCase):
        rows = 16
        t0 = time.perf_counter()
        oracle.quaternary_gemm(case.x[:rows], case.w)
        dt = time.perf_counter() - t0
        rows = int(max(rows, min(case.n, rows * budget_s / max(dt, 1e-6))))
        t0 = time.perf_counter()
        oracle.quaternary_gemm(case.x[:rows], case.w)
        dt = time.perf_counter() - t0
        return 2.0 * rows * case.n * case.n / dt, dt, f"first {rows} of {case.n} rows, all columns"
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


def oracle_body_sample(case, budget_s=12.0):
    """The CPU oracle on the body's first residual block (two 3x3 layers with the hand-over between
    them) for as many images as fit the time budget.  Returns (ops per second, seconds, description)."""
    import oracle
    if isinstance(case, FullCase):
        # the stem's output for the sampled images, in torch on the CPU (full precision, outside the path)
        import torch
        with torch.no_grad():
            s_all = case.stem(torch, torch.from_numpy(case.images[:4]), torch.from_numpy(case.ends[0])).numpy()
        if case.blocks is None:
            case.calibrate(torch, torch.from_numpy(s_all))
    else:
        s_all = case.x
    c1, c2 = case.blocks[0]["conv1"], case.blocks[0]["conv2"]
    nxt = case.blocks[1]["conv1"]

    def run(nb):
        s = s_all[:nb]
        t0 = time.perf_counter()
        p = oracle.ternarize(s, c1.t_lo, c1.t_hi)
        _, pre1, _ = oracle.conv2d(p, c1.w_codes, 1, 1, oracle.PAD_CODE_ZERO, c1.a_scale, c1.a_offset, c1.w_scale, c1.w_offset)
        _, q, _ = oracle.next_layer(pre1, True, None, c2.t_lo, c2.t_hi)
        _, pre2, _ = oracle.conv2d(q, c2.w_codes, 1, 1, oracle.PAD_CODE_ZERO, c2.a_scale, c2.a_offset, c2.w_scale, c2.w_offset)
        oracle.next_layer(pre2, True, s, nxt.t_lo, nxt.t_hi)
        dt = time.perf_counter() - t0
        return 2 * 2.0 * nb * 56 * 56 * 64 * 64 * 9, dt
    ops, dt = run(1)
    nb = int(max(1, min(len(s_all), budget_s / max(dt, 1e-6))))
    if nb > 1:
        ops, dt = run(nb)
    return ops / dt, dt, f"first residual block (layer1.0.conv1, conv2 and their hand-over) on {nb} of {case.B} images"


def run_reference(args, name):
    """The reference arm: the CPU oracle, as it stands, on a bounded sample of the workload per step."""
    import oracle
    if int(os.environ.get("RANK", "0")) != 0:
        return
    case = WORKLOADS[name]()
    per_step_budget = max(0.2, min(12.0, 60.0 / max(1, args.steps + args.warmup)))
    sample = ""
    for _ in range(min(args.warmup, 3)):
        _, _, sample = oracle_sample(case, per_step_budget, args.io)
    rates, secs = [], []
    for _ in range(args.steps):
        r, dt, sample = oracle_sample(case, per_step_budget, args.io)
        rates.append(r)
        secs.append(dt)
    value = float(np.mean(rates)) / 1e12
    metric = "effective 2-bit TOPS (2MNK/s)" if isinstance(case, QuaternaryCase) else METRIC
    print(json.dumps({
        "impl": "reference", "metric": metric, "value": value, "unit": "TOPS", "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": 1e3 * float(np.mean(secs)),
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "int64", "data": "synthetic",
        "config": {"workload": name, "io": args.io, "note": "CPU oracle on a bounded sample per step"},
        "cpu_baseline": {"value": value, "unit": "TOPS", "cores": oracle.threads(), "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": "TOPS", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0}))


# ------------------------------------------------------------------------------------------------
def run_ours(args):
    import paper_1912_02057_b200 as rtn
    ctx = Ctx(args)
    names = [args.workload] if args.workload else list(SUITE)
    headline = args.workload or HEADLINE
    peaks = run_peaks(ctx)
    entries, head_case = [], None
    for name in names:
        entry, case = bench_one(ctx, name, peaks)
        entries.append(entry)
        if name == headline:
            head_case = case
        else:
            del case
    head = next(e for e in entries if e["workload"] == headline)
    if ctx.rank == 0:
        line = {
            "metric": head.get("metric", METRIC), "value": head["value"], "unit": "TOPS", "n_gpus": ctx.world,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": head["ms_per_step"],
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": DTYPE, "data": "synthetic",
            "config": {"workload": headline, "io": head["io"], "variant": head["variant"], "l2": head["l2"],
                       "weights": "packed before the timed region (offline step)",
                       "launch": head["timing"]["launch"],
                       "timing": f"median of {REGIONS} regions of at least {REGION_MS:.0f} ms, each a whole number of --steps repeats",
                       "suite": names,
                       "parallelism": "replicas only" if ctx.world > 1 else "1 GPU"},
            "clocks": head["clocks"], "e2e": head["e2e"], "gpu_launches": int(ctx.launches),
            "roofline": head["roofline"], "peaks": peaks,
        }
        for k in ("images_per_s", "body_images_per_s"):
            if k in head:
                line["config"][k] = head[k]
        if not args.no_cpu_baseline and ctx.world == 1:
            import oracle
            rate, dt, sample = oracle_sample(head_case, 12.0, args.io, fill_budget=True)
            line["cpu_baseline"] = {"value": rate / 1e12, "unit": "TOPS", "cores": oracle.threads(),
                                    "kind": "oracle", "sample": sample, "seconds": dt}
        if len(entries) > 1:
            line["per_config"] = entries
        else:
            line["detail"] = head
        print(json.dumps(line))
    assert rtn.rtn_last_device_status() == 0
    ctx.close()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default=None, choices=sorted(WORKLOADS),
                    help="one configuration instead of the whole list")
    ap.add_argument("--variant", default="auto", choices=["auto", "popc", "i8"],
                    help="kernel family of the single-layer workloads: the library's choice, the bit-plane "
                         "(AND / popcount) kernels, or the tensor-core kernels")
    ap.add_argument("--io", default="fp32", choices=["fp32", "packed"],
                    help="conv workloads: fp32 NCHW in and out (rtn_ternary_conv2d), or packed pixel rows in and "
                         "out with the hand-over to the next layer fused (rtn_ternary_conv2d_packed)")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--eager", action="store_true",
                    help="launch the timed steps one by one instead of through a CUDA graph (for profilers)")
    args = ap.parse_args()
    if args.warmup < 3:
        args.warmup = 3
    if args.steps < 1:
        args.steps = 1
    if args.impl == "reference":
        run_reference(args, args.workload or HEADLINE)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
