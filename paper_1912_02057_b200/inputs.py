"""Seeded synthetic inputs shaped like the paper's ResNet-18 / ImageNet layers.

This module only draws random numbers (numpy ``default_rng``, PCG64) and names shapes.  It
holds none of the method's arithmetic: no thresholding, no packing, no sums.  Both the CUDA
library's callers and the CPU checker's callers take their inputs from here, so both sides see
the same bytes.

The paper (arXiv 1912.02057, section "Experiments") evaluates on ImageNet and CIFAR-10 with
trained weights; neither is needed for the forward contraction, and these tensors stand in:
post-ReLU activations are max(0, N(0,1)), weight codes are i.i.d. with a chosen zero fraction
and symmetric signs, scales are U(0.5, 1.5) and offsets U(-0.1, 0.1) (the learned values the
paper lists in its appendix table of scales and offsets have the same order of magnitude).
"""
from dataclasses import dataclass, field

import numpy as np


def rng(seed):
    return np.random.default_rng(seed)


def weight_codes(g, shape, p_zero):
    """i.i.d. codes: P(0) = p_zero, P(+1) = P(-1) = (1 - p_zero) / 2."""
    u = g.random(shape, dtype=np.float32)
    half = (1.0 - p_zero) / 2.0
    codes = np.zeros(shape, np.int8)
    codes[u < half] = -1
    codes[u >= 1.0 - half] = 1
    return codes


def relu_normal(g, shape):
    """fp32 max(0, N(0,1)): what a ReLU layer hands to the next layer's BN + ternarizer."""
    a = g.standard_normal(shape, dtype=np.float32)
    np.maximum(a, 0.0, out=a)
    return a


def uniform(g, lo, hi, shape=()):
    return (lo + (hi - lo) * g.random(shape, dtype=np.float64)).astype(np.float32)


@dataclass
class GemmCase:
    """One ternary GEMM problem: fp32 activations [M,K], weight codes [N,K], parameters."""
    name: str
    a: np.ndarray          # fp32 [M,K]
    w_codes: np.ndarray    # int8 [N,K]
    t_lo: np.ndarray       # fp32 [1] or [K]
    t_hi: np.ndarray
    a_scale: np.ndarray    # fp32 [1] or [M]
    a_offset: np.ndarray
    w_scale: np.ndarray    # fp32 [1] or [N]
    w_offset: np.ndarray

    @property
    def M(self): return self.a.shape[0]
    @property
    def N(self): return self.w_codes.shape[0]
    @property
    def K(self): return self.a.shape[1]


@dataclass
class ConvCase:
    """One ternary conv2d problem: fp32 NCHW input, weight codes [N,C,kh,kw], parameters."""
    name: str
    x: np.ndarray          # fp32 [B,C,H,W]
    w_codes: np.ndarray    # int8 [N,C,kh,kw]
    stride: int
    pad: int
    t_lo: np.ndarray       # fp32 [1] or [C]
    t_hi: np.ndarray
    a_scale: float
    a_offset: float
    w_scale: np.ndarray    # fp32 [1] or [N]
    w_offset: np.ndarray
    notes: dict = field(default_factory=dict)

    @property
    def B(self): return self.x.shape[0]
    @property
    def C(self): return self.x.shape[1]
    @property
    def H(self): return self.x.shape[2]
    @property
    def W(self): return self.x.shape[3]
    @property
    def N(self): return self.w_codes.shape[0]
    @property
    def kh(self): return self.w_codes.shape[2]
    @property
    def kw(self): return self.w_codes.shape[3]
    @property
    def Ho(self): return (self.H + 2 * self.pad - self.kh) // self.stride + 1
    @property
    def Wo(self): return (self.W + 2 * self.pad - self.kw) // self.stride + 1
    @property
    def gemm_mnk(self):
        return (self.B * self.Ho * self.Wo, self.N, self.C * self.kh * self.kw)


def gemm_case(name, M, N, K, seed, p_zero, act="relu", thresholds=(0.3, 1.0),
              per_row_act_params=False, a_scale=None, a_offset=None, per_k_thresholds=False):
    g = rng(seed)
    w = weight_codes(g, (N, K), p_zero)
    if act == "relu":
        a = relu_normal(g, (M, K))
    elif act == "uniform3":          # U(-1.5, 1.5): thresholds -0.5/+0.5 split it in thirds
        a = (3.0 * g.random((M, K), dtype=np.float32) - 1.5).astype(np.float32)
    else:
        raise ValueError(act)
    if per_k_thresholds:
        lo = uniform(g, thresholds[0] - 0.1, thresholds[0] + 0.1, (K,))
        hi = uniform(g, thresholds[1] - 0.1, thresholds[1] + 0.1, (K,))
    else:
        lo = np.array([thresholds[0]], np.float32)
        hi = np.array([thresholds[1]], np.float32)
    w_s, w_o = uniform(g, 0.5, 1.5, (N,)), uniform(g, -0.1, 0.1, (N,))
    if per_row_act_params:
        a_s, a_o = uniform(g, 0.5, 1.5, (M,)), uniform(g, -0.1, 0.1, (M,))
    else:
        a_s = np.array([1.0 if a_scale is None else a_scale], np.float32)
        a_o = np.array([0.05 if a_offset is None else a_offset], np.float32)
    return GemmCase(name, a, w, lo, hi, a_s, a_o, w_s, w_o)


def conv_case(name, B, C, H, W, N, k, stride, pad, seed, p_zero, thresholds="around_offset",
              per_channel_thresholds=False):
    g = rng(seed)
    w = weight_codes(g, (N, C, k, k), p_zero)
    x = relu_normal(g, (B, C, H, W))
    w_s, w_o = uniform(g, 0.5, 1.5, (N,)), uniform(g, -0.1, 0.1, (N,))
    a_s, a_o = float(uniform(g, 0.5, 1.5)), float(uniform(g, -0.1, 0.1))
    if thresholds == "around_offset":      # +-0.5 around the activation offset
        lo, hi = a_o - 0.5, a_o + 0.5
    else:
        lo, hi = thresholds
    if per_channel_thresholds:
        t_lo = uniform(g, lo - 0.1, lo + 0.1, (C,))
        t_hi = uniform(g, hi - 0.1, hi + 0.1, (C,))
    else:
        t_lo, t_hi = np.array([lo], np.float32), np.array([hi], np.float32)
    return ConvCase(name, x, w, stride, pad, t_lo, t_hi, a_s, a_o, w_s, w_o)


# ------------------------------------------------------------------ the five named workloads
def config1():
    """GEMM 64x64x576 (a 3x3x64 conv unrolled), P(0)=0.4, thresholds 0.3 / 1.0, seed 0."""
    return gemm_case("cfg1_gemm_64x64x576", 64, 64, 576, seed=0, p_zero=0.4,
                     thresholds=(0.3, 1.0), a_scale=1.0, a_offset=0.05)


def config2(batch=32, thresholds="around_offset"):
    """conv 3x3 s1 p1, 64->64, 56x56, batch 32; thresholds +-0.5 around the activation offset."""
    return conv_case(f"cfg2_conv3x3_c64_56x56_b{batch}", batch, 64, 56, 56, 64, 3, 1, 1,
                     seed=2, p_zero=0.4, thresholds=thresholds)


def config3a(p_zero=0.5, batch=128):
    """conv 3x3 s1 p1, 256->256, 14x14, batch 128; weight-zero fraction swept."""
    return conv_case(f"cfg3a_conv3x3_c256_14x14_b{batch}_z{p_zero}", batch, 256, 14, 14, 256, 3,
                     1, 1, seed=3, p_zero=p_zero)


def config3b(p_zero=0.5, batch=128):
    """1x1 stride-2 downsample conv 128->256 at 28x28, batch 128."""
    return conv_case(f"cfg3b_conv1x1s2_c128_28x28_b{batch}_z{p_zero}", batch, 128, 28, 28, 256, 1,
                     2, 0, seed=31, p_zero=p_zero)


def config5(n):
    """Square GEMM M=N=K=n, codes 1/3 each, per-row activation and per-column weight params."""
    return gemm_case(f"cfg5_gemm_{n}", n, n, n, seed=5, p_zero=1.0 / 3.0, act="uniform3",
                     thresholds=(-0.5, 0.5), per_row_act_params=True)


def resnet18_ternary_layers():
    """The 19 ternary conv layers of ResNet-18 (stages 1-4; stem and FC stay full precision),
    in the order of the paper's appendix table of learned scales and offsets.
    Tuples: (name, C_in, C_out, k, stride, pad, H_in)."""
    L = []
    L += [(f"layer1.{b}.conv{c}", 64, 64, 3, 1, 1, 56) for b in (0, 1) for c in (1, 2)]
    for s, (cin, cout, hin) in enumerate([(64, 128, 56), (128, 256, 28), (256, 512, 14)], start=2):
        hout = hin // 2
        L += [(f"layer{s}.0.conv1", cin, cout, 3, 2, 1, hin),
              (f"layer{s}.0.conv2", cout, cout, 3, 1, 1, hout),
              (f"layer{s}.0.downsample.0", cin, cout, 1, 2, 0, hin),
              (f"layer{s}.1.conv1", cout, cout, 3, 1, 1, hout),
              (f"layer{s}.1.conv2", cout, cout, 3, 1, 1, hout)]
    return L


def resnet18_layer(name, batch=128, p_zero=0.5):
    """One of the 19 ternary conv layers of ResNet-18 as a ConvCase (thresholds around the offset)."""
    for i, (lname, cin, cout, k, stride, pad, hin) in enumerate(resnet18_ternary_layers()):
        if lname == name:
            return conv_case(f"r18_{name}_b{batch}", batch, cin, hin, hin, cout, k, stride, pad,
                             seed=400 + i, p_zero=p_zero)
    raise KeyError(name)


def resnet18_fp32_ends(seed=46):
    """Random-init weights of the two full-precision ends of ResNet-18 (section "Implementation Details":
    first and last layer stay full precision): stem conv [64,3,7,7] ~ N(0, 2/(64*49)), classifier
    [1000,512] ~ U(-1/sqrt(512), 1/sqrt(512)) with a bias of the same range."""
    g = rng(seed)
    stem = (g.standard_normal((64, 3, 7, 7), dtype=np.float32) * np.float32(np.sqrt(2.0 / (64 * 49)))).astype(np.float32)
    bound = 1.0 / np.sqrt(512.0)
    return stem, uniform(g, -bound, bound, (1000, 512)), uniform(g, -bound, bound, (1000,))


# ------------------------------------------------------------------ the ternary body of ResNet-18 as a chain
@dataclass
class BodyLayer:
    """One ternary conv layer of the chain with everything it needs (random init, seeded)."""
    name: str
    cin: int
    cout: int
    k: int
    stride: int
    pad: int
    hin: int               # input height = width
    w_codes: np.ndarray    # int8 [cout, cin, k, k]
    a_scale: float         # gamma, beta of the layer's activation (Eq. 4)
    a_offset: float
    w_scale: np.ndarray    # alpha per filter (Eq. 5) and the weight offset the library adds, fp32 [cout]
    w_offset: np.ndarray
    t_lo: np.ndarray       # thresholds of the ternarizer in FRONT of this layer (its BN folded, Eq. 3), fp32 [1]
    t_hi: np.ndarray
    sigma_out: float       # estimated standard deviation of the layer's conv output (sets the thresholds downstream)


def resnet18_body(seed=4, p_zero=0.5, dyadic=False, hin=56):
    """The 19 ternary conv layers of ResNet-18 (paper's appendix table) with random-init codes and
    parameters, plus thresholds that keep all three codes in use along the chain.

    Threshold rule: the ternarizer in front of a layer sees y = phi(conv) [+ skip] with standard
    deviation about sigma (conv: c1 * sqrt(K * q_x * q_w) with q the non-zero fractions, estimated
    as 0.5; the residual stream adds the variances of its branches); t_lo = 0.3 sigma, t_hi =
    1.0 sigma, the pair config 1 uses for a unit-scale post-ReLU input.  dyadic=True rounds every
    parameter to a small multiple of a power of two, so that every product and sum of the
    epilogues is exact in fp32 and in double (both sides of a parity test then take identical
    threshold decisions along the whole chain).
    """
    g = rng(seed)
    layers = []
    size = {1: hin}                                    # input size of each stage's stride-1 layers
    for st in (2, 3, 4):
        size[st] = (size[st - 1] + 2 - 3) // 2 + 1     # after the stage's 3x3 stride-2 conv (1x1 stride 2 gives the same)
    for (name, cin, cout, k, stride, pad, _) in resnet18_ternary_layers():
        st = int(name[5])
        h = size[st - 1] if stride == 2 else size[st]
        w = weight_codes(g, (cout, cin, k, k), p_zero)
        if dyadic:
            w_s = (g.integers(2, 7, cout) / 4.0).astype(np.float32)
            w_o = (g.integers(-2, 3, cout) / 16.0).astype(np.float32)
            a_s, a_o = 0.75, 0.125
        else:
            w_s, w_o = uniform(g, 0.5, 1.5, (cout,)), uniform(g, -0.1, 0.1, (cout,))
            a_s, a_o = float(uniform(g, 0.5, 1.5)), float(uniform(g, -0.1, 0.1))
        K = cin * k * k
        sigma = float(a_s * np.mean(w_s) * np.sqrt(K * 0.5 * (1.0 - p_zero)))
        layers.append(BodyLayer(name, cin, cout, k, stride, pad, h, w, a_s, a_o, w_s, w_o,
                                np.zeros(1, np.float32), np.ones(1, np.float32), sigma))
    return layers


def set_thresholds(layer, sigma, dyadic=False):
    lo, hi = 0.3 * sigma, 1.0 * sigma
    if dyadic:
        lo, hi = np.round(lo * 4) / 4, np.round(hi * 4) / 4
    layer.t_lo = np.array([lo], np.float32)
    layer.t_hi = np.array([hi], np.float32)


def resnet18_body_blocks(layers, sigma_in=1.0, dyadic=False):
    """Groups the 19 layers into the 8 residual blocks and sets every layer's input thresholds.
    Returns a list of dicts {conv1, conv2, down (or None)}; sigma_in is the scale of the body's fp32
    input (the stem's max-pooled output; max(0, N(0,1)) in the synthetic workload)."""
    by_name = {l.name: l for l in layers}
    blocks = []
    sigma_stream = sigma_in
    for s in (1, 2, 3, 4):
        for b in (0, 1):
            c1, c2 = by_name[f"layer{s}.{b}.conv1"], by_name[f"layer{s}.{b}.conv2"]
            down = by_name.get(f"layer{s}.{b}.downsample.0")
            set_thresholds(c1, sigma_stream, dyadic)            # ternarizer of the block's input
            if down is not None:
                set_thresholds(down, sigma_stream, dyadic)
            set_thresholds(c2, 0.6 * c1.sigma_out, dyadic)      # input = relu(conv1): about 0.6 sigma
            skip_sigma = 0.6 * down.sigma_out if down is not None else sigma_stream
            sigma_stream = float(np.sqrt((0.6 * c2.sigma_out) ** 2 + skip_sigma ** 2))
            blocks.append({"conv1": c1, "conv2": c2, "down": down})
    return blocks
