"""The ternary body of ResNet-18 (the 19 ternary conv layers of the paper's appendix table) as a
chain of library calls: every layer hands its result to the next one from its epilogue, as packed
pixel rows where the consumer is a ternary layer and as fp32 where the residual stream needs it.

Sequencing and argument marshalling only; every layer runs in the library's kernels.

Block (reading of the paper's "Layer Order" appendix, whose figure is lost: BN sits after the ReLU,
so each layer's BN folds into the thresholds of the ternarizer in front of it):

    s (fp32 residual stream), p = codes of s against conv1's thresholds
    q      = codes of relu(conv1(p))            against conv2's thresholds      [packed only]
    skip   = s, or relu(down(codes of s against down's thresholds)) in a stage's first block
    s_next = relu(conv2(q)) + skip                                            [fp32]
    p_next = codes of s_next against the next block's conv1 thresholds        [packed]
"""
import numpy as np
import torch

from . import binding as rtn


class Body:
    """Device-resident parameters and buffers of the chain for one batch size."""

    def __init__(self, blocks, batch, pad_mode=rtn.PAD_CODE_ZERO):
        self.blocks, self.B, self.pad_mode = blocks, batch, pad_mode
        dev = lambda a: torch.from_numpy(np.ascontiguousarray(a)).cuda()
        self.d = {}
        for blk in blocks:
            for l in (blk["conv1"], blk["conv2"], blk["down"]):
                if l is None:
                    continue
                wp, ws = rtn.rtn_pack_weights(dev(l.w_codes))
                self.d[l.name] = dict(wp=wp, ws=ws, w_s=dev(l.w_scale), w_o=dev(l.w_offset),
                                      t_lo=dev(l.t_lo), t_hi=dev(l.t_hi))
        # buffers: residual stream (two, alternating), skip of a downsampling block, packed rows
        self.bufs = []
        for blk in blocks:
            c1, c2 = blk["conv1"], blk["conv2"]
            ho = rtn.rtn_conv_out_dim(c1.hin, c1.k, c1.stride, c1.pad)
            e = {}
            e["q"] = torch.empty((batch * ho * ho, rtn.rtn_packed_row_bytes(c1.cout)), dtype=torch.uint8, device="cuda")
            e["s_next"] = torch.empty((batch, c2.cout, ho, ho), dtype=torch.float32, device="cuda")
            e["p_next"] = torch.empty((batch * ho * ho, rtn.rtn_packed_row_bytes(c2.cout)), dtype=torch.uint8, device="cuda")
            e["skip"] = (torch.empty((batch, c2.cout, ho, ho), dtype=torch.float32, device="cuda")
                         if blk["down"] is not None else None)
            self.bufs.append(e)
        self.launches = 0

    def _args(self, l):
        d = self.d[l.name]
        return (d["wp"], d["ws"], l.cout, l.k, l.k, l.stride, l.pad, self.pad_mode, l.a_scale, l.a_offset,
                d["w_s"], d["w_o"])

    def forward(self, s, dbg=None):
        """s: fp32 [B, 64, H, H] (the stem's output).  Returns (final residual stream fp32, per-block
        packed rows p_next) -- the last block's p_next uses its own conv1 thresholds as a stand-in for
        the classifier's (full-precision) input and is not consumed.  dbg: optional dict, layer name ->
        int32 tensor of the layer's output shape that receives the raw S_xw (the entry points' dbg_acc)."""
        acc = (lambda l: None) if dbg is None else (lambda l: dbg.get(l.name))
        p = None
        for i, blk in enumerate(self.blocks):
            c1, c2, down, e = blk["conv1"], blk["conv2"], blk["down"], self.bufs[i]
            n2 = self.d[c2.name]
            if p is None:       # the body's first layer ternarizes the fp32 stream itself
                d1 = self.d[c1.name]
                rtn.rtn_ternary_conv2d_fused(s, d1["t_lo"], d1["t_hi"], *self._args(c1), relu=True,
                                             next_t_lo=n2["t_lo"], next_t_hi=n2["t_hi"], out_packed=e["q"],
                                             dbg_acc=acc(c1))
            else:
                rtn.rtn_ternary_conv2d_packed(p, self.B, c1.cin, c1.hin, c1.hin, *self._args(c1), relu=True,
                                              next_t_lo=n2["t_lo"], next_t_hi=n2["t_hi"], out_packed=e["q"],
                                              dbg_acc=acc(c1))
            skip = s
            if down is not None:
                dd = self.d[down.name]
                rtn.rtn_ternary_conv2d_fused(s, dd["t_lo"], dd["t_hi"], *self._args(down), relu=True, out=e["skip"],
                                             dbg_acc=acc(down))
                skip = e["skip"]
            nxt = self.blocks[i + 1]["conv1"] if i + 1 < len(self.blocks) else c1
            nn = self.d[nxt.name]
            rtn.rtn_ternary_conv2d_packed(e["q"], self.B, c2.cin, c2.hin, c2.hin, *self._args(c2), relu=True,
                                          skip=skip, out=e["s_next"], next_t_lo=nn["t_lo"], next_t_hi=nn["t_hi"],
                                          out_packed=e["p_next"], dbg_acc=acc(c2))
            s, p = e["s_next"], e["p_next"]
        return s, [e["p_next"] for e in self.bufs]

    def layers(self):
        return [l for blk in self.blocks for l in (blk["conv1"], blk["conv2"], blk["down"]) if l is not None]

    def kernel_launches(self):
        """Kernel launches of one forward pass."""
        return sum(rtn.rtn_conv_next_kernel_launches(self.B, l.cin, l.hin, l.hin, l.cout, l.k, l.k, l.stride, l.pad)
                   for l in self.layers())

    def algorithmic_bytes(self):
        """Bytes one forward pass must move: per layer its input once (packed rows; fp32 where the layer
        ternarizes the residual stream itself), its outputs once (packed rows and / or fp32), the skip it adds,
        and its packed filters."""
        rb = rtn.rtn_packed_row_bytes
        total = 0
        for i, blk in enumerate(self.blocks):
            c1, c2, down = blk["conv1"], blk["conv2"], blk["down"]
            ho = rtn.rtn_conv_out_dim(c1.hin, c1.k, c1.stride, c1.pad)
            px_in, px_out = self.B * c1.hin * c1.hin, self.B * ho * ho
            total += (4 * c1.cin if i == 0 else rb(c1.cin)) * px_in + rb(c1.cout) * px_out      # conv1
            total += rb(c2.cin) * px_out + (4 * c2.cout + 4 * c2.cout + rb(c2.cout)) * px_out    # conv2: q in; skip in, s out, p out
            if down is not None:
                total += 4 * down.cin * (px_in // (down.stride * down.stride)) + 4 * down.cout * px_out
            for l in (c1, c2, down):
                if l is not None:
                    total += l.cout * rb(rtn.rtn_conv_packed_k(l.cin, l.k, l.k))
        return total

    def ops(self):
        """2*M*N*K summed over the 19 layers for this batch."""
        total = 0.0
        for blk in self.blocks:
            for l in (blk["conv1"], blk["conv2"], blk["down"]):
                if l is None:
                    continue
                ho = rtn.rtn_conv_out_dim(l.hin, l.k, l.stride, l.pad)
                total += 2.0 * self.B * ho * ho * l.cout * l.cin * l.k * l.k
        return total
