"""ResNet-18-shaped stack of encoded convolutions (driver; every step runs in libmpq's kernels).

The network shape is the one the paper's ImageNet experiments name (Section 5): a 7x7 stride-2
stem and a 3x3 max-pool, then four stages of two basic blocks (64, 128, 256, 512 channels), the
first block of stages 2-4 strided with a 1x1 stride-2 shortcut convolution.  The stem stays
fp32 (first layer kept in full precision); the 19 convolutions after it are encoded layers:

    range (HReLU: max of the positive side) -> encode_nchw -> conv on packed planes (+ scale)

There is no batch normalisation and no bias; a block computes
    out = max(conv2(max(conv1(x), 0)) + shortcut(x), 0)
where the inner max(.,0) is the HReLU range limiter of conv2's encoder (Table 1) and the outer
one is a single fp32 add + max.  Weights are encoded once, at construction, with one range per
output channel.  All buffers are allocated at construction; ``forward`` only launches kernels
on the current stream and never synchronises.

With ``static_ranges`` (a dict: encoded convolution name -> range of its input encoder) the ranges
are fixed before the network runs -- the paper's own setting, where HReLU limits every activation
to a known interval (Table 1), or constants calibrated on sample data with ``calibrated_ranges``.
Then every convolution also runs its consumer's Encoder in its store and writes the packed planes
directly: a block is  conv, conv (+ shortcut conv)  with no encode pass and no fp32 tensor between
conv1 and conv2; the block output is still stored in fp32 where the next block adds it as shortcut.

With ``fused=True`` (the default) the glue rides in the convolutions' stores: conv2 adds the
shortcut and applies max(.,0) itself, and every producer (max-pool, conv1, conv2) raises the
range of the encoder that consumes it, so a block is  encode, conv, encode, conv (+ shortcut
conv)  with no separate range or add kernels.  ``fused=False`` runs range, encode, conv and
add as separate kernels; both give bit-identical results.
"""
from __future__ import annotations

from typing import Dict, List, Optional, Tuple

import numpy as np
import torch

from . import binding as mpq

# (name, C_in, C_out, kernel, stride) of the encoded convolutions, in execution order per block:
# conv1, conv2, then the shortcut convolution when the block has one.
BLOCKS = [
    ("layer1.0", 64, 64, 1, False), ("layer1.1", 64, 64, 1, False),
    ("layer2.0", 64, 128, 2, True), ("layer2.1", 128, 128, 1, False),
    ("layer3.0", 128, 256, 2, True), ("layer3.1", 256, 256, 1, False),
    ("layer4.0", 256, 512, 2, True), ("layer4.1", 512, 512, 1, False),
]


class _QConv:
    """One encoded convolution: pre-encoded weights and its output buffer."""

    def __init__(self, name, w: torch.Tensor, w_bits: int, stride: int, pad: int):
        self.name = name
        self.O, self.C, self.KH, self.KW = w.shape
        self.stride, self.pad, self.w_bits = stride, pad, w_bits
        self.w_scale = mpq.absmax(w, mpq.SCALE_PER_ROW)
        self.w_planes, self.tap_sums = mpq.encode_oihw(w, self.w_scale, w_bits, mpq.SCALE_PER_ROW)

    def out_hw(self, H, W):
        return ((H + 2 * self.pad - self.KH) // self.stride + 1, (W + 2 * self.pad - self.KW) // self.stride + 1)


class QuantResNet18Stack:
    def __init__(self, weights: Dict[str, np.ndarray], batch: int, size: int = 224,
                 a_bits: int = 4, w_bits: int = 4, device: Optional[torch.device] = None,
                 keep_int32: bool = False, fused: bool = True,
                 static_ranges: Optional[Dict[str, float]] = None):
        dev = device or torch.device("cuda", torch.cuda.current_device())
        self.dev, self.batch, self.size, self.a_bits, self.w_bits = dev, batch, size, a_bits, w_bits
        self.keep_int32 = keep_int32
        self.fused = fused
        up = lambda a: torch.from_numpy(np.ascontiguousarray(a)).to(dev)
        self.stem_w = up(weights["conv1"])
        self.convs: Dict[str, _QConv] = {}
        for blk, cin, cout, stride, has_ds in BLOCKS:
            self.convs[blk + ".conv1"] = _QConv(blk + ".conv1", up(weights[blk + ".conv1"]), w_bits, stride, 1)
            self.convs[blk + ".conv2"] = _QConv(blk + ".conv2", up(weights[blk + ".conv2"]), w_bits, 1, 1)
            if has_ds:
                self.convs[blk + ".downsample"] = _QConv(blk + ".downsample", up(weights[blk + ".downsample"]),
                                                         w_bits, stride, 0)
        f32 = lambda *shape: torch.empty(shape, dtype=torch.float32, device=dev)
        h1 = (size - 1) // 2 + 1
        h2 = (h1 - 1) // 2 + 1
        self.stem_out = f32(batch, 64, h1, h1)
        self.pooled = f32(batch, 64, h2, h2)
        # per-convolution buffers: range, packed input planes, fp32 output (and int32 when asked)
        self.scales = f32(2 * len(BLOCKS))          # one range per encoder, contiguous: zeroed once per forward
        self.x_scale: Dict[str, torch.Tensor] = {}
        self.x_planes: Dict[str, torch.Tensor] = {}
        self.y: Dict[str, torch.Tensor] = {}
        self.y_i32: Dict[str, torch.Tensor] = {}
        self.block_out: Dict[str, torch.Tensor] = {}
        self.in_shape: Dict[str, Tuple[int, int, int]] = {}
        H = h2
        for blk, cin, cout, stride, has_ds in BLOCKS:
            c1, c2 = self.convs[blk + ".conv1"], self.convs[blk + ".conv2"]
            Ho, _ = c1.out_hw(H, H)
            for name, C, Hin, conv in ((blk + ".conv1", cin, H, c1), (blk + ".conv2", cout, Ho, c2)):
                self.x_scale[name] = self.scales[len(self.x_scale):len(self.x_scale) + 1]
                self.x_planes[name] = torch.empty((a_bits, batch, Hin, Hin, C // 32), dtype=torch.int32, device=dev)
                oh, _ = conv.out_hw(Hin, Hin)
                self.y[name] = f32(batch, conv.O, oh, oh)
                self.in_shape[name] = (C, Hin, Hin)
                if keep_int32:
                    self.y_i32[name] = torch.empty((batch, conv.O, oh, oh), dtype=torch.int32, device=dev)
            if has_ds:
                name = blk + ".downsample"
                self.y[name] = f32(batch, cout, Ho, Ho)
                self.in_shape[name] = (cin, H, H)
                if keep_int32:
                    self.y_i32[name] = torch.empty((batch, cout, Ho, Ho), dtype=torch.int32, device=dev)
            self.block_out[blk] = f32(batch, cout, Ho, Ho)
            H = Ho
        self.static = static_ranges is not None
        if self.static:
            missing = [n for n in self.x_scale if n not in static_ranges]
            if missing:
                raise ValueError("static_ranges lacks %s" % ", ".join(missing))
            host = torch.tensor([float(static_ranges[n]) for n in self.x_scale], dtype=torch.float32)
            self.scales.copy_(host.to(dev))                # x_scale[name] are views of this tensor, in this order
        self.layer_names: List[str] = ["stem", "maxpool"]
        for blk, _, _, _, has_ds in BLOCKS:
            self.layer_names += [blk + ".conv1", blk + ".conv2"] + ([blk + ".downsample"] if has_ds else [])

    # -- one encoded convolution on planes that are already packed ------------------------------
    def _conv(self, name: str, planes: torch.Tensor, scale: torch.Tensor):
        c = self.convs[name]
        C, H, W = self.in_shape[name]
        mpq.conv(planes, self.a_bits, self.batch, C, H, W, c.w_planes, self.w_bits, c.tap_sums,
                 c.O, c.KH, c.KW, c.stride, c.pad, self.y_i32.get(name), self.y[name],
                 scale, c.w_scale, mpq.SCALE_PER_ROW)
        return self.y[name]

    def _encode(self, name: str, x: torch.Tensor):
        s = mpq.absmax(x, mpq.SCALE_PER_TENSOR, mpq.ACT_HRELU, out=self.x_scale[name])
        p = mpq.encode_nchw(x, s, self.a_bits, mpq.ACT_HRELU, out=self.x_planes[name])
        return p, s

    def forward(self, x: torch.Tensor, events: Optional[dict] = None) -> torch.Tensor:
        """x [batch][3][size][size] fp32 on the device -> output of the last block, fp32.
        With ``events`` (a dict), CUDA events are recorded around every layer:
        events[name] = (start, end); an encoded layer's span covers its (range +) encode + conv
        (the shortcut convolution reuses conv1's packed input, so its span is the conv alone)."""
        def span(name, fn):
            if events is None:
                return fn()
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record()
            r = fn()
            e1.record()
            events[name] = (e0, e1)
            return r

        if self.static:
            return self._forward_static(x, span)
        if self.fused:
            return self._forward_fused(x, span)
        span("stem", lambda: mpq.stem_conv7x7(x, self.stem_w, True, out=self.stem_out))
        cur = span("maxpool", lambda: mpq.maxpool3x3s2(self.stem_out, out=self.pooled))
        for blk, cin, cout, stride, has_ds in BLOCKS:
            n1, n2, nd = blk + ".conv1", blk + ".conv2", blk + ".downsample"
            enc = {}

            def first():
                enc["p"], enc["s"] = self._encode(n1, cur)
                return self._conv(n1, enc["p"], enc["s"])
            t = span(n1, first)

            def second():
                p, s = self._encode(n2, t)
                return self._conv(n2, p, s)
            u = span(n2, second)
            shortcut = span(nd, lambda: self._conv(nd, enc["p"], enc["s"])) if has_ds else cur
            cur = span(blk + ".add_relu", lambda: mpq.add_relu(u, shortcut, self.block_out[blk]))
        return cur

    def _conv_fused(self, name, planes, scale, out, residual, relu, out_max):
        c = self.convs[name]
        C, H, W = self.in_shape[name]
        mpq.conv_fused(planes, self.a_bits, self.batch, C, H, W, c.w_planes, self.w_bits, c.tap_sums,
                       c.O, c.KH, c.KW, c.stride, c.pad, self.y_i32.get(name), out,
                       scale, c.w_scale, mpq.SCALE_PER_ROW, residual, relu, out_max)
        return out

    def _forward_fused(self, x, span):
        mpq.zero(self.scales)
        span("stem", lambda: mpq.stem_conv7x7(x, self.stem_w, True, out=self.stem_out))
        first_scale = self.x_scale[BLOCKS[0][0] + ".conv1"]
        cur = span("maxpool", lambda: mpq.maxpool3x3s2(self.stem_out, out=self.pooled, out_max=first_scale))
        for bi, (blk, cin, cout, stride, has_ds) in enumerate(BLOCKS):
            n1, n2, nd = blk + ".conv1", blk + ".conv2", blk + ".downsample"
            s1, s2 = self.x_scale[n1], self.x_scale[n2]
            next_scale = self.x_scale[BLOCKS[bi + 1][0] + ".conv1"] if bi + 1 < len(BLOCKS) else None
            enc = {}

            def first():
                enc["p"] = mpq.encode_nchw(cur, s1, self.a_bits, mpq.ACT_HRELU, out=self.x_planes[n1])
                return self._conv_fused(n1, enc["p"], s1, self.y[n1], None, False, s2)
            t = span(n1, first)
            shortcut = span(nd, lambda: self._conv_fused(nd, enc["p"], s1, self.y[nd], None, False, None)) if has_ds else cur

            def second():
                p = mpq.encode_nchw(t, s2, self.a_bits, mpq.ACT_HRELU, out=self.x_planes[n2])
                return self._conv_fused(n2, p, s2, self.block_out[blk], shortcut, True, next_scale)
            cur = span(n2, second)
        return cur

    def calibrated_ranges(self) -> Dict[str, float]:
        """The ranges the encoders saw in the last (non-static) forward, as ``static_ranges`` input."""
        vals = self.scales.cpu().tolist()
        return {name: vals[i] for i, name in enumerate(self.x_scale)}

    def _conv_encoded(self, name, planes, scale, out, residual, relu, next_name):
        """Convolution `name`; with `next_name` its store also writes that consumer's packed planes."""
        c = self.convs[name]
        C, H, W = self.in_shape[name]
        if next_name is None:
            mpq.conv_fused(planes, self.a_bits, self.batch, C, H, W, c.w_planes, self.w_bits, c.tap_sums,
                           c.O, c.KH, c.KW, c.stride, c.pad, self.y_i32.get(name), out,
                           scale, c.w_scale, mpq.SCALE_PER_ROW, residual, relu, None)
        else:
            mpq.conv_encoded(planes, self.a_bits, self.batch, C, H, W, c.w_planes, self.w_bits, c.tap_sums,
                             c.O, c.KH, c.KW, c.stride, c.pad, self.y_i32.get(name), out,
                             scale, c.w_scale, mpq.SCALE_PER_ROW, residual, relu, None,
                             self.x_scale[next_name], mpq.ACT_HRELU, self.a_bits, self.x_planes[next_name])
        return out

    def _forward_static(self, x, span):
        span("stem", lambda: mpq.stem_conv7x7(x, self.stem_w, True, out=self.stem_out))
        cur = span("maxpool", lambda: mpq.maxpool3x3s2(self.stem_out, out=self.pooled))
        first = BLOCKS[0][0] + ".conv1"
        span("encode", lambda: mpq.encode_nchw(cur, self.x_scale[first], self.a_bits, mpq.ACT_HRELU, out=self.x_planes[first]))
        for bi, (blk, cin, cout, stride, has_ds) in enumerate(BLOCKS):
            n1, n2, nd = blk + ".conv1", blk + ".conv2", blk + ".downsample"
            last = bi + 1 == len(BLOCKS)
            next_n1 = None if last else BLOCKS[bi + 1][0] + ".conv1"
            next_has_ds = (not last) and BLOCKS[bi + 1][4]
            # conv1 feeds conv2 only: no fp32 tensor, just conv2's planes
            span(n1, lambda: self._conv_encoded(n1, self.x_planes[n1], self.x_scale[n1], None, None, False, n2))
            shortcut = span(nd, lambda: self._conv_encoded(nd, self.x_planes[n1], self.x_scale[n1], self.y[nd], None, False, None)) \
                if has_ds else cur
            # conv2 adds the shortcut, applies max(.,0) and writes the next block's planes; its fp32 output is
            # kept only where somebody adds it later (the next block's shortcut) or reads it (the last block)
            keep = last or not next_has_ds
            out = self.block_out[blk] if keep else None
            span(n2, lambda: self._conv_encoded(n2, self.x_planes[n2], self.x_scale[n2], out, shortcut, True, next_n1))
            cur = self.block_out[blk]
        return cur
