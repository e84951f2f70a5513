"""GPU parity of the ResNet-18-shaped stack of encoded convolutions (W4A4) against the CPU oracle.

The oracle runs the whole network on its own from the raw input: the fp32 stem and max-pool (glue,
defined as one fused-multiply-add chain per output, so bit-exact), then the chain of encoded layers
(range -> quantize -> integer convolution -> scale, residual add + max in fp32); every layer must
agree: int32 accumulators bit-exact, fp32 outputs within 1e-5 relative.  The small case is compared
element by element through the whole chain.  At full size (batch 128, 224 x 224) the oracle cannot
run the chain (2.2e11 multiply-adds), so the stem + max-pool are compared in full and every encoded
layer on sampled outputs that the oracle computes one by one from that layer's input on the device.
"""
import numpy as np
import pytest
import torch

import oracle
from paper_1905_13389_b200 import inputs
from paper_1905_13389_b200.resnet18 import BLOCKS, QuantResNet18Stack
from tests._util import rel_close

pytestmark = pytest.mark.gpu


def test_stem_and_maxpool_against_float64(mpq, cuda):
    x = inputs.config5_input(2, 70)                        # odd output size 35 -> ragged tiles
    w = inputs.config5_weights()["conv1"]
    y = mpq.stem_conv7x7(torch.from_numpy(x).to(cuda), torch.from_numpy(w).to(cuda), relu=False)
    ref = torch.nn.functional.conv2d(torch.from_numpy(x).double(), torch.from_numpy(w).double(), stride=2, padding=3)
    assert tuple(y.shape) == tuple(ref.shape) == (2, 64, 35, 35)
    err = (y.cpu().double() - ref).abs().max().item()
    assert err <= 1e-5 * ref.abs().max().item()            # 147-term fp32 sums against float64
    assert np.array_equal(y.cpu().numpy(), oracle.stem(x, w, relu=False))   # same fma chain: same bits
    yr = mpq.stem_conv7x7(torch.from_numpy(x).to(cuda), torch.from_numpy(w).to(cuda), relu=True)
    assert torch.equal(yr, torch.clamp_min(y, 0))
    p = mpq.maxpool3x3s2(yr)
    assert torch.equal(p.cpu(), torch.nn.functional.max_pool2d(yr.cpu(), 3, 2, 1))


def _oracle_block(x, ws, blk, stride, has_ds, a_bits, w_bits):
    """One basic block on the CPU; returns {conv name: (acc, out)} and the block output."""
    res = {}
    acc1, t, _, _ = oracle.conv_layer(x, ws[blk + ".conv1"], a_bits, w_bits, stride, 1, True, oracle.HRELU)
    res[blk + ".conv1"] = (acc1, t)
    acc2, u, _, _ = oracle.conv_layer(t, ws[blk + ".conv2"], a_bits, w_bits, 1, 1, True, oracle.HRELU)
    res[blk + ".conv2"] = (acc2, u)
    if has_ds:
        accd, sc, _, _ = oracle.conv_layer(x, ws[blk + ".downsample"], a_bits, w_bits, stride, 0, True, oracle.HRELU)
        res[blk + ".downsample"] = (accd, sc)
    else:
        sc = x
    return res, np.maximum(u + sc, np.float32(0))


@pytest.mark.parametrize("fused", [False, True])
@pytest.mark.parametrize("a_bits,w_bits", [(4, 4), (2, 3)])
def test_stack_small_chain_elementwise(mpq, cuda, a_bits, w_bits, fused):
    """fused=False: range, encode, conv, add as separate kernels; fused=True: residual add, max(.,0)
    and the next encoder's range folded into the convolutions' stores.  Same results either way."""
    batch, size = 2, 64
    ws = inputs.config5_weights()
    x = inputs.config5_input(batch, size)
    net = QuantResNet18Stack(ws, batch, size, a_bits, w_bits, cuda, keep_int32=True, fused=fused)
    out = net.forward(torch.from_numpy(x).to(cuda))
    torch.cuda.synchronize()
    cur = oracle.maxpool3x3s2(oracle.stem(x, ws["conv1"]))  # the oracle's own chain, from the raw input
    assert cur.shape == (batch, 64, 16, 16) and cur.min() >= 0 and cur.max() > 0
    assert np.array_equal(net.pooled.cpu().numpy(), cur)
    for blk, _, _, stride, has_ds in BLOCKS:
        res, cur = _oracle_block(cur, ws, blk, stride, has_ds, a_bits, w_bits)
        for name, (acc, ref) in res.items():
            assert np.array_equal(net.y_i32[name].cpu().numpy(), acc), name
            if not (fused and name.endswith("conv2")):      # fused: conv2 stores the block output only
                assert rel_close(net.y[name].cpu().numpy(), ref), name
        assert np.array_equal(net.block_out[blk].cpu().numpy(), cur), blk
        assert np.unique(res[blk + ".conv2"][0]).size > 16
    assert np.array_equal(out.cpu().numpy(), cur)


def test_stack_full_size_sampled(mpq, cuda):
    """Batch 128 at 224 x 224 in W4A4: every encoded layer, in the launch configuration that is
    timed, on 40 sampled outputs (image corners and borders included) computed one by one."""
    batch, size, a_bits, w_bits = 128, 224, 4, 4
    ws = inputs.config5_weights()
    net = QuantResNet18Stack(ws, batch, size, a_bits, w_bits, cuda, keep_int32=True, fused=True)
    x = inputs.config5_input(batch, size)
    net.forward(torch.from_numpy(x).to(cuda))
    torch.cuda.synchronize()
    assert np.array_equal(net.pooled.cpu().numpy(), oracle.maxpool3x3s2(oracle.stem(x, ws["conv1"])))
    rng = np.random.default_rng(5)
    layer_in = net.pooled
    for blk, _, _, stride, has_ds in BLOCKS:
        jobs = [(blk + ".conv1", layer_in), (blk + ".conv2", net.y[blk + ".conv1"])]
        if has_ds:
            jobs.append((blk + ".downsample", layer_in))
        shortcut = (net.y[blk + ".downsample"] if has_ds else layer_in).cpu().numpy()
        for name, xin in jobs:
            conv = net.convs[name]
            x = xin.cpu().numpy()
            s_a = oracle.absmax(x, False, oracle.HRELU)
            assert np.array_equal(net.x_scale[name if "downsample" not in name else blk + ".conv1"].cpu().numpy(), s_a)
            s_w = oracle.absmax(ws[name], True)
            qx = oracle.quantize(x, s_a, a_bits, act=oracle.HRELU)
            qw = oracle.quantize(ws[name], s_w, w_bits, per_row=True)
            yi = net.y_i32[name].cpu().numpy()
            is_conv2 = name.endswith("conv2")            # fused: stored as max(conv + shortcut, 0) in the block output
            yf = (net.block_out[blk] if is_conv2 else net.y[name]).cpu().numpy()
            _, O, Ho, Wo = yi.shape
            pts = [(0, 0, 0, 0), (batch - 1, O - 1, Ho - 1, Wo - 1), (1, 1, 0, Wo - 1), (2, O // 2, Ho - 1, 0)]
            pts += [tuple(int(v) for v in (rng.integers(batch), rng.integers(O), rng.integers(Ho), rng.integers(Wo)))
                    for _ in range(36)]
            for (b, o, oh, ow) in pts:
                acc = oracle.conv_at(qx, qw, conv.stride, conv.pad, b, o, oh, ow)
                assert int(yi[b, o, oh, ow]) == acc, (name, b, o, oh, ow)
                ref = oracle.scale(np.array([[acc]], np.int32), s_a[0], s_w[o:o + 1], a_bits, w_bits)[0, 0]
                if is_conv2:
                    ref = max(np.float32(ref) + shortcut[b, o, oh, ow], np.float32(0))
                assert abs(float(yf[b, o, oh, ow]) - float(ref)) <= 1e-5 * abs(float(ref)), (name, b, o, oh, ow)
        layer_in = net.block_out[blk]


def test_stack_repeated_forwards_are_identical(mpq, cuda):
    """Back-to-back forwards on one stream (ranges are re-zeroed and re-raised every time, kernels of
    consecutive forwards overlap at their edges): outputs and ranges repeat bit for bit."""
    batch, size = 8, 96
    net = QuantResNet18Stack(inputs.config5_weights(), batch, size, 4, 4, cuda, fused=True)
    x = torch.from_numpy(inputs.config5_input(batch, size)).to(cuda)
    first = net.forward(x).clone()
    scales = net.scales.clone()
    for _ in range(20):
        out = net.forward(x)
    torch.cuda.synchronize()
    assert torch.equal(out, first) and torch.equal(net.scales, scales)
    assert float(scales.min()) > 0


@pytest.mark.parametrize("a_bits,w_bits", [(4, 4), (3, 5)])
def test_stack_static_ranges_write_planes_from_the_store(mpq, cuda, a_bits, w_bits):
    """Ranges fixed before the network runs (here: calibrated on the same batch, so the codes must be
    the dynamic run's): every convolution writes its consumer's packed planes from its store, there is
    no encode pass after the first one and no fp32 tensor between conv1 and conv2 -- and the output,
    every accumulator and every plane word equal the dynamic run's, which the oracle pins."""
    batch, size = 2, 64
    ws = inputs.config5_weights()
    x = torch.from_numpy(inputs.config5_input(batch, size)).to(cuda)
    dyn = QuantResNet18Stack(ws, batch, size, a_bits, w_bits, cuda, keep_int32=True, fused=True)
    ref = dyn.forward(x).clone()
    torch.cuda.synchronize()
    ranges = dyn.calibrated_ranges()
    assert len(ranges) == 16 and min(ranges.values()) > 0
    net = QuantResNet18Stack(ws, batch, size, a_bits, w_bits, cuda, keep_int32=True, static_ranges=ranges)
    for t in net.y.values():
        t.fill_(float("nan"))                                 # nothing may depend on the fp32 intermediates
    out = net.forward(x)
    torch.cuda.synchronize()
    assert torch.equal(out, ref)
    for name in dyn.y_i32:
        assert torch.equal(net.y_i32[name], dyn.y_i32[name]), name
    for name in dyn.x_planes:
        assert torch.equal(net.x_planes[name], dyn.x_planes[name]), name
    for blk, _, _, _, _ in BLOCKS:
        assert bool(torch.isnan(net.y[blk + ".conv1"]).all())  # conv1 -> conv2 went through planes only
    # the paper's own setting: one fixed range for every encoder (HReLU to [0, s]); the chain still
    # equals the oracle's chain with that range, block by block
    fixed = {n: 2.0 for n in ranges}
    net2 = QuantResNet18Stack(ws, batch, size, a_bits, w_bits, cuda, keep_int32=True, static_ranges=fixed)
    out2 = net2.forward(x).cpu().numpy()
    cur = net2.pooled.cpu().numpy()
    s = np.array([2.0], np.float32)
    for blk, _, _, stride, has_ds in BLOCKS:
        qx = oracle.quantize(cur, s, a_bits, act=oracle.HRELU)
        def conv(name, q, st, pad):
            s_w = oracle.absmax(ws[name], True)
            acc = oracle.conv(q, oracle.quantize(ws[name], s_w, w_bits, per_row=True), st, pad)
            assert np.array_equal(net2.y_i32[name].cpu().numpy(), acc), name
            return oracle.scale(acc, s[0], s_w, a_bits, w_bits)
        t = conv(blk + ".conv1", qx, stride, 1)
        u = conv(blk + ".conv2", oracle.quantize(t, s, a_bits, act=oracle.HRELU), 1, 1)
        sc = conv(blk + ".downsample", qx, stride, 0) if has_ds else cur
        cur = oracle.epilogue(u, None, sc, True)
    assert np.array_equal(out2, cur)
