"""Per-workload measurements behind ``bench.py --full FILE``: the five synthetic workloads
(single small GEMM, fully-connected layer, 3x3 convolution, bit-width sweep, ResNet-18-shaped
stack) and the encoders, each timed with CUDA events on the launching stream after warm-up.
Everything goes through the C ABI binding; nothing here touches the CPU oracle."""
from __future__ import annotations

import json
import statistics

import numpy as np
import torch

from paper_1905_13389_b200 import binding as mpq
from paper_1905_13389_b200 import context, inputs
from paper_1905_13389_b200.resnet18 import QuantResNet18Stack


def _events_ms(fn, iters=20, warmup=5):
    for _ in range(warmup):
        fn()
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(iters):
        fn()
    e1.record()
    torch.cuda.synchronize()
    return e0.elapsed_time(e1) / iters


def _graph_ms(fn, iters=20, warmup=5):
    """Short kernels: replay `iters` launches from one CUDA graph so that host launch cost
    (ctypes marshalling, ~10 us per call) does not sit between the kernels being timed."""
    for _ in range(warmup):
        fn()
    torch.cuda.synchronize()
    g = torch.cuda.CUDAGraph()
    st = torch.cuda.Stream()
    with torch.cuda.stream(st):
        with torch.cuda.graph(g, stream=st):
            for _ in range(iters):
                fn()
    g.replay()
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    g.replay()
    e1.record()
    torch.cuda.synchronize()
    return e0.elapsed_time(e1) / iters


def run_suite(dev: torch.device, hbm_gbs: float, path=None):
    """Times every workload; returns the figures as a dict and, when `path` is given, writes them there as JSON."""
    up = lambda a: torch.from_numpy(np.ascontiguousarray(a)).to(dev)
    popc_peak, mhz, sms = mpq.measure_popc_peak()
    mix, _, _ = mpq.measure_mix_peak(4)
    branch_peak = 2.0 * mix
    out = {"popc_peak_gpopc_s": popc_peak / 1e9, "branch_peak_gpopc_s": branch_peak / 1e9, "probe_sm_mhz": mhz,
           "hbm_gbs": hbm_gbs}

    def product_record(ms, m, n, k, a_bits, w_bits, popcs):
        return {"ms": ms, "equivalent_tops": 2.0 * m * n * k / (ms * 1e-3) / 1e12,
                "binary_tops": 2.0 * m * n * k * a_bits * w_bits / (ms * 1e-3) / 1e12,
                "gpopc_s": popcs / (ms * 1e-3) / 1e9, "frac_of_branch_peak": popcs / (ms * 1e-3) / branch_peak,
                "frac_of_plain_popc_peak": popcs / (ms * 1e-3) / popc_peak}

    # ---- workload 1: one small GEMM (launch-latency bound) --------------------------------------
    c = inputs.config1()
    x, w = up(c["x"]), up(c["w"])
    sa, sw = mpq.absmax(x, 0, mpq.ACT_HRELU), mpq.absmax(w)
    ap, wp = mpq.encode(x, sa, 2, 0, mpq.ACT_HRELU), mpq.encode(w, sw, 2)
    ci = torch.empty((64, 64), dtype=torch.int32, device=dev)
    cf = torch.empty((64, 64), dtype=torch.float32, device=dev)
    ms = _graph_ms(lambda: mpq.gemm(ap, 2, wp, 2, 64, 64, 512, ci, cf, sa, sw), 50)
    out["gemm_w2a2_64x64x512"] = {"us": ms * 1e3}

    # ---- workload 4: the bit-width sweep at 4096^3 ----------------------------------------------
    size = 4096
    c4 = inputs.config4(2, 2, size)
    x, w = up(c4["x"]), up(c4["w"])
    sa, sw = mpq.absmax(x, 0, mpq.ACT_HRELU), mpq.absmax(w)
    ci = torch.empty((size, size), dtype=torch.int32, device=dev)
    sweep = {}
    for (w_bits, a_bits) in inputs.SWEEP_BITS:
        ap, wp = mpq.encode(x, sa, a_bits, 0, mpq.ACT_HRELU), mpq.encode(w, sw, w_bits)
        ms = _events_ms(lambda: mpq.gemm(ap, a_bits, wp, w_bits, size, size, size, ci, None), 10, 3)
        sweep["w%da%d" % (w_bits, a_bits)] = product_record(ms, size, size, size, a_bits, w_bits,
                                                             float(a_bits * w_bits) * size * size * (size // 32))
    out["gemm_sweep_4096"] = sweep
    # context only, not this path: what a library int8 tensor-core GEMM of the same shape costs
    # (the product of the DECODED integers, which fit int8 up to 7 bits; cuBLASLt through torch)
    try:
        qa = torch.randint(-3, 4, (size, size), dtype=torch.int8, device=dev)
        qb = torch.randint(-3, 4, (size, size), dtype=torch.int8, device=dev)
        ms = _events_ms(lambda: torch._int_mm(qa, qb), 10, 3)
        out["context_library_int8_gemm_4096"] = {"ms": ms, "tops": 2.0 * size ** 3 / (ms * 1e-3) / 1e12,
                                                 "note": "decoded-integer product on the tensor cores (library kernel); "
                                                         "not the bit-plane path and not part of this library"}
        del qa, qb
    except Exception as exc:                                    # library kernel unavailable: the context line is dropped
        out["context_library_int8_gemm_4096"] = {"unavailable": str(exc)[:200]}
    # context only: this repository's own decoded-integer tensor-core kernel (tcgen05 kind::i8, TMA, TMEM) on the
    # same shape -- signed form (codes up to 7 bits) and unsigned form with Eq. 17's correction (8-bit codes)
    qa = torch.randint(-3, 4, (size, size), dtype=torch.int8, device=dev)
    qb = torch.randint(-3, 4, (size, size), dtype=torch.int8, device=dev)
    co = torch.empty((size, size), dtype=torch.int32, device=dev)
    err = torch.zeros(1, dtype=torch.int32, device=dev)
    ms = _events_ms(lambda: context.i8_gemm(qa, qb, co, err), 10, 3)
    ua = torch.randint(0, 256, (size, size), dtype=torch.uint8, device=dev)
    ub = torch.randint(0, 256, (size, size), dtype=torch.uint8, device=dev)
    sa8, sb8 = context.row_sums_u8(ua), context.row_sums_u8(ub)
    ms_u = _events_ms(lambda: context.i8_gemm(ua, ub, co, err, unsigned_levels=(255, 255), sums=(sa8, sb8)), 10, 3)
    out["context_own_tcgen05_i8_gemm_4096"] = {
        "signed_ms": ms, "signed_tops": 2.0 * size ** 3 / (ms * 1e-3) / 1e12,
        "unsigned_eq17_ms": ms_u, "unsigned_eq17_tops": 2.0 * size ** 3 / (ms_u * 1e-3) / 1e12,
        "bounded_wait_ran_out": int(err.cpu()[0]),
        "note": "decoded-integer product on the 5th-generation tensor cores, own kernel (persistent, 128 x 256 tile, two TMEM accumulators, "
                "no multicast); context for the bit-plane numbers, not part of the library"}
    del qa, qb, ua, ub, co

    # ---- encoders on the sweep's operands (64 MiB fp32 each; four buffers in rotation) ----------
    xs = [x, w, torch.randn_like(x), torch.randn_like(x)]
    enc = {}
    for bits in (1, 2, 3, 4, 8):
        planes = torch.empty((bits, size, mpq.row_words(size)), dtype=torch.int32, device=dev)
        i = [0]

        def f():
            mpq.encode(xs[i[0] % 4], sa, bits, 0, mpq.ACT_HTANH, out=planes)
            i[0] += 1
        ms = _graph_ms(f)
        by = size * size * (4 + bits / 8.0)
        enc["rows_4096x4096_b%d" % bits] = {"us": ms * 1e3, "gb_s": by / (ms * 1e-3) / 1e9,
                                            "frac_of_hbm": by / (ms * 1e-3) / 1e9 / hbm_gbs}
    i = [0]
    s1 = torch.empty(1, dtype=torch.float32, device=dev)

    def f():
        mpq.absmax(xs[i[0] % 4], out=s1)
        i[0] += 1
    ms = _graph_ms(f)
    enc["absmax_4096x4096"] = {"us": ms * 1e3, "gb_s": size * size * 4 / (ms * 1e-3) / 1e9,
                               "frac_of_hbm": size * size * 4 / (ms * 1e-3) / 1e9 / hbm_gbs}
    del xs, x, w

    # ---- workload 2: fully-connected layer W2A2 --------------------------------------------------
    c = inputs.config2()
    x, w = up(c["x"]), up(c["w"])
    m, n, k = c["m"], c["n"], c["k"]
    sa, sw = mpq.absmax(x, 0, mpq.ACT_HRELU), mpq.absmax(w, mpq.SCALE_PER_ROW)
    ap = mpq.encode(x, sa, 2, 0, mpq.ACT_HRELU)
    wp = torch.empty((2, n, mpq.row_words(k)), dtype=torch.int32, device=dev)
    w2 = w.clone()
    i = [0]

    def f():
        mpq.encode(w if i[0] % 2 == 0 else w2, sw, 2, mpq.SCALE_PER_ROW, out=wp)
        i[0] += 1
    ms_we = _graph_ms(f)
    by = n * k * 4.25
    cf = torch.empty((m, n), dtype=torch.float32, device=dev)
    ms = _graph_ms(lambda: mpq.gemm(ap, 2, wp, 2, m, n, k, None, cf, sa, sw, mpq.SCALE_PER_ROW))
    rec = product_record(ms, m, n, k, 2, 2, 4.0 * m * n * (k // 32))
    rec["weight_encode"] = {"us": ms_we * 1e3, "gb_s": by / (ms_we * 1e-3) / 1e9,
                            "frac_of_hbm": by / (ms_we * 1e-3) / 1e9 / hbm_gbs}
    enc["rows_4096x9216_b2_per_row_scale"] = rec["weight_encode"]
    # range + encode of the same weights in one pass over memory (mpq_encode_ranged) against the two-pass route
    ms_two = _graph_ms(lambda: (mpq.absmax(w, mpq.SCALE_PER_ROW, out=sw), mpq.encode(w, sw, 2, mpq.SCALE_PER_ROW, out=wp)))
    ms_one = _graph_ms(lambda: mpq.lib().mpq_encode_ranged(w.data_ptr(), n, k, k, mpq.ACT_HTANH, 2, sw.data_ptr(), wp.data_ptr(),
                                                           torch.cuda.current_stream().cuda_stream))
    enc["rows_4096x9216_b2_range_and_encode_one_pass"] = {"us": ms_one * 1e3, "gb_s": by / (ms_one * 1e-3) / 1e9,
                                                          "frac_of_hbm": by / (ms_one * 1e-3) / 1e9 / hbm_gbs,
                                                          "two_pass_us": ms_two * 1e3}
    out["fc_w2a2_64x4096x9216"] = rec
    del w, w2

    # ---- workload 3: 3x3 convolution W3A3 --------------------------------------------------------
    c = inputs.config3()
    x, w = up(c["x"]), up(c["w"])
    N, C, H, W = x.shape
    O = w.shape[0]
    sa, sw = mpq.absmax(x, 0, mpq.ACT_HRELU), mpq.absmax(w, mpq.SCALE_PER_ROW)
    xp = mpq.encode_nchw(x, sa, 3, mpq.ACT_HRELU)
    wpl, taps = mpq.encode_oihw(w, sw, 3, mpq.SCALE_PER_ROW)
    yf = torch.empty((N, O, H, W), dtype=torch.float32, device=dev)
    ms = _graph_ms(lambda: mpq.conv(xp, 3, N, C, H, W, wpl, 3, taps, O, 3, 3, 1, 1, None, yf, sa, sw, mpq.SCALE_PER_ROW))
    M, K = N * H * W, 9 * C
    out["conv3x3_w3a3_32x256x14x14"] = product_record(ms, M, O, K, 3, 3, 9.0 * M * O * (K // 32))
    ms = _graph_ms(lambda: mpq.encode_nchw(x, sa, 3, mpq.ACT_HRELU, out=xp))
    out["conv3x3_w3a3_32x256x14x14"]["encode_nchw_us"] = ms * 1e3

    # ---- deconvolution (Section 3.1): a generator-sized upsampling layer, W4A4 ----------------------
    N, C, H, O, ks, st, pd = 32, 256, 28, 128, 4, 2, 1
    x, w = up(inputs.normal(34, 0, (N, C, H, H), relu=True)), up(inputs.normal(34, 1, (O, C, ks, ks), std=0.05))
    sa, sw = mpq.absmax(x, 0, mpq.ACT_HRELU), mpq.absmax(w, mpq.SCALE_PER_ROW)
    xp = mpq.encode_nchw(x, sa, 4, mpq.ACT_HRELU)
    wpl, taps = mpq.encode_deconv_weights(w, sw, 4, st)
    Ho = (H - 1) * st - 2 * pd + ks
    yf = torch.empty((N, O, Ho, Ho), dtype=torch.float32, device=dev)
    ms = _graph_ms(lambda: mpq.deconv(xp, 4, N, C, H, H, wpl, 4, taps, O, ks, ks, st, pd, None, yf, sa, sw, mpq.SCALE_PER_ROW))
    M, K = N * Ho * Ho, (ks // st) * (ks // st) * C                # every output sums 2 x 2 taps x C products
    out["deconv4x4s2_w4a4_32x256x28x28"] = product_record(ms, M, O, K, 4, 4, 16.0 * M * O * (K // 32))
    del x, w, yf

    # ---- workload 5: ResNet-18-shaped stack, W4A4, batch 128 -------------------------------------
    batch = 128
    net = QuantResNet18Stack(inputs.config5_weights(), batch, 224, 4, 4, dev)
    x = up(inputs.config5_input(batch, 224))
    for _ in range(3):
        net.forward(x)
    torch.cuda.synchronize()
    steps, evs = 5, []
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(steps):
        ev = {}
        net.forward(x, ev)
        evs.append(ev)
    e1.record()
    torch.cuda.synchronize()
    ms = e0.elapsed_time(e1) / steps
    layers = {}
    quant_ms = 0.0
    for name in evs[0]:
        t = statistics.mean(ev[name][0].elapsed_time(ev[name][1]) for ev in evs)
        rec = {"ms": t}
        if name in net.convs:
            cv = net.convs[name]
            Cc, Hh, Ww = net.in_shape[name]
            Ho, Wo = cv.out_hw(Hh, Ww)
            popcs = 16.0 * batch * Ho * Wo * cv.O * (cv.KH * cv.KW * Cc // 32)
            rec.update({"span": "encode + conv (range, residual add and max(.,0) ride in the producers' stores)"
                        if "downsample" not in name else "conv",
                        "frac_of_branch_peak": popcs / (t * 1e-3) / branch_peak,
                        "frac_of_plain_popc_peak": popcs / (t * 1e-3) / popc_peak})
            quant_ms += t
        layers[name] = rec
    out["resnet18_stack_w4a4_b128"] = {"ms_per_step": ms, "images_per_s": batch / (ms * 1e-3),
                                       "quantized_layers_ms": quant_ms, "layers": layers}
    # the same stack with ranges fixed beforehand (calibrated on this batch): every convolution writes its
    # consumer's packed planes from its store, no encode pass after the first
    static = QuantResNet18Stack(inputs.config5_weights(), batch, 224, 4, 4, dev, static_ranges=net.calibrated_ranges())
    ms_static = _events_ms(lambda: static.forward(x), 5, 3)
    out["resnet18_stack_w4a4_b128"]["static_ranges"] = {"ms_per_step": ms_static, "images_per_s": batch / (ms_static * 1e-3)}
    del static
    # activation encoder of the first stage (NCHW variant, 102.8 MB in)
    xin = net.pooled
    i = [0]
    alt = torch.relu(torch.randn_like(xin))
    s_in = mpq.absmax(xin, 0, mpq.ACT_HRELU)
    pl = net.x_planes["layer1.0.conv1"]

    def f():
        mpq.encode_nchw(xin if i[0] % 2 == 0 else alt, s_in, 4, mpq.ACT_HRELU, out=pl)
        i[0] += 1
    ms = _graph_ms(f)
    by = xin.numel() * 4.5
    enc["nchw_128x64x56x56_b4"] = {"us": ms * 1e3, "gb_s": by / (ms * 1e-3) / 1e9,
                                   "frac_of_hbm": by / (ms * 1e-3) / 1e9 / hbm_gbs}
    out["encoders"] = enc
    if path:
        with open(path, "w") as fh:
            json.dump(out, fh, indent=1)
    return out


def compact(d: dict) -> dict:
    """The suite's headline figures, small enough to ride in the benchmark's one JSON line.
    `frac` = algorithmic word-popcounts per second / the carry-save mix peak measured in the same run."""
    r3 = lambda v: round(float(v), 3)
    c = {"peaks": {"mix_peak_gpopc_s": r3(d["branch_peak_gpopc_s"]), "plain_popc_gpopc_s": r3(d["popc_peak_gpopc_s"]),
                   "hbm_gbs": d["hbm_gbs"]},
         "gemm_w2a2_64x64x512": {"us": r3(d["gemm_w2a2_64x64x512"]["us"])}}
    for name in ("fc_w2a2_64x4096x9216", "conv3x3_w3a3_32x256x14x14", "deconv4x4s2_w4a4_32x256x28x28"):
        r = d[name]
        c[name] = {"us": r3(r["ms"] * 1e3), "equivalent_tops": r3(r["equivalent_tops"]), "frac": r3(r["frac_of_branch_peak"])}
    c["conv3x3_w3a3_32x256x14x14"]["encode_nchw_us"] = r3(d["conv3x3_w3a3_32x256x14x14"]["encode_nchw_us"])
    c["gemm_sweep_4096"] = {k: {"ms": r3(r["ms"]), "equivalent_tops": r3(r["equivalent_tops"]), "frac": r3(r["frac_of_branch_peak"])}
                            for k, r in d["gemm_sweep_4096"].items()}
    s = d["resnet18_stack_w4a4_b128"]
    c["resnet18_stack_w4a4_b128"] = {
        "ms_per_step": r3(s["ms_per_step"]), "images_per_s": round(s["images_per_s"], 1),
        "quantized_layers_ms": r3(s["quantized_layers_ms"]),
        "static_ranges_ms_per_step": r3(s["static_ranges"]["ms_per_step"]),
        "layers": {n: ([r3(r["ms"]), r3(r["frac_of_branch_peak"])] if "frac_of_branch_peak" in r else [r3(r["ms"])])
                   for n, r in s["layers"].items()},
        "layers_key": "[ms] or [ms, frac of mix peak]"}
    own = d.get("context_own_tcgen05_i8_gemm_4096", {})
    if "signed_ms" in own:
        c["context_int8_tensor_core_gemm_4096"] = {"own_tcgen05_ms": r3(own["signed_ms"]), "own_tcgen05_tops": round(own["signed_tops"], 1),
                                                   "own_tcgen05_unsigned_eq17_ms": r3(own["unsigned_eq17_ms"]),
                                                   "library_ms": r3(d.get("context_library_int8_gemm_4096", {}).get("ms", float("nan")))}
    c["encoders"] = {n: {"us": r3(r["us"]), "gb_s": round(r["gb_s"], 1), "frac_of_hbm": r3(r["frac_of_hbm"])}
                     for n, r in d["encoders"].items()}
    return c


def summary_markdown(d: dict) -> str:
    """The suite's figures as the tables committed under profiles/."""
    L = ["# Suite: all workloads on one B200 (`python bench.py --steps 20 --warmup 5 --full FILE`)\n",
         "CUDA events on the launching stream after warm-up; short kernels replayed from a CUDA graph (no host launch",
         "gaps).  Peaks measured in the same run: plain POPC pipe %.0f Gpopc/s, carry-save mix peak %.0f Gpopc/s"
         % (d["popc_peak_gpopc_s"], d["branch_peak_gpopc_s"]),
         "(probe at %.0f MHz), HBM copy %.0f GB/s (MEASURED_PEAKS.json).\n" % (d["probe_sm_mhz"], d["hbm_gbs"]),
         "## Bit-width sweep, GEMM m = n = k = 4096, int32 out\n",
         "| (w,a) bits | ms | equivalent TOPS | binary TOPS | frac of mix peak | frac of plain POPC pipe |",
         "|---|---|---|---|---|---|"]
    for k, r in d["gemm_sweep_4096"].items():
        L.append("| %s | %.3f | %.1f | %.1f | %.3f | %.3f |" % (k, r["ms"], r["equivalent_tops"], r["binary_tops"],
                                                             r["frac_of_branch_peak"], r["frac_of_plain_popc_peak"]))
    ctx = d.get("context_library_int8_gemm_4096", {})
    if "ms" in ctx:
        L.append("\nContext only (not this path): a library int8 tensor-core GEMM of the decoded integers, same shape: "
                 "%.3f ms = %.0f TOPS." % (ctx["ms"], ctx["tops"]))
    own = d.get("context_own_tcgen05_i8_gemm_4096", {})
    if "signed_ms" in own:
        L.append("Own tcgen05 kind::i8 kernel (context, not the library's path): signed codes %.3f ms = %.0f TOPS; 8-bit level "
                 "indices with the Eq. 17 correction %.3f ms = %.0f TOPS."
                 % (own["signed_ms"], own["signed_tops"], own["unsigned_eq17_ms"], own["unsigned_eq17_tops"]))
    L += ["\n## Other products\n", "| workload | time | equivalent TOPS | frac of mix peak | frac of plain POPC pipe |",
          "|---|---|---|---|---|",
          "| GEMM W2A2 64x64x512 (int32 + fp32 out) | %.1f us | launch-latency bound | – | – |" % d["gemm_w2a2_64x64x512"]["us"]]
    r = d["fc_w2a2_64x4096x9216"]
    L.append("| FC W2A2 64 x 4096 x 9216 (fp32 out, per-channel scale) | %.1f us | %.1f | %.3f | %.3f |"
             % (r["ms"] * 1e3, r["equivalent_tops"], r["frac_of_branch_peak"], r["frac_of_plain_popc_peak"]))
    r = d["conv3x3_w3a3_32x256x14x14"]
    L.append("| conv 3x3 W3A3 32x256x14x14 -> 256 (fp32 out) | %.1f us (+ encode_nchw %.1f us) | %.1f | %.3f | %.3f |"
             % (r["ms"] * 1e3, r["encode_nchw_us"], r["equivalent_tops"], r["frac_of_branch_peak"], r["frac_of_plain_popc_peak"]))
    r = d["deconv4x4s2_w4a4_32x256x28x28"]
    L.append("| deconv 4x4 stride 2 W4A4 32x256x28x28 -> 128 x 56 x 56 (fp32 out, one launch per output phase) | %.1f us | %.1f | %.3f | %.3f |"
             % (r["ms"] * 1e3, r["equivalent_tops"], r["frac_of_branch_peak"], r["frac_of_plain_popc_peak"]))
    s = d["resnet18_stack_w4a4_b128"]
    L += ["\n## ResNet-18-shaped stack, W4A4, batch 128, 224 x 224\n",
          "%.2f ms per step = **%.0f images/s** end to end (fp32 stem + max-pool + 19 encoded convolutions; residual add,"
          % (s["ms_per_step"], s["images_per_s"]),
          "max(.,0) and every encoder's range ride in the producers' stores); encoded layers %.2f ms.  Span of an encoded"
          % s["quantized_layers_ms"],
          "layer = encode_nchw + conv (shortcut convolutions reuse conv1's planes).  With ranges fixed beforehand",
          "(every convolution writes its consumer's planes from its store): %.2f ms per step = %.0f images/s.\n"
          % (s["static_ranges"]["ms_per_step"], s["static_ranges"]["images_per_s"]),
          "| layer | ms | frac of mix peak | frac of plain POPC pipe |", "|---|---|---|---|"]
    for n, r in s["layers"].items():
        if "frac_of_branch_peak" in r:
            L.append("| %s | %.3f | %.3f | %.3f |" % (n, r["ms"], r["frac_of_branch_peak"], r["frac_of_plain_popc_peak"]))
        else:
            L.append("| %s | %.3f | – | – |" % (n, r["ms"]))
    L += ["\n## Encoders and range (HBM-bound)\n", "| kernel / tensor | us | GB/s | frac of measured copy bandwidth |", "|---|---|---|---|"]
    for n, r in d["encoders"].items():
        L.append("| %s | %.1f | %.0f | %.3f |" % (n, r["us"], r["gb_s"], r["frac_of_hbm"]))
    if "cpu_oracle" in d:
        o = d["cpu_oracle"]
        L += ["\n## CPU oracle on the same host (%d cores), as it stands: a reported baseline, not a target\n" % o["cores"],
              "| workload | seconds | equivalent TOPS |", "|---|---|---|"]
        for n, r in o.items():
            if isinstance(r, dict):
                L.append("| %s | %.4f | %.4f |" % (n, r["seconds"], r["equivalent_tops"]))
    return "\n".join(L) + "\n"


def _single(argv):
    """One product on its own, a few launches, for profiler captures:
        python bench_suite.py gemm A_BITS W_BITS SIZE
        python bench_suite.py conv BITS N C HW O KSIZE STRIDE
        python bench_suite.py fc A_BITS W_BITS M N K
        python bench_suite.py deconv BITS N C HW O KSIZE STRIDE PAD
        python bench_suite.py encode BITS ROWS K            (row encoder, four inputs in rotation)
        python bench_suite.py nchw BITS N C HW              (NCHW encoder)
        python bench_suite.py absmax ROWS K
        python bench_suite.py i8 SIZE                       (context: own tensor-core kernel, signed form)
    Prints the CUDA-event time of the last 10 launches."""
    dev = torch.device("cuda:0")
    torch.cuda.set_device(0)
    if argv[0] == "gemm":
        ab, wb, size = (int(a) for a in argv[1:4])
        x = torch.randn(size, size, device=dev).relu_()
        w = torch.randn(size, size, device=dev)
        sa, sw = mpq.absmax(x), mpq.absmax(w)
        ap, wp = mpq.encode(x, sa, ab), mpq.encode(w, sw, wb)
        ci = torch.empty((size, size), dtype=torch.int32, device=dev)
        fn = lambda: mpq.gemm(ap, ab, wp, wb, size, size, size, ci, None)
        popcs = float(ab * wb) * size * size * (size // 32)
    elif argv[0] == "conv":
        bits, N, C, HW, O, ks, stride = (int(a) for a in argv[1:8])
        x = torch.randn(N, C, HW, HW, device=dev).relu_()
        w = torch.randn(O, C, ks, ks, device=dev)
        sa, sw = mpq.absmax(x, 0, mpq.ACT_HRELU), mpq.absmax(w, mpq.SCALE_PER_ROW)
        xp = mpq.encode_nchw(x, sa, bits, mpq.ACT_HRELU)
        wp, taps = mpq.encode_oihw(w, sw, bits, mpq.SCALE_PER_ROW)
        pad = ks // 2
        Ho = (HW + 2 * pad - ks) // stride + 1
        y = torch.empty((N, O, Ho, Ho), dtype=torch.float32, device=dev)
        fn = lambda: mpq.conv(xp, bits, N, C, HW, HW, wp, bits, taps, O, ks, ks, stride, pad, None, y, sa, sw,
                              mpq.SCALE_PER_ROW)
        popcs = float(bits * bits) * N * Ho * Ho * O * (ks * ks * C // 32)
    elif argv[0] == "deconv":
        bits, N, C, HW, O, ks, stride, pad = (int(a) for a in argv[1:9])
        x = torch.randn(N, C, HW, HW, device=dev).relu_()
        w = torch.randn(O, C, ks, ks, device=dev)
        sa, sw = mpq.absmax(x, 0, mpq.ACT_HRELU), mpq.absmax(w, mpq.SCALE_PER_ROW)
        xp = mpq.encode_nchw(x, sa, bits, mpq.ACT_HRELU)
        wp, taps = mpq.encode_deconv_weights(w, sw, bits, stride)
        Ho = (HW - 1) * stride - 2 * pad + ks
        y = torch.empty((N, O, Ho, Ho), dtype=torch.float32, device=dev)
        fn = lambda: mpq.deconv(xp, bits, N, C, HW, HW, wp, bits, taps, O, ks, ks, stride, pad, None, y, sa, sw,
                                mpq.SCALE_PER_ROW)
        popcs = float(bits * bits) * N * HW * HW * O * (ks * ks * C // 32)   # every input pixel meets every tap once
    elif argv[0] == "fc":
        ab, wb, m, n, k = (int(a) for a in argv[1:6])
        x = torch.randn(m, k, device=dev).relu_()
        w = torch.randn(n, k, device=dev)
        sa, sw = mpq.absmax(x, 0, mpq.ACT_HRELU), mpq.absmax(w, mpq.SCALE_PER_ROW)
        ap, wp = mpq.encode(x, sa, ab, 0, mpq.ACT_HRELU), mpq.encode(w, sw, wb, mpq.SCALE_PER_ROW)
        cf = torch.empty((m, n), dtype=torch.float32, device=dev)
        fn = lambda: mpq.gemm(ap, ab, wp, wb, m, n, k, None, cf, sa, sw, mpq.SCALE_PER_ROW)
        popcs = float(ab * wb) * m * n * (k // 32)
    elif argv[0] in ("encode", "absmax"):
        bits = int(argv[1]) if argv[0] == "encode" else 0
        rows, k = (int(a) for a in argv[-2:])
        xs = [torch.randn(rows, k, device=dev) for _ in range(4)]
        sa = mpq.absmax(xs[0])
        planes = torch.empty((max(bits, 1), rows, mpq.row_words(k)), dtype=torch.int32, device=dev)
        i = [0]

        def fn():
            if bits:
                mpq.encode(xs[i[0] % 4], sa, bits, out=planes)
            else:
                mpq.absmax(xs[i[0] % 4], out=sa)
            i[0] += 1
        popcs = 0.0
        print("bytes per launch: %.0f" % (rows * k * (4 + bits / 8.0)))
    elif argv[0] == "nchw":
        bits, N, C, HW = (int(a) for a in argv[1:5])
        xs = [torch.randn(N, C, HW, HW, device=dev).relu_() for _ in range(2)]
        sa = mpq.absmax(xs[0], 0, mpq.ACT_HRELU)
        planes = torch.empty((bits, N, HW, HW, C // 32), dtype=torch.int32, device=dev)
        i = [0]

        def fn():
            mpq.encode_nchw(xs[i[0] % 2], sa, bits, mpq.ACT_HRELU, out=planes)
            i[0] += 1
        popcs = 0.0
        print("bytes per launch: %.0f" % (xs[0].numel() * (4 + bits / 8.0)))
    elif argv[0] == "i8":
        size = int(argv[1])
        qa = torch.randint(-3, 4, (size, size), dtype=torch.int8, device=dev)
        qb = torch.randint(-3, 4, (size, size), dtype=torch.int8, device=dev)
        co = torch.empty((size, size), dtype=torch.int32, device=dev)
        err = torch.zeros(1, dtype=torch.int32, device=dev)
        fn = lambda: context.i8_gemm(qa, qb, co, err)
        popcs = 0.0
    else:
        raise SystemExit(_single.__doc__)
    ms = _events_ms(fn, 10, 4)
    print("%s: %.4f ms per launch, %.1f Gpopc/s" % (" ".join(argv), ms, popcs / (ms * 1e-3) / 1e9))


if __name__ == "__main__":
    import sys
    _single(sys.argv[1:])
