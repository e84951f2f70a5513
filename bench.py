#!/usr/bin/env python
"""Benchmark of the encoded-layer hot path on B200.

One step = one pass of the whole path over one batch of synthetic input, through the C ABI:
range (max-abs) of both operands -> fused quantize+pack of both -> branch-fused binary GEMM with
the decoder scale fused into the store (int32 accumulators and scaled fp32 output).
Workload at N = 1: the W2A2 square GEMM m = n = k = 4096 of the bit-width sweep (the setting the
throughput target is quoted on).  With N > 1 every rank runs the same workload on its own GPU
(independent problems, no exchange step): weak scaling, replicas only.

Prints ONE JSON line (rank 0).  ``--impl reference`` times the CPU oracle instead.
After the timed region the other workloads (fully-connected layer, convolution, bit-width sweep,
ResNet-18-shaped stack, encoders) are timed too and a compact ``suite`` object is added to the line;
``--full FILE`` additionally writes all their figures to FILE.
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import threading
import time


ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

METRIC = "equivalent W2A2 TOPS of the encoded layer (2*m*n*k / step time)"
UNIT = "TOPS"
SIZE = 4096
A_BITS = W_BITS = 2
HBM_FALLBACK_GBS = 6650.0      # used only when MEASURED_PEAKS.json is absent
# DRAM bytes per launch of the GEMM kernel (dram__bytes_read.sum + dram__bytes_write.sum) from the
# kept ncu capture of this command: 8.46 MB + 79.54 MB.
# Set back to None whenever branch_kernel changes after that capture.
GEMM_DRAM_TRAFFIC_BYTES = 88.0e6
ORACLE_SAMPLE_ROWS = 1024      # activation rows of the bounded sample the CPU oracle is timed on


def _peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            return json.load(f), "measured"
    return {"hbm_gbs": HBM_FALLBACK_GBS}, "fallback"


class NvmlClockSampler:
    """Reads SM clock, power and clock-event reasons through NVML every 5 ms in a thread while the timed
    region runs (read-only queries; nothing on the GPU is set).  ``mark()`` brackets the timed region:
    the summary uses the samples taken inside it."""
    REASONS = (("hw_slowdown", "nvmlClocksEventReasonHwSlowdown"),
               ("hw_thermal_slowdown", "nvmlClocksEventReasonHwThermalSlowdown"),
               ("sw_thermal_slowdown", "nvmlClocksEventReasonSwThermalSlowdown"),
               ("sw_power_cap", "nvmlClocksEventReasonSwPowerCap"))

    def __init__(self, torch_index: int):
        import pynvml
        import torch
        self.nv = pynvml
        pynvml.nvmlInit()
        props = torch.cuda.get_device_properties(torch_index)
        try:
            bus = "%08X:%02X:%02X.0" % (props.pci_domain_id, props.pci_bus_id, props.pci_device_id)
            self.handle = pynvml.nvmlDeviceGetHandleByPciBusId(bus.encode())
        except Exception:
            self.handle = pynvml.nvmlDeviceGetHandleByIndex(torch_index)
        self.samples = []                       # (time, sm_mhz, reasons bitmask)
        self.max_mhz = float(pynvml.nvmlDeviceGetMaxClockInfo(self.handle, pynvml.NVML_CLOCK_SM))
        self.marks = []
        self.stop = threading.Event()
        self.thread = threading.Thread(target=self._run, daemon=True)

    def _run(self):
        nv = self.nv
        while not self.stop.is_set():
            try:
                mhz = float(nv.nvmlDeviceGetClockInfo(self.handle, nv.NVML_CLOCK_SM))
                mask = int(nv.nvmlDeviceGetCurrentClocksEventReasons(self.handle))
                self.samples.append((time.perf_counter(), mhz, mask))
            except Exception:
                pass
            time.sleep(0.005)

    def __enter__(self):
        self.thread.start()
        return self

    def mark(self):
        self.marks.append(time.perf_counter())

    def __exit__(self, *exc):
        self.stop.set()
        self.thread.join(timeout=2)

    def summary(self):
        lo, hi = (self.marks[0], self.marks[-1]) if len(self.marks) >= 2 else (0.0, float("inf"))
        inside = [s for s in self.samples if lo <= s[0] <= hi] or self.samples
        if not inside:
            return {"sm_mhz": None, "sm_max_mhz": self.max_mhz, "reasons": [], "samples": 0}
        mask = 0
        for s in inside:
            mask |= s[2]
        reasons = sorted(name for name, attr in self.REASONS if mask & int(getattr(self.nv, attr, 0)))
        return {"sm_mhz": statistics.median(s[1] for s in inside), "sm_max_mhz": self.max_mhz, "reasons": reasons,
                "samples": len(inside), "source": "NVML, 5 ms period, inside the timed region"}


def clock_sampler(index: int):
    """NVML sampler when the NVML binding is importable, else the nvidia-smi one."""
    try:
        return NvmlClockSampler(index)
    except Exception:
        return ClockSampler(index)


class ClockSampler:
    """Samples nvidia-smi clocks and throttle reasons every 200 ms while the timed region runs."""
    QUERY = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
             "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
             "clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.index = index
        self.rows = []
        self.proc = None

    def mark(self):
        pass

    def __enter__(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", "-i", str(self.index), "--query-gpu=" + self.QUERY, "--format=csv,noheader,nounits",
                 "-lms", "200"], stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=self._read, daemon=True)
            self.thread.start()
        except OSError:
            self.proc = None
        return self

    def _read(self):
        for line in self.proc.stdout:
            parts = [p.strip() for p in line.split(",")]
            if len(parts) >= 7:
                self.rows.append(parts)

    def __exit__(self, *exc):
        if self.proc is not None:
            time.sleep(0.25)
            self.proc.terminate()
            try:
                self.proc.wait(timeout=5)
            except subprocess.TimeoutExpired:
                self.proc.kill()

    def summary(self):
        sm, mx, reasons = [], [], set()
        for r in self.rows:
            try:
                sm.append(float(r[0])); mx.append(float(r[1]))
            except ValueError:
                continue
            for name, v in zip(("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"), r[3:7]):
                if v.lower().startswith("active"):
                    reasons.add(name)
        if not sm:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": [], "samples": 0}
        return {"sm_mhz": statistics.median(sm), "sm_max_mhz": max(mx), "reasons": sorted(reasons), "samples": len(sm)}


def max_over_ranks(value: float, world: int, device=None) -> float:
    """Slowest rank's figure: every rank contributes its own time, all get the maximum.
    (The replicas share nothing else: the path has no exchange step.)"""
    if world <= 1:
        return float(value)
    import torch
    import torch.distributed as dist
    t = torch.tensor([value], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def whole_job_tops(world: int, m: int, n: int, k: int, ms_per_step: float) -> float:
    """Aggregate equivalent TOPS of `world` independent replicas that each do one m x n x k layer per step."""
    return world * 2.0 * m * n * k / (ms_per_step * 1e-3) / 1e12


def _config():
    """The workload both arms report on (the reference arm times a bounded sample of it)."""
    return {"workload": "gemm_w2a2_4096", "m": SIZE, "n": SIZE, "k": SIZE, "a_bits": A_BITS, "w_bits": W_BITS,
            "step": "absmax x2 + encode x2 + branch-fused GEMM (int32 + scaled fp32 out)",
            "l2": "fp32 inputs (128 MiB) and outputs (128 MiB) per step exceed the 126 MB L2; no flush"}


def _workload_arrays():
    from paper_1905_13389_b200 import inputs
    c = inputs.config4(W_BITS, A_BITS, SIZE)
    return c["x"], c["w"]


# ------------------------------------------------------------------------------------------------
# reference arm / cpu_baseline: the oracle as it stands, on the host cores, on a bounded sample
# ------------------------------------------------------------------------------------------------
def _oracle_sample_step(x, w, rows):
    """Oracle pass over `rows` rows of the activations against the full weight matrix."""
    import oracle
    s_a = oracle.absmax(x)
    s_w = oracle.absmax(w)
    qa = oracle.quantize(x[:rows], s_a, A_BITS)
    qb = oracle.quantize(w, s_w, W_BITS)
    acc = oracle.gemm(qa, qb)
    return oracle.scale(acc, s_a[0], s_w, A_BITS, W_BITS)


def _time_oracle(x, w, rows, steps, warmup):
    import oracle
    oracle.build()
    for _ in range(warmup):
        _oracle_sample_step(x, w, rows)
    t0 = time.perf_counter()
    for _ in range(steps):
        _oracle_sample_step(x, w, rows)
    dt = (time.perf_counter() - t0) / steps
    tops = 2.0 * rows * SIZE * SIZE / dt / 1e12
    sample = "rows 0..%d of the %dx%d activations against all %d weight rows (k=%d): range, quantize, " \
             "integer GEMM and scale; throughput = 2*rows*n*k / time" % (rows - 1, SIZE, SIZE, SIZE, SIZE)
    return tops, dt, oracle.threads(), sample


def _oracle_other_workloads():
    """CPU-baseline leg of --full: the oracle as it stands, timed once on workloads 1-3 in full
    (range, quantize, integer product, scale).  Reported next to the GPU figures, never a target."""
    import oracle
    from paper_1905_13389_b200 import inputs
    oracle.build()
    out = {"cores": oracle.threads()}
    c = inputs.config1()
    t0 = time.perf_counter(); oracle.linear(c["x"], c["w"], 2, 2, a_act=oracle.HRELU); dt = time.perf_counter() - t0
    out["gemm_w2a2_64x64x512"] = {"seconds": dt, "equivalent_tops": 2.0 * 64 * 64 * 512 / dt / 1e12}
    c = inputs.config2()
    t0 = time.perf_counter(); oracle.linear(c["x"], c["w"], 2, 2, w_per_row=True, a_act=oracle.HRELU); dt = time.perf_counter() - t0
    out["fc_w2a2_64x4096x9216"] = {"seconds": dt, "equivalent_tops": 2.0 * c["m"] * c["n"] * c["k"] / dt / 1e12}
    c = inputs.config3()
    t0 = time.perf_counter(); oracle.conv_layer(c["x"], c["w"], 3, 3, 1, 1, True, oracle.HRELU); dt = time.perf_counter() - t0
    out["conv3x3_w3a3_32x256x14x14"] = {"seconds": dt, "equivalent_tops": 2.0 * 6272 * 256 * 2304 / dt / 1e12}
    return out


def run_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    x, w = _workload_arrays()
    tops, dt, cores, sample = _time_oracle(x, w, ORACLE_SAMPLE_ROWS, args.steps, args.warmup)
    line = {
        "impl": "reference", "metric": METRIC, "value": tops, "unit": UNIT, "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": dt * 1e3, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "int32", "data": "synthetic",
        "config": _config(),
        "cpu_baseline": {"value": tops, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": sample},
        "e2e": {"value": tops, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line), flush=True)


# ------------------------------------------------------------------------------------------------
# CUDA arm
# ------------------------------------------------------------------------------------------------
def run_cuda(args):
    import torch
    import torch.distributed as dist
    from paper_1905_13389_b200 import binding as mpq

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise RuntimeError("bench.py needs a CUDA device (there is no CPU fallback)")
    torch.cuda.set_device(local_rank)
    dev = torch.device("cuda", local_rank)
    if world > 1:
        dist.init_process_group("nccl", device_id=dev)
    mpq.lib()

    x_np, w_np = _workload_arrays()
    x = torch.from_numpy(x_np).to(dev)
    w = torch.from_numpy(w_np).to(dev)
    m = n = k = SIZE
    rw = mpq.row_words(k)
    s_a = torch.empty(1, dtype=torch.float32, device=dev)
    s_w = torch.empty(1, dtype=torch.float32, device=dev)
    ap = torch.empty((A_BITS, m, rw), dtype=torch.int32, device=dev)
    wp = torch.empty((W_BITS, n, rw), dtype=torch.int32, device=dev)
    ci = torch.empty((m, n), dtype=torch.int32, device=dev)
    cf = torch.empty((m, n), dtype=torch.float32, device=dev)

    ev = lambda: torch.cuda.Event(enable_timing=True)
    enc_events, gemm_events = [], []

    def step(record: bool):
        mpq.absmax(x, mpq.SCALE_PER_TENSOR, mpq.ACT_HTANH, out=s_a)
        mpq.absmax(w, mpq.SCALE_PER_TENSOR, mpq.ACT_HTANH, out=s_w)
        if record:
            e0, e1, e2 = ev(), ev(), ev()
            e0.record()
        mpq.encode(x, s_a, A_BITS, out=ap)
        mpq.encode(w, s_w, W_BITS, out=wp)
        if record:
            e1.record()
        mpq.gemm(ap, A_BITS, wp, W_BITS, m, n, k, ci, cf, s_a, s_w, mpq.SCALE_PER_TENSOR)
        if record:
            e2.record()
            enc_events.append((e0, e1))
            gemm_events.append((e1, e2))

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    for _ in range(max(args.warmup, 3)):
        step(False)
    barrier()
    # Roofline denominators, all measured live with register-only probes at the clocks of this run:
    # the plain POPC issue rate; the legacy one-bit tensor instruction; and the two integer pipes'
    # joint issue rate for groups of L logic ops + 1 POPC + 1 multiply-add, L = 0..8.  A carry-save
    # reduction that spends f full adders per xor word executes 1 + 2f logic ops and 1 - f POPCs per
    # word, i.e. L = (1 + 2f)/(1 - f) logic ops per POPC and (L + 2)/3 algorithmic word-popcounts per
    # group; the ceiling of the XOR/POPC route is the best of those over L.
    popc_peak, probe_mhz, sms = mpq.measure_popc_peak()
    mix_table = []
    for L in range(0, 9):
        rate, mhz_l, _ = mpq.measure_mix_peak(L)
        words = (L + 2) / 3.0 if L >= 1 else 0.0           # L = 0 has no xor: not a branch product
        mix_table.append({"logic_per_popc": L, "groups_per_s": rate, "probe_sm_mhz": mhz_l,
                          "clk_per_warp_group_per_subpartition": 32.0 * 4 * sms * mhz_l * 1e6 / rate,
                          "word_popc_per_group": words, "word_popc_per_s": rate * words})
    own_mix_peak = mix_table[4]["word_popc_per_s"]         # the shipped kernel: one adder per two xor words, L = 4
    best_mix = max(mix_table, key=lambda r: r["word_popc_per_s"])
    branch_peak = best_mix["word_popc_per_s"]
    b1 = {}
    for name, and_popc in (("xor_popc", False), ("and_popc", True)):
        rate, mhz_b, _ = mpq.measure_b1_mma_peak(and_popc)
        b1[name] = {"warp_mma_per_s": rate, "warp_mma_per_clk_per_sm": rate / (mhz_b * 1e6 * sms),
                    "word_popc_per_s": rate * 1024.0}

    with clock_sampler(local_rank) as clocks:
        barrier()
        clocks.mark()
        t0, t1 = ev(), ev()
        t0.record()
        for _ in range(args.steps):
            step(True)
        t1.record()
        barrier()
        clocks.mark()
    elapsed_ms = max_over_ranks(t0.elapsed_time(t1), world, dev)
    ms_per_step = elapsed_ms / args.steps
    value = whole_job_tops(world, m, n, k, ms_per_step)

    gemm_ms = statistics.mean(a.elapsed_time(b) for a, b in gemm_events)
    enc_ms = statistics.mean(a.elapsed_time(b) for a, b in enc_events)
    popcs = float(A_BITS * W_BITS) * m * n * (k // 32)                 # algorithmic popcounts per launch
    achieved = popcs / (gemm_ms * 1e-3)
    peaks, peak_kind = _peaks()
    enc_bytes = (m * k + n * k) * 4.0 + (A_BITS * m + W_BITS * n) * rw * 4.0
    enc_gbs = enc_bytes / (enc_ms * 1e-3) / 1e9
    # the encode kernel alone: 20 launches on alternating operands replayed from one CUDA graph, so that
    # neither host launch cost nor the event records of the step sit between the kernels
    g = torch.cuda.CUDAGraph()
    side = torch.cuda.Stream()
    torch.cuda.synchronize()
    with torch.cuda.stream(side):
        with torch.cuda.graph(g, stream=side):
            for i in range(10):
                mpq.encode(x, s_a, A_BITS, out=ap)
                mpq.encode(w, s_w, W_BITS, out=wp)
    g.replay()
    torch.cuda.synchronize()
    k0, k1 = ev(), ev()
    k0.record()
    g.replay()
    k1.record()
    torch.cuda.synchronize()
    enc_kernel_ms = k0.elapsed_time(k1) / 20
    enc_kernel_gbs = 0.5 * enc_bytes / (enc_kernel_ms * 1e-3) / 1e9

    # end to end through the host-buffer entry point: pinned host inputs, H2D + D2H inside the timed region
    xh, wh = torch.from_numpy(x_np).pin_memory(), torch.from_numpy(w_np).pin_memory()
    oi = torch.empty((m, n), dtype=torch.int32).pin_memory()
    of = torch.empty((m, n), dtype=torch.float32).pin_memory()
    ws = torch.empty(mpq.linear_host_workspace(m, n, k, A_BITS, W_BITS), dtype=torch.uint8, device=dev)
    e2e_steps = max(3, min(args.steps, 10))
    for _ in range(2):
        mpq.linear_host(xh, wh, A_BITS, W_BITS, out_i32_host=oi, out_f32_host=of, workspace=ws)
    barrier()
    t0, t1 = ev(), ev()
    t0.record()
    for _ in range(e2e_steps):
        mpq.linear_host(xh, wh, A_BITS, W_BITS, out_i32_host=oi, out_f32_host=of, workspace=ws)
    t1.record()
    barrier()
    e2e_ms = max_over_ranks(t0.elapsed_time(t1), world, dev)
    e2e_value = whole_job_tops(world, m, n, k, e2e_ms / e2e_steps)
    # the deployed form: weights encoded once and resident, only activations up and results down
    ws2 = torch.empty(mpq.linear_host_prepared_workspace(m, n, k, A_BITS), dtype=torch.uint8, device=dev)
    for _ in range(2):
        mpq.linear_host_prepared(xh, wp, s_w, n, A_BITS, W_BITS, out_i32_host=oi, out_f32_host=of, workspace=ws2)
    barrier()
    t0, t1 = ev(), ev()
    t0.record()
    for _ in range(e2e_steps):
        mpq.linear_host_prepared(xh, wp, s_w, n, A_BITS, W_BITS, out_i32_host=oi, out_f32_host=of, workspace=ws2)
    t1.record()
    barrier()
    e2e_prepared_ms = max_over_ranks(t0.elapsed_time(t1), world, dev)

    if rank == 0:
        line = {
            "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
            "warmup": max(args.warmup, 3), "ms_per_step": ms_per_step, "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "int32", "data": "synthetic",
            "config": _config(), "binary_tops": value * A_BITS * W_BITS,
            "roofline": {"bound": "alu", "kernel": "branch_kernel<2,2,4,gemm> (XOR + carry-save + POPC GEMM, 64 x 64 tile, 3 CTAs per SM)",
                         "achieved": achieved / 1e9, "peak": branch_peak / 1e9, "unit": "Gpopc/s",
                         "frac": achieved / branch_peak, "traffic": GEMM_DRAM_TRAFFIC_BYTES,
                         "peak_source": "measured live at %.0f MHz on %d SMs: the best, over L = 1..8, of the two integer "
                                        "pipes' joint issue rate for groups of L three-input logic ops + 1 POPC + 1 integer "
                                        "multiply-add (mpq_measure_mix_peak) x the (L + 2)/3 algorithmic word-popcounts a "
                                        "carry-save reduction gets out of such a group; best L = %d"
                                        % (probe_mhz, sms, best_mix["logic_per_popc"]),
                         "frac_of_own_mix": achieved / own_mix_peak,
                         "own_mix": "L = 4 (one full adder per two xor words): %.1f Gpopc/s" % (own_mix_peak / 1e9),
                         "mix_table": mix_table,
                         "plain_popc_pipe": {"peak": popc_peak / 1e9, "frac": achieved / popc_peak,
                                             "lanes_per_clk_per_sm": popc_peak / (probe_mhz * 1e6 * sms),
                                             "note": "one POPC per xor word (no carry-save) cannot exceed this; the "
                                                     "kernel issues half as many POPCs as algorithmic popcounts"},
                         "b1_mma": {"xor_popc": dict(b1["xor_popc"], frac=achieved / b1["xor_popc"]["word_popc_per_s"]),
                                    "and_popc": dict(b1["and_popc"], frac=achieved / b1["and_popc"]["word_popc_per_s"]),
                                    "note": "legacy mma.sync.m16n8k256 b1 in a register-only loop with constant operands "
                                            "(mpq_measure_b1_mma_peak); one warp instruction = 1024 word-popcounts; frac = "
                                            "achieved / that ceiling (above 1: the instruction is slower than this kernel "
                                            "even with no operand traffic, so no tensor variant ships)"},
                         "ms_per_launch": gemm_ms, "algorithmic_popc_per_launch": popcs,
                         "equivalent_tops_of_this_kernel": 2.0 * m * n * k / (gemm_ms * 1e-3) / 1e12},
            "encode": {"bound": "hbm", "achieved": enc_gbs, "peak": peaks["hbm_gbs"], "unit": "GB/s",
                       "frac": enc_gbs / peaks["hbm_gbs"], "peak_source": "%s copy bandwidth" % peak_kind,
                       "ms_per_step": enc_ms, "bytes_per_step": enc_bytes,
                       "note": "achieved = both operands' encodes inside the timed step, launch gaps and event records "
                               "included; kernel_only = one encode launch (64 MiB fp32 in, 4 MiB planes out) replayed "
                               "back to back from a CUDA graph",
                       "kernel_only": {"us_per_launch": enc_kernel_ms * 1e3, "achieved": enc_kernel_gbs,
                                       "frac": enc_kernel_gbs / peaks["hbm_gbs"]}},
            "e2e": {"value": e2e_value, "unit": UNIT, "h2d_bytes_per_step": 2 * m * k * 4,
                    "d2h_bytes_per_step": 2 * m * n * 4, "ms_per_step": e2e_ms / e2e_steps,
                    "api": "mpq_linear_host (pinned host buffers; both operands copied and encoded every step)",
                    "resident_weights": {"value": whole_job_tops(world, m, n, k, e2e_prepared_ms / e2e_steps), "unit": UNIT,
                                         "ms_per_step": e2e_prepared_ms / e2e_steps, "h2d_bytes_per_step": m * k * 4,
                                         "d2h_bytes_per_step": 2 * m * n * 4,
                                         "api": "mpq_linear_host_prepared (weights encoded once, resident on the device)"}},
            # per step: 2 x (zeroing kernel + range kernel), 2 x encoder, 1 x branch GEMM
            "gpu_launches": 7 * args.steps,
            "clocks": clocks.summary(),
        }
        suite = None
        if world == 1 and not args.no_suite:
            # the other workloads (fully-connected layer, convolution, sweep, stack, encoders), timed after
            # the step above; a compact copy rides in this line, --full FILE keeps everything
            import bench_suite
            del x, w, ap, wp, ci, cf, xh, wh, oi, of, ws, ws2
            torch.cuda.empty_cache()
            suite = bench_suite.run_suite(dev, peaks["hbm_gbs"], args.full)
            line["suite"] = bench_suite.compact(suite)
        if world == 1 and not args.no_cpu_baseline:
            tops, dt, cores, sample = _time_oracle(x_np, w_np, ORACLE_SAMPLE_ROWS, args.steps, args.warmup)
            line["cpu_baseline"] = {"value": tops, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": sample,
                                    "seconds_per_sample": dt}
        print(json.dumps(line), flush=True)
        if args.full and suite is not None:
            if not args.no_cpu_baseline:
                suite["cpu_oracle"] = _oracle_other_workloads()
                with open(args.full, "w") as fh:
                    json.dump(suite, fh, indent=1)
            with open(args.full + ".md", "w") as fh:
                fh.write(bench_suite.summary_markdown(suite))
    if world > 1:
        dist.destroy_process_group()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="cuda", choices=["cuda", "reference"])
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-suite", action="store_true", help="skip the other workloads (only the timed step)")
    ap.add_argument("--full", metavar="FILE", default=None,
                    help="also time every workload (sweep, FC, conv, stack, encoders) and write them to FILE as JSON")
    args = ap.parse_args()
    if args.impl == "reference":
        run_reference(args)
    else:
        run_cuda(args)


if __name__ == "__main__":
    main()
