#!/usr/bin/env python
"""Benchmark of the quantized linear layer on B200.

A *step* is one pass of the whole hot path over one decoder layer's worth of synthetic
input: the activation quantizer for each distinct layer input (the q/k/v projections share
one input, gate/up share one) followed by the seven quantized linears.  Layers rotate through
distinct weight/activation buffers whose total exceeds twice the L2 size, so no step finds
its operands cached.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload NAME] [--impl ours|reference]

Prints ONE JSON line: `value` = whole-step throughput with inputs resident on the device (TOPS for
prefill workloads, GB/s of algorithmic bytes for decode workloads); `roofline` = the GEMM launches alone
against the measured peak; `quantize*` = the quantizer and its variants against the measured copy rate;
`e2e` = the same step with pinned-host inputs copied in and outputs copied out; `cpu_baseline` = the CPU
oracle on a row sample; `clocks` = SM clocks and throttle reasons sampled during the timed region.
`--impl reference` times the CPU oracle instead (a deliberately plain program; a baseline, not a target).
Linears that share their input are issued as one grouped call (`--no-group`: one call per linear).
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

import numpy as np  # noqa: E402

from paper_2512_23367_b200 import synth  # noqa: E402

L2_BYTES = 126 * 1024 * 1024
DEFAULT_WORKLOAD = "c2_w8a8_1b_prefill"
DATASHEET_INT8_TOPS = 4500.0
FALLBACK_PEAKS = {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0}


# --------------------------------------------------------------------------- host-side logic

def layer_plan(wl: synth.Workload):
    """Groups the linears of a workload by shared input: [(K, [linear indices])].
    q/k/v share the layer input, gate/up share the MLP input; everything else has its own."""
    groups: list[tuple[int, list[int]]] = []
    share = {"q_proj": "attn_in", "k_proj": "attn_in", "v_proj": "attn_in", "gate_proj": "mlp_in", "up_proj": "mlp_in"}
    seen: dict[str, int] = {}
    for i, lin in enumerate(wl.linears):
        key = share.get(lin.name)
        if key is not None and key in seen:
            groups[seen[key]][1].append(i)
        else:
            if key is not None:
                seen[key] = len(groups)
            groups.append((lin.K, [i]))
    return groups


def step_ops(wl: synth.Workload, M: int) -> int:
    """Integer operations (2 per multiply-add) of the GEMMs of one step."""
    return sum(2 * M * lin.N * lin.K for lin in wl.linears)


def weight_bytes(wl: synth.Workload) -> int:
    per = 1.0 if wl.w_bits == 8 else 0.5
    total = 0
    for lin in wl.linears:
        total += int(lin.N * lin.K * per)
        total += lin.N * 4 if wl.w_bits == 8 else (lin.K // synth.GROUP) * lin.N * 2
    return total


def step_bytes(wl: synth.Workload, M: int) -> dict:
    """Algorithmic bytes of one step: quantizer (2 B read + 1 B written per element + scale) and
    GEMMs (codes + scales read once, weights read once, FP16 result written once)."""
    quant = sum(3 * M * K + 4 * M for K, _ in layer_plan(wl))
    gemm = weight_bytes(wl) + sum(M * lin.K + 4 * M + 2 * M * lin.N for lin in wl.linears)
    return {"quantize": quant, "gemm": gemm}


def layers_for_rotation(wl: synth.Workload, M: int) -> int:
    """How many distinct layer buffer sets make the rotation exceed twice the L2 size."""
    per_layer = weight_bytes(wl) + sum(2 * M * K for K, _ in layer_plan(wl))
    return max(2, int(np.ceil(2.0 * L2_BYTES / per_layer)) + 1)


def aggregate_over_ranks(local_ms: float, local_units: float, world_size: int):
    """Whole-job figures from per-rank ones: time = max over ranks, units = sum over ranks.
    Uses torch.distributed when world_size > 1 (any backend)."""
    if world_size <= 1:
        return local_ms, local_units
    import torch
    import torch.distributed as dist
    dev = "cuda" if dist.get_backend() == "nccl" else "cpu"
    t = torch.tensor([local_ms], dtype=torch.float64, device=dev)
    u = torch.tensor([local_units], dtype=torch.float64, device=dev)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    dist.all_reduce(u, op=dist.ReduceOp.SUM)
    return float(t.item()), float(u.item())


def load_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            return json.load(f), "measured"
    return dict(FALLBACK_PEAKS), "fallback"


def load_traffic(wl: synth.Workload, M: int, grouped: bool = False):
    """DRAM bytes per launch of the dominant (GEMM) kernel, averaged over the step's GEMM launches, from
    the committed ncu summaries (profiles/traffic.json: "gemm_w<bits>a8:MxKxN" -> bytes of one launch;
    "...xN*G" for a grouped launch of G linears of width N).  None unless every launch of the step has
    an entry taken from the current kernel."""
    path = os.path.join(ROOT, "profiles", "traffic.json")
    if not os.path.exists(path):
        return None
    with open(path) as f:
        table = json.load(f)
    keys = []
    for K, idxs in layer_plan(wl):
        widths = {wl.linears[i].N for i in idxs}
        if grouped and len(idxs) > 1 and len(widths) == 1:
            keys.append(f"gemm_w{wl.w_bits}a8:{M}x{K}x{widths.pop()}*{len(idxs)}")
        elif grouped and len(idxs) > 1:
            return None
        else:
            keys += [f"gemm_w{wl.w_bits}a8:{M}x{K}x{wl.linears[i].N}" for i in idxs]
    vals = [table.get(k) for k in keys]
    if any(v is None for v in vals):
        return None
    return sum(vals) / len(vals)


class ClockSampler:
    """Samples SM clocks and throttle reasons with nvidia-smi while the timed region runs."""

    Q = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
         "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
         "clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.index, self.rows, self.proc = index, [], None

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", f"--id={self.index}", f"--query-gpu={self.Q}", "--format=csv,noheader,nounits",
                 "-lms", "100"], stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            threading.Thread(target=self._read, daemon=True).start()
        except OSError:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.rows.append([c.strip() for c in line.split(",")])

    def stop(self) -> dict:
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        time.sleep(0.15)
        self.proc.terminate()
        rows = [r for r in self.rows if len(r) == 7]
        if not rows:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["no samples"]}
        mhz = [float(r[0]) for r in rows if r[0].replace(".", "").isdigit()]
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        reasons = [n for i, n in enumerate(names) if any(r[3 + i] == "Active" for r in rows)]
        return {"sm_mhz": statistics.median(mhz) if mhz else None, "sm_max_mhz": float(rows[0][1]),
                "power_w_max": max(float(r[2]) for r in rows), "samples": len(rows), "reasons": reasons}


# --------------------------------------------------------------------------- CPU oracle arm

class OracleLayer:
    """One layer of seeded inputs prepared for the CPU oracle (weights packed offline, untimed)."""

    def __init__(self, wl: synth.Workload, M: int, max_rows: int):
        import oracle
        self.wl, self.M, self.max_rows = wl, M, min(max_rows, M)
        self.groups = layer_plan(wl)
        self.x = [synth.activations(self.max_rows, K, wl.seed(idxs[0]), wl.n_outlier) for K, idxs in self.groups]
        self.w = []
        for i, lin in enumerate(wl.linears):
            w = synth.weights(lin.N, lin.K, wl.seed(i))
            self.w.append(oracle.pack_w8(w) if wl.w_bits == 8 else oracle.pack_w4(w, synth.GROUP))

    def run(self, rows: int):
        """Quantize + GEMM + dequant of `rows` token rows through every linear; returns (seconds, ops)."""
        import oracle
        rows = min(rows, self.max_rows)
        t0 = time.perf_counter()
        ops = 0
        for gi, (K, idxs) in enumerate(self.groups):
            q, s_tok = oracle.quantize_act(self.x[gi][:rows])
            for i in idxs:
                lin = self.wl.linears[i]
                a, b = self.w[i]
                if self.wl.w_bits == 8:
                    oracle.gemm_w8a8(q, s_tok, a, b, want_acc=False)
                else:
                    oracle.gemm_w4a8(q, s_tok, a, b, synth.GROUP, want_acc=False)
                ops += 2 * rows * lin.N * lin.K
        return time.perf_counter() - t0, ops


def cpu_baseline(wl: synth.Workload, M: int, budget_s: float = 12.0) -> dict:
    """The oracle as it stands, timed on the host cores on a bounded sample of the workload
    (about `budget_s` seconds of CPU work: a row sample of one layer, repeated if it is short)."""
    import oracle
    layer = OracleLayer(wl, M, M)
    t, ops = layer.run(2)                                  # calibration
    rows = int(max(2, min(layer.max_rows, budget_s * (2 / t))))
    t1, ops1 = layer.run(rows)
    reps = int(max(1, min(50, budget_s / max(t1, 1e-3))))
    t_sum, ops_sum = t1, ops1
    for _ in range(reps - 1):
        t, ops = layer.run(rows)
        t_sum += t
        ops_sum += ops
    return {"value": ops_sum / t_sum / 1e12, "unit": "TOPS", "cores": oracle.num_threads(), "kind": "oracle",
            "sample": f"{rows} of {M} token rows through each of the {len(wl.linears)} linears of one layer "
                      f"(quantize + GEMM + dequant), {reps} passes, {t_sum:.1f} s"}


def run_reference(args, wl: synth.Workload, M: int):
    """`--impl reference`: the CPU oracle on the same workload; every step is a bounded row sample."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    import oracle
    layer = OracleLayer(wl, M, 64)
    t, _ = layer.run(2)
    total_budget_s = 90.0
    rows = int(max(1, min(layer.max_rows, total_budget_s / max(args.steps + args.warmup, 1) * (2 / t))))
    for _ in range(args.warmup):
        layer.run(rows)
    t_sum, ops_sum = 0.0, 0
    for _ in range(args.steps):
        t, ops = layer.run(rows)
        t_sum += t
        ops_sum += ops
    tops = ops_sum / t_sum / 1e12
    sample = f"each step = {rows} of {M} token rows through every linear of one layer (quantize + GEMM + dequant)"
    base = {"value": tops, "unit": "TOPS", "cores": oracle.num_threads(), "kind": "oracle", "sample": sample}
    print(json.dumps({
        "impl": "reference", "metric": "quantized_linear_tops", "value": tops, "unit": "TOPS",
        "n_gpus": args.gpus, "steps": args.steps, "warmup": args.warmup,
        "ms_per_step": t_sum / max(args.steps, 1) * 1e3, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "int8", "data": "synthetic",
        "config": {"workload": wl.name, "M": M, "w_bits": wl.w_bits, "sample": sample},
        "cpu_baseline": base,
        "e2e": {"value": tops, "unit": "TOPS", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }))


# --------------------------------------------------------------------------- GPU arm

class LayerBuffers:
    """Device buffers of one decoder layer: inputs, packed weights, scales, outputs."""

    def __init__(self, pq, torch, wl, M, dev, src_x, src_w):
        self.xs, self.qs, self.s_toks, self.s_invs, self.groups = [], [], [], [], layer_plan(wl)
        for gi, (K, _) in enumerate(self.groups):
            self.xs.append(src_x[gi].clone())
            # column factors for the Eq. 3 quantizer timing (any positive vector has the same cost)
            self.s_invs.append(torch.rand((K,), dtype=torch.float32, device=dev) + 0.5)
            self.qs.append(torch.empty((M, K), dtype=torch.int8, device=dev))
            self.s_toks.append(torch.empty((M,), dtype=torch.float32, device=dev))
        self.static_scale = torch.full((1,), 0.05, dtype=torch.float32, device=dev)   # any calibrated value costs the same
        self.packed, self.ys = [], []
        for i, lin in enumerate(wl.linears):
            self.packed.append(tuple(t.clone() for t in src_w[i]))
            self.ys.append(torch.empty((M, lin.N), dtype=torch.float16, device=dev))


def run_ours(args, wl: synth.Workload, M: int):
    import torch
    import torch.distributed as dist

    import paper_2512_23367_b200 as pq

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py: no CUDA device; this library has no CPU path")
    torch.cuda.set_device(local_rank)
    dev = torch.device("cuda", local_rank)
    if world > 1:
        dist.init_process_group("nccl", device_id=dev)
    pq.lib()

    # One layer of seeded inputs, packed once (offline step); further layers of the rotation are
    # copies in distinct buffers -- only their addresses matter for cache behaviour.
    groups = layer_plan(wl)
    src_x = [torch.from_numpy(synth.activations(M, K, wl.seed(idxs[0]), wl.n_outlier)).to(dev) for K, idxs in groups]
    src_w = []
    for i, lin in enumerate(wl.linears):
        w = torch.from_numpy(synth.weights(lin.N, lin.K, wl.seed(i))).to(dev)
        src_w.append(pq.pq_pack_w8(w) if wl.w_bits == 8 else pq.pq_pack_w4(w))
        del w
    n_layers = layers_for_rotation(wl, M)
    layers = [LayerBuffers(pq, torch, wl, M, dev, src_x, src_w) for _ in range(n_layers)]

    # The grouped calls schedule their members in one launch.
    grouped = not args.no_group

    def run_layer(L: LayerBuffers, only: str | None = None):
        for gi, (K, idxs) in enumerate(L.groups):
            if only == "quantize_smooth":
                pq.pq_quantize_act_smooth(L.xs[gi], L.s_invs[gi], L.qs[gi], L.s_toks[gi])
                continue
            if only == "quantize_static":
                pq.pq_quantize_act_static(L.xs[gi], L.static_scale, L.qs[gi], L.s_toks[gi])
                continue
            if only == "quantize_hadamard":
                pq.pq_quantize_act_hadamard(L.xs[gi], L.qs[gi], L.s_toks[gi])
                continue
            if only != "gemm":
                pq.pq_quantize_act(L.xs[gi], L.qs[gi], L.s_toks[gi])
            if only == "quantize":
                continue
            if grouped and len(idxs) > 1:
                # linears over the same codes (q/k/v, gate/up): one grouped call, one kernel launch
                group_call = pq.pq_gemm_w8a8_group if wl.w_bits == 8 else pq.pq_gemm_w4a8_group
                group_call(L.qs[gi], L.s_toks[gi], [(L.packed[i][0], L.packed[i][1], wl.linears[i].N) for i in idxs],
                           [L.ys[i] for i in idxs])
                continue
            for i in idxs:
                N = wl.linears[i].N
                a, b = L.packed[i]
                if wl.w_bits == 8:
                    pq.pq_gemm_w8a8(L.qs[gi], L.s_toks[gi], a, b, N, y=L.ys[i])
                else:
                    pq.pq_gemm_w4a8(L.qs[gi], L.s_toks[gi], a, b, N, y=L.ys[i])

    gemm_per_layer = sum(1 if grouped and len(idxs) > 1 else len(idxs) for _, idxs in groups)   # GEMM launches
    launches_per_step = len(groups) + gemm_per_layer

    # Eager warm-up (also sets kernel attributes), then one CUDA graph per layer buffer set.
    stream = torch.cuda.Stream(device=dev)
    with torch.cuda.stream(stream):
        for L in layers:
            run_layer(L)
    stream.synchronize()
    graphs = []
    if not args.no_graph:
        for L in layers:
            g = torch.cuda.CUDAGraph()
            with torch.cuda.graph(g, stream=stream):
                run_layer(L)
            graphs.append(g)

    def step(i: int):
        if graphs:
            graphs[i % n_layers].replay()
        else:
            run_layer(layers[i % n_layers])

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    # ---- device-resident throughput
    sampler = ClockSampler(local_rank)
    with torch.cuda.stream(stream):
        for i in range(args.warmup):
            step(i)
        barrier()
        if rank == 0:
            sampler.start()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(stream)
        for i in range(args.steps):
            step(args.warmup + i)
        e1.record(stream)
        barrier()
    clocks = sampler.stop() if rank == 0 else None
    local_ms = e0.elapsed_time(e1)
    ops = step_ops(wl, M)
    total_ms, total_ops = aggregate_over_ranks(local_ms, float(ops) * args.steps, world)

    # ---- per-kernel durations: the same launches on the same buffers, replayed as graphs that hold
    # only the GEMMs (or only the quantizers) of a layer, timed with CUDA events on the launching
    # stream.  Event time / launches = average launch duration of that kernel inside a back-to-back
    # stream of its own kind (launch gaps included, so the figure is conservative).
    def kind_graphs(which: str):
        gs = []
        for L in layers:
            g = torch.cuda.CUDAGraph()
            with torch.cuda.graph(g, stream=stream):
                run_layer(L, only=which)
            gs.append(g)
        return gs

    def time_kind(gs, launches_per_replay: int, budget_ms: float = 400.0):
        with torch.cuda.stream(stream):
            for g in gs:
                g.replay()
            torch.cuda.synchronize()
            a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            a.record(stream)
            for g in gs:
                g.replay()
            b.record(stream)
            torch.cuda.synchronize()
            rounds = int(max(3, min(2000, budget_ms / max(a.elapsed_time(b), 1e-3))))
            a.record(stream)
            for _ in range(rounds):
                for g in gs:
                    g.replay()
            b.record(stream)
            torch.cuda.synchronize()
        n = rounds * len(gs) * launches_per_replay
        return a.elapsed_time(b) / n, n

    gemm_avg_ms, gemm_launches = time_kind(kind_graphs("gemm"), gemm_per_layer)
    quant_avg_ms, quant_launches = time_kind(kind_graphs("quantize"), len(groups))
    smooth_avg_ms, _ = time_kind(kind_graphs("quantize_smooth"), len(groups), budget_ms=200.0)
    hadamard_avg_ms, _ = time_kind(kind_graphs("quantize_hadamard"), len(groups), budget_ms=200.0)
    static_avg_ms, _ = time_kind(kind_graphs("quantize_static"), len(groups), budget_ms=200.0)

    # ---- context (not a target): the same seven shapes as FP16 GEMMs from the vendor library
    # (torch.matmul -> cuBLAS), the comparison the paper's prefill table makes on its own hardware.
    fp16_ctx = None
    if not args.no_fp16_context:
        xs16 = [torch.randn((M, K), dtype=torch.float16, device=dev) for K, _ in groups]
        ws16 = [[torch.randn((lin.N, lin.K), dtype=torch.float16, device=dev) * 0.02 for lin in wl.linears]
                for _ in range(n_layers)]
        ys16 = [torch.empty((M, lin.N), dtype=torch.float16, device=dev) for lin in wl.linears]

        def fp16_layer(ws):
            for gi, (K, idxs) in enumerate(groups):
                for i in idxs:
                    torch.matmul(xs16[gi], ws[i].t(), out=ys16[i])

        with torch.cuda.stream(stream):
            for ws in ws16:
                fp16_layer(ws)
        stream.synchronize()
        gs16 = []
        for ws in ws16:
            g = torch.cuda.CUDAGraph()
            with torch.cuda.graph(g, stream=stream):
                fp16_layer(ws)
            gs16.append(g)
        fp16_avg_ms, _ = time_kind(gs16, len(wl.linears), budget_ms=200.0)
        fp16_ctx = {"kernel": "torch.matmul FP16 (cuBLAS), same shapes", "avg_launch_us": fp16_avg_ms * 1e3,
                    "tflops": ops / (fp16_avg_ms * len(wl.linears) * 1e-3) / 1e12,
                    "int8_over_fp16_speedup": (fp16_avg_ms * len(wl.linears)) / (gemm_avg_ms * gemm_per_layer),
                    "paper_context": "the paper reports 1.2x-1.5x INT8 over FP16 end-to-end prefill on Atlas A2"}
        del xs16, ws16, ys16, gs16
        # The vendor library's own INT8 GEMM (torch._int_mm -> cuBLASLt, INT32 output, no dequantization)
        # on the same shapes: a second context figure, not a target either.
        try:
            xs8 = [torch.randint(-127, 128, (M, K), dtype=torch.int8, device=dev) for K, _ in groups]
            ws8 = [[torch.randint(-127, 128, (lin.N, lin.K), dtype=torch.int8, device=dev) for lin in wl.linears]
                   for _ in range(n_layers)]
            ys8 = [torch.empty((M, lin.N), dtype=torch.int32, device=dev) for lin in wl.linears]

            def int8_layer(ws):
                for gi, (K, idxs) in enumerate(groups):
                    for i in idxs:
                        torch._int_mm(xs8[gi], ws[i].t(), out=ys8[i])

            with torch.cuda.stream(stream):
                for ws in ws8:
                    int8_layer(ws)
            stream.synchronize()
            gs8 = []
            for ws in ws8:
                g = torch.cuda.CUDAGraph()
                with torch.cuda.graph(g, stream=stream):
                    int8_layer(ws)
                gs8.append(g)
            lib8_avg_ms, _ = time_kind(gs8, len(wl.linears), budget_ms=200.0)
            fp16_ctx["library_int8"] = {
                "kernel": "torch._int_mm (cuBLASLt INT8 -> INT32, no dequantization), same shapes",
                "tops": ops / (lib8_avg_ms * len(wl.linears) * 1e-3) / 1e12,
                "ours_over_library": (lib8_avg_ms * len(wl.linears)) / (gemm_avg_ms * gemm_per_layer)}
            del xs8, ws8, ys8, gs8
        except Exception as e:   # the library call is context only: its absence must not fail the benchmark
            fp16_ctx["library_int8"] = {"unavailable": f"{type(e).__name__}: {str(e)[:120]}"}
    gemm_tops = ops / (gemm_avg_ms * gemm_per_layer * 1e-3) / 1e12
    sbytes = step_bytes(wl, M)
    quant_gbs = sbytes["quantize"] / (quant_avg_ms * len(groups) * 1e-3) / 1e9
    smooth_bytes = sbytes["quantize"] + sum(4 * K for K, _ in groups)   # + the [K] FP32 factor vector per call
    smooth_gbs = smooth_bytes / (smooth_avg_ms * len(groups) * 1e-3) / 1e9
    hadamard_gbs = sbytes["quantize"] / (hadamard_avg_ms * len(groups) * 1e-3) / 1e9
    static_gbs = sbytes["quantize"] / (static_avg_ms * len(groups) * 1e-3) / 1e9

    # ---- end to end: pinned host inputs -> device -> quantize + GEMMs -> pinned host outputs
    L0 = layers[0]
    host_x = [x.cpu().pin_memory() for x in L0.xs]
    host_y = [torch.empty(y.shape, dtype=y.dtype).pin_memory() for y in L0.ys]
    h2d = sum(x.numel() * 2 for x in host_x)
    d2h = sum(y.numel() * 2 for y in host_y)
    e2e_steps = max(3, min(args.steps, 20))

    # Three streams: copy-in of step i+1, compute of step i and copy-out of step i-1 overlap (PCIe
    # is full duplex).  A layer buffer set is reused every n_layers steps; events keep a step from
    # overwriting inputs still being read or outputs still being copied out.
    s_in, s_out = torch.cuda.Stream(device=dev), torch.cuda.Stream(device=dev)
    comp_done: dict[int, torch.cuda.Event] = {}
    out_done: dict[int, torch.cuda.Event] = {}

    def e2e_step(i: int):
        L = layers[i % n_layers]
        prev = i - n_layers
        with torch.cuda.stream(s_in):
            if prev in comp_done:
                s_in.wait_event(comp_done[prev])        # the set's inputs are no longer being read
            for hx, dx in zip(host_x, L.xs):
                dx.copy_(hx, non_blocking=True)
            in_done = torch.cuda.Event()
            in_done.record(s_in)
        with torch.cuda.stream(stream):
            stream.wait_event(in_done)
            if prev in out_done:
                stream.wait_event(out_done[prev])       # the set's outputs have been copied out
            run_layer(L)
            comp_done[i] = torch.cuda.Event()
            comp_done[i].record(stream)
        with torch.cuda.stream(s_out):
            s_out.wait_event(comp_done[i])
            for hy, dy in zip(host_y, L.ys):
                hy.copy_(dy, non_blocking=True)
            out_done[i] = torch.cuda.Event()
            out_done[i].record(s_out)
        comp_done.pop(prev - n_layers, None)
        out_done.pop(prev - n_layers, None)

    def join_all():
        stream.wait_stream(s_in)
        stream.wait_stream(s_out)

    for i in range(3):
        e2e_step(i)
    join_all()
    barrier()
    f0, f1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    f0.record(stream)
    s_in.wait_event(f0)
    s_out.wait_event(f0)
    for i in range(e2e_steps):
        e2e_step(3 + i)
    join_all()
    f1.record(stream)
    barrier()
    e2e_ms, e2e_ops = aggregate_over_ranks(f0.elapsed_time(f1), float(ops) * e2e_steps, world)

    status = pq.pq_device_status()
    if status != 0:
        raise SystemExit(f"bench.py: device status {status} after the timed region")

    if rank == 0:
        peaks, peak_kind = load_peaks()
        if wl.w_bits and M > 64:
            peak = 2.0 * float(peaks["bf16_tflops"])
            roof = {"bound": "tensor", "achieved": gemm_tops, "peak": peak, "unit": "TOPS",
                    "frac": gemm_tops / peak, "traffic": load_traffic(wl, M, grouped),
                    "kernel": f"gemm_w{wl.w_bits}a8 (tcgen05 kind::i8)",
                    "peak_kind": f"2 x bf16_tflops (burst) of {peak_kind}: INT8 peak = bf16 peak x nominal 4.5/2.25",
                    "frac_of_sustained": gemm_tops / (2.0 * float(peaks["bf16_tflops_sustained"])),
                    "frac_of_datasheet_4500": gemm_tops / DATASHEET_INT8_TOPS,
                    "avg_launch_us": gemm_avg_ms * 1e3, "launches_timed": gemm_launches}
        else:
            gbs = sbytes["gemm"] / (gemm_avg_ms * gemm_per_layer * 1e-3) / 1e9
            peak = float(peaks["hbm_gbs"])
            roof = {"bound": "hbm", "achieved": gbs, "peak": peak, "unit": "GB/s", "frac": gbs / peak,
                    "traffic": load_traffic(wl, M, grouped),
                    "kernel": f"small-M gemm_w{wl.w_bits}a8", "peak_kind": f"hbm_gbs of {peak_kind}",
                    "avg_launch_us": gemm_avg_ms * 1e3, "launches_timed": gemm_launches}
        decode = M <= 64
        if decode:
            metric, unit = "quantized_linear_gbs", "GB/s"
            per_step = sbytes["gemm"] + sbytes["quantize"]
            value = per_step * args.steps * world / (total_ms * 1e-3) / 1e9
            e2e_value = per_step * e2e_steps * world / (e2e_ms * 1e-3) / 1e9
        else:
            metric, unit = "quantized_linear_tops", "TOPS"
            value = total_ops / (total_ms * 1e-3) / 1e12
            e2e_value = e2e_ops / (e2e_ms * 1e-3) / 1e12
        out = {
            "metric": metric, "value": value, "unit": unit, "n_gpus": world, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": total_ms / args.steps, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "int8", "data": "synthetic",
            "config": {"workload": wl.name, "M": M, "w_bits": wl.w_bits,
                       "linears": [[lin.name, lin.K, lin.N] for lin in wl.linears],
                       "step": f"{len(groups)} activation quantizations + {len(wl.linears)} quantized linears "
                               f"(one decoder layer) in {launches_per_step} kernel launches",
                       "grouped_calls": bool(grouped),
                       "cache": f"rotation over {n_layers} distinct layer buffer sets (> 2 x L2)",
                       "launch": "cuda_graph_per_layer" if graphs else "eager", "parallelism": "replicas"},
            "roofline": roof,
            "fp16_context": fp16_ctx,
            "quantize": {"achieved_gbs": quant_gbs, "frac_of_hbm": quant_gbs / float(peaks["hbm_gbs"]),
                         "avg_launch_us": quant_avg_ms * 1e3, "launches_timed": quant_launches},
            "quantize_smooth": {"achieved_gbs": smooth_gbs, "frac_of_hbm": smooth_gbs / float(peaks["hbm_gbs"]),
                                "avg_launch_us": smooth_avg_ms * 1e3,
                                "what": "pq_quantize_act_smooth (Eq. 3: X S^-1) on the same inputs; not part of the step"},
            "quantize_hadamard": {"achieved_gbs": hadamard_gbs, "frac_of_hbm": hadamard_gbs / float(peaks["hbm_gbs"]),
                                  "avg_launch_us": hadamard_avg_ms * 1e3,
                                  "what": "pq_quantize_act_hadamard (Eq. 4: X H) on the same inputs; not part of the step"},
            "quantize_static": {"achieved_gbs": static_gbs, "frac_of_hbm": static_gbs / float(peaks["hbm_gbs"]),
                                "avg_launch_us": static_avg_ms * 1e3,
                                "what": "pq_quantize_act_static (one calibrated scale) on the same inputs; not part of the step"},
            "e2e": {"value": e2e_value, "unit": unit, "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h,
                    "steps": e2e_steps, "overlap": "copy-in, compute and copy-out on three streams"},
            "gpu_launches": launches_per_step * args.steps,
            "clocks": clocks,
        }
        if not args.no_cpu_baseline and world == 1:
            out["cpu_baseline"] = cpu_baseline(wl, M)
        print(json.dumps(out))
    if world > 1:
        dist.destroy_process_group()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20000)
    ap.add_argument("--warmup", type=int, default=50)
    ap.add_argument("--impl", choices=["ours", "reference"], default="ours")
    ap.add_argument("--workload", default=DEFAULT_WORKLOAD, choices=sorted(synth.WORKLOADS))
    ap.add_argument("--M", type=int, default=None, help="token count (default: the workload's largest)")
    ap.add_argument("--no-graph", action="store_true", help="launch eagerly instead of replaying CUDA graphs")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-group", action="store_true",
                    help="one GEMM call per linear instead of grouped calls for linears that share their input")
    ap.add_argument("--no-fp16-context", action="store_true", help="skip the cuBLAS FP16 same-shape timing")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3) if args.impl == "ours" else args.warmup
    wl = synth.WORKLOADS[args.workload]
    M = args.M if args.M is not None else max(wl.Ms)
    if args.impl == "reference":
        run_reference(args, wl, M)
    else:
        run_ours(args, wl, M)


if __name__ == "__main__":
    main()
