#!/usr/bin/env python
"""Benchmark of the quantized linear layer on B200.

A *step* is one pass of the whole hot path over one decoder layer's worth of synthetic
input: the activation quantizer for each distinct layer input (the q/k/v projections share
one input, gate/up share one) followed by the seven quantized linears.  Layers rotate through
distinct weight/activation buffers whose total exceeds twice the L2 size, so no step finds
its operands cached.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload NAME] [--impl ours|reference]

Prints ONE JSON line.  The timed region of K steps is repeated (each repetition bracketed by a barrier
and a device synchronization) until at least half a second has been timed; `ms_per_step` is the median
over the repetitions and `value` the whole-step throughput that follows from it, inputs resident on the
device (TOPS for prefill workloads, GB/s of algorithmic bytes for decode workloads).  `roofline` = the
GEMM launches alone against the measured peak (and against the datasheet figure); `workloads` = the same
two figures for the other benchmark configurations (1B-class layer, 7B-class layer at M = 512, W4A8, the
decode sweep for both weight formats), each timed for at least 0.3 s; `quantize*` = the quantizer and its
variants against the measured copy rate; `e2e` = the same step with pinned-host inputs copied in and
outputs copied out; `cpu_baseline` = the CPU oracle on a row sample; `clocks` = SM clocks and throttle
reasons sampled over the whole timed span.
`--impl reference` times the CPU oracle instead (a deliberately plain program; a baseline, not a target).
Linears that share their input are issued as one grouped call (`--no-group`: one call per linear).

    python bench.py --one-op gemm_w8a8 --shape M,K,N [--members G] [--eager 3]

runs ONE operation on one seeded shape: with --eager a few plain launches (for profilers: one kernel, few
launches, bounded memory), otherwise a timed CUDA-graph replay of back-to-back launches that rotate over
buffer sets larger than twice the L2.
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
DEFAULT_WORKLOAD = "c3_w8a8_7b_prefill"      # at its largest token count (M = 4096): the largest single-GPU configuration
# The other benchmark configurations, reported in the `workloads` block of the same JSON line.
SIDE_WORKLOADS = (
    [("c2_w8a8_1b_prefill", 2048), ("c3_w8a8_7b_prefill", 512), ("c4_w4a8_7b_prefill", 2048)]
    + [("c5_w8a8_7b_decode", m) for m in (1, 4, 16, 64)]
    + [("c5_w4a8_7b_decode", m) for m in (1, 4, 16, 64)]
)
NOMINAL_HBM_GBS = 8000.0
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
    quant = 0
    for K, idxs in layer_plan(wl):
        fused = wl.chain and wl.linears[idxs[0]].name == "down_proj"     # reads gate and up (4 B), writes codes (1 B)
        quant += (5 if fused else 3) * M * K + 4 * M
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


def gemm_launches(wl: synth.Workload, grouped: bool):
    """The GEMM launches of one step: [(K, [widths])] -- one entry per kernel launch."""
    out = []
    for K, idxs in layer_plan(wl):
        if grouped and len(idxs) > 1:
            out.append((K, [wl.linears[i].N for i in idxs]))
        else:
            out += [(K, [wl.linears[i].N]) for i in idxs]
    return out


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

    def __init__(self, torch, wl, M, dev, src_x, src_w):
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


class GpuWorkload:
    """One benchmark configuration resident on the device: seeded inputs, packed weights, the rotation of
    layer buffer sets, the workspace of the compute stream, and CUDA graphs of the step and of its parts."""

    def __init__(self, pq, torch, wl: synth.Workload, M: int, dev, stream, grouped: bool, use_graphs: bool = True):
        self.pq, self.torch, self.wl, self.M, self.dev, self.stream = pq, torch, wl, M, dev, stream
        self.grouped, self.groups = grouped, layer_plan(wl)
        names = [lin.name for lin in wl.linears]
        self.i_gate = names.index("gate_proj") if "gate_proj" in names else -1
        self.i_up = names.index("up_proj") if "up_proj" in names else -1
        # One layer of seeded inputs, packed once (offline step); further layers of the rotation are
        # copies in distinct buffers -- only their addresses matter for cache behaviour.
        src_x = [torch.from_numpy(synth.activations(M, K, wl.seed(idxs[0]), wl.n_outlier)).to(dev) for K, idxs in self.groups]
        src_w = []
        for i, lin in enumerate(wl.linears):
            w = torch.from_numpy(synth.weights(lin.N, lin.K, wl.seed(i))).to(dev)
            src_w.append(pq.pq_pack_w8(w) if wl.w_bits == 8 else pq.pq_pack_w4(w))
            del w
        self.n_layers = layers_for_rotation(wl, M)
        self.layers = [LayerBuffers(torch, wl, M, dev, src_x, src_w) for _ in range(self.n_layers)]
        self.launches = gemm_launches(wl, grouped)
        self.gemm_per_layer = len(self.launches)
        self.launches_per_step = len(self.groups) + self.gemm_per_layer
        # Split-K scratch of the compute stream (W8A8 with few tiles and a long K): the caller's to
        # provide, sized for the largest need among the step's launches; None when no launch splits.
        need = max([pq.pq_workspace_bytes(M, Ns, K) for K, Ns in self.launches]) if wl.w_bits == 8 else 0
        self.workspace = pq.pq_workspace_init(torch.empty((need,), dtype=torch.uint8, device=dev)) if need else None
        self.workspace_bytes = need
        # Eager warm-up (also sets kernel attributes), then one CUDA graph per layer buffer set.
        with torch.cuda.stream(stream):
            for L in self.layers:
                self.run_layer(L)
        stream.synchronize()
        self.use_graphs = use_graphs
        self.graphs = self.kind_graphs(None) if use_graphs else []

    def run_layer(self, L: LayerBuffers, only: str | None = None):
        pq, wl = self.pq, self.wl
        for gi, (K, idxs) in enumerate(L.groups):
            if only == "linear":
                # every linear as ONE call (quantizer + GEMM; one launch where the row kernel serves)
                for i in idxs:
                    a, b = L.packed[i]
                    if wl.w_bits == 8:
                        pq.pq_linear_w8a8(L.xs[gi], a, b, wl.linears[i].N, y=L.ys[i], q_tmp=L.qs[gi], s_tok_tmp=L.s_toks[gi],
                                          workspace=self.workspace)
                    else:
                        pq.pq_linear_w4a8(L.xs[gi], a, b, wl.linears[i].N, y=L.ys[i], q_tmp=L.qs[gi], s_tok_tmp=L.s_toks[gi])
                continue
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
                if wl.chain and wl.linears[idxs[0]].name == "down_proj":
                    # the layer as a chain: SwiGLU of this step's gate/up outputs, quantized in the same pass
                    pq.pq_swiglu_quantize(L.ys[self.i_gate], L.ys[self.i_up], L.qs[gi], L.s_toks[gi])
                else:
                    pq.pq_quantize_act(L.xs[gi], L.qs[gi], L.s_toks[gi])
            if only == "quantize":
                continue
            if self.grouped and len(idxs) > 1:
                # linears over the same codes (q/k/v, gate/up): one grouped call, one kernel launch
                members = [(L.packed[i][0], L.packed[i][1], wl.linears[i].N) for i in idxs]
                if wl.w_bits == 8:
                    pq.pq_gemm_w8a8_group(L.qs[gi], L.s_toks[gi], members, [L.ys[i] for i in idxs], workspace=self.workspace)
                else:
                    pq.pq_gemm_w4a8_group(L.qs[gi], L.s_toks[gi], members, [L.ys[i] for i in idxs])
                continue
            for i in idxs:
                N = wl.linears[i].N
                a, b = L.packed[i]
                if wl.w_bits == 8:
                    pq.pq_gemm_w8a8(L.qs[gi], L.s_toks[gi], a, b, N, y=L.ys[i], workspace=self.workspace)
                else:
                    pq.pq_gemm_w4a8(L.qs[gi], L.s_toks[gi], a, b, N, y=L.ys[i])

    def kind_graphs(self, which: str | None):
        """One CUDA graph per layer buffer set holding the whole step (which=None) or only its GEMMs /
        only its quantizers (same buffers, same launch configuration)."""
        torch, gs = self.torch, []
        for L in self.layers:
            g = torch.cuda.CUDAGraph()
            with torch.cuda.graph(g, stream=self.stream):
                self.run_layer(L, only=which)
            gs.append(g)
        return gs

    def step(self, i: int):
        if self.graphs:
            self.graphs[i % self.n_layers].replay()
        else:
            self.run_layer(self.layers[i % self.n_layers])

    def time_replays(self, gs, launches_per_replay: int, min_ms: float):
        """Average launch duration (ms) of the kernels in `gs`, replayed back to back on the launching
        stream and timed with CUDA events there: event time / launches (launch gaps included, so the
        figure is conservative).  Repeats until at least `min_ms` have been timed."""
        torch, stream = self.torch, self.stream
        with torch.cuda.stream(stream):
            for _ in range(3):
                for g in gs:
                    g.replay()
            torch.cuda.synchronize()
            a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            a.record(stream)
            for g in gs:
                g.replay()
            b.record(stream)
            torch.cuda.synchronize()
            rounds = int(max(3, min(20000, 1.1 * min_ms / max(a.elapsed_time(b), 1e-3))))
            a.record(stream)
            for _ in range(rounds):
                for g in gs:
                    g.replay()
            b.record(stream)
            torch.cuda.synchronize()
        n = rounds * len(gs) * launches_per_replay
        return a.elapsed_time(b) / n, n

    def roofline(self, gemm_avg_ms: float, gemm_launches_timed: int, peaks: dict, peak_kind: str) -> dict:
        """The GEMM launches of the step against the roofline that bounds them."""
        wl, M = self.wl, self.M
        if M > 64:
            tops = step_ops(wl, M) / (gemm_avg_ms * self.gemm_per_layer * 1e-3) / 1e12
            peak = 2.0 * float(peaks["bf16_tflops"])
            return {"bound": "tensor", "achieved": tops, "peak": peak, "unit": "TOPS", "frac": tops / peak,
                    "traffic": load_traffic(wl, M, self.grouped),
                    "kernel": f"gemm_w{wl.w_bits}a8 (tcgen05 kind::i8)",
                    "peak_kind": f"2 x bf16_tflops (burst) of {peak_kind}: INT8 peak = bf16 peak x nominal 4.5/2.25",
                    "frac_of_sustained": tops / (2.0 * float(peaks["bf16_tflops_sustained"])),
                    "frac_of_datasheet_4500": tops / DATASHEET_INT8_TOPS,
                    "avg_launch_us": gemm_avg_ms * 1e3, "launches_timed": gemm_launches_timed}
        gbs = step_bytes(wl, M)["gemm"] / (gemm_avg_ms * self.gemm_per_layer * 1e-3) / 1e9
        peak = float(peaks["hbm_gbs"])
        return {"bound": "hbm", "achieved": gbs, "peak": peak, "unit": "GB/s", "frac": gbs / peak,
                "traffic": load_traffic(wl, M, self.grouped),
                "kernel": f"small-M gemm_w{wl.w_bits}a8", "peak_kind": f"hbm_gbs of {peak_kind}",
                "frac_of_nominal_8000": gbs / NOMINAL_HBM_GBS,
                "avg_launch_us": gemm_avg_ms * 1e3, "launches_timed": gemm_launches_timed}

    def value_of(self, ms_per_step: float, world: int = 1):
        """(metric, unit, value) of the whole job for a step time."""
        wl, M = self.wl, self.M
        if M <= 64:
            b = step_bytes(wl, M)
            return "quantized_linear_gbs", "GB/s", (b["gemm"] + b["quantize"]) * world / (ms_per_step * 1e-3) / 1e9
        return "quantized_linear_tops", "TOPS", step_ops(wl, M) * world / (ms_per_step * 1e-3) / 1e12


def side_workload(pq, torch, name: str, M: int, dev, stream, grouped: bool, peaks, peak_kind, min_ms: float = 300.0) -> dict:
    """Whole-step throughput and GEMM-only roofline of one more benchmark configuration."""
    wl = synth.WORKLOADS[name]
    w = GpuWorkload(pq, torch, wl, M, dev, stream, grouped)
    step_ms, _ = w.time_replays(w.graphs, 1, min_ms)
    gemm_ms, n = w.time_replays(w.kind_graphs("gemm"), w.gemm_per_layer, min_ms)
    quant_ms, _ = w.time_replays(w.kind_graphs("quantize"), len(w.groups), min_ms / 3)
    _, unit, value = w.value_of(step_ms)
    roof = w.roofline(gemm_ms, n, peaks, peak_kind)
    quant_gbs = step_bytes(wl, M)["quantize"] / (quant_ms * len(w.groups) * 1e-3) / 1e9
    out = {"workload": name, "M": M, "w_bits": wl.w_bits, "value": value, "unit": unit, "ms_per_step": step_ms,
           "launches_per_step": w.launches_per_step, "frac": roof["frac"], "avg_launch_us": roof["avg_launch_us"],
           "roofline": roof, "quantize_frac_of_hbm": quant_gbs / float(peaks["hbm_gbs"]),
           "rotation_layers": w.n_layers}
    if M <= 4:
        # the same step with every linear as one call (pq_linear_*: the row kernel quantizes its own tokens)
        lin_ms, _ = w.time_replays(w.kind_graphs("linear"), 1, min_ms)
        out["one_call_linear"] = {"ms_per_step": lin_ms, "value": w.value_of(lin_ms)[2], "unit": unit,
                                  "calls_per_step": sum(len(idxs) for _, idxs in w.groups)}
    return out


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
    peaks, peak_kind = load_peaks()

    grouped = not args.no_group
    stream = torch.cuda.Stream(device=dev)
    W = GpuWorkload(pq, torch, wl, M, dev, stream, grouped, use_graphs=not args.no_graph)
    groups, n_layers, layers = W.groups, W.n_layers, W.layers

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    # ---- device-resident throughput: rounds of exactly `steps` steps, each bracketed by a barrier and a
    # device synchronization and timed with CUDA events on the launching stream, repeated until at least
    # MIN_TIMED_MS have been timed; the clock sampler runs over the whole span.
    MIN_TIMED_MS, MAX_ROUNDS = 500.0, 400
    sampler = ClockSampler(local_rank)
    round_ms = []
    with torch.cuda.stream(stream):
        for i in range(args.warmup):
            W.step(i)
        barrier()
        if rank == 0:
            sampler.start()
        it = args.warmup
        while True:
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            barrier()
            e0.record(stream)
            for i in range(args.steps):
                W.step(it + i)
            e1.record(stream)
            barrier()
            it += args.steps
            local = e0.elapsed_time(e1)
            total_ms, _ = aggregate_over_ranks(local, 0.0, world)     # max over ranks: the same on every rank
            round_ms.append(total_ms)
            if sum(round_ms) >= MIN_TIMED_MS or len(round_ms) >= MAX_ROUNDS:
                break
    clocks = sampler.stop() if rank == 0 else None
    ms_per_step = statistics.median(round_ms) / args.steps
    ops = step_ops(wl, M)

    # ---- per-kernel durations: the same launches on the same buffers, replayed as graphs that hold
    # only the GEMMs (or only the quantizers) of a layer.
    gemm_per_layer = W.gemm_per_layer
    gemm_avg_ms, gemm_launches_timed = W.time_replays(W.kind_graphs("gemm"), gemm_per_layer, 400.0)
    quant_avg_ms, quant_launches = W.time_replays(W.kind_graphs("quantize"), len(groups), 300.0)
    smooth_avg_ms, _ = W.time_replays(W.kind_graphs("quantize_smooth"), len(groups), 150.0)
    hadamard_avg_ms, _ = W.time_replays(W.kind_graphs("quantize_hadamard"), len(groups), 150.0)
    static_avg_ms, _ = W.time_replays(W.kind_graphs("quantize_static"), len(groups), 150.0)

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
        fp16_avg_ms, _ = W.time_replays(gs16, len(wl.linears), 200.0)
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
            lib8_avg_ms, _ = W.time_replays(gs8, len(wl.linears), 200.0)
            fp16_ctx["library_int8"] = {
                "kernel": "torch._int_mm (cuBLASLt INT8 -> INT32, no dequantization), same shapes",
                "tops": ops / (lib8_avg_ms * len(wl.linears) * 1e-3) / 1e12,
                "ours_over_library": (lib8_avg_ms * len(wl.linears)) / (gemm_avg_ms * gemm_per_layer)}
            del xs8, ws8, ys8, gs8
        except Exception as e:   # the library call is context only: its absence must not fail the benchmark
            fp16_ctx["library_int8"] = {"unavailable": f"{type(e).__name__}: {str(e)[:120]}"}
    # ---- the layer as a chain against the same chain in FP16 (cuBLAS GEMMs + torch's SwiGLU): the analogue
    # of the paper's prefill-latency comparison, here per decoder layer (attention itself left out on both sides).
    chain_ctx = None
    if wl.chain and not args.no_fp16_context:
        xs16 = [torch.randn((M, K), dtype=torch.float16, device=dev) for K, _ in groups]
        ws16 = [[torch.randn((lin.N, lin.K), dtype=torch.float16, device=dev) * 0.02 for lin in wl.linears]
                for _ in range(n_layers)]
        ys16 = [torch.empty((M, lin.N), dtype=torch.float16, device=dev) for lin in wl.linears]
        h16 = torch.empty((M, wl.linears[W.i_gate].N), dtype=torch.float16, device=dev)

        def fp16_chain(ws):
            for gi, (K, idxs) in enumerate(groups):
                for i in idxs:
                    if wl.linears[i].name == "down_proj":
                        torch.mul(torch.nn.functional.silu(ys16[W.i_gate]), ys16[W.i_up], out=h16)
                        torch.matmul(h16, ws[i].t(), out=ys16[i])
                    else:
                        torch.matmul(xs16[gi], ws[i].t(), out=ys16[i])

        with torch.cuda.stream(stream):
            for ws in ws16:
                fp16_chain(ws)
        stream.synchronize()
        gs16 = []
        for ws in ws16:
            g = torch.cuda.CUDAGraph()
            with torch.cuda.graph(g, stream=stream):
                fp16_chain(ws)
            gs16.append(g)
        fp16_layer_ms, _ = W.time_replays(gs16, 1, 300.0)
        chain_ctx = {"ms_per_layer": ms_per_step, "fp16_ms_per_layer": fp16_layer_ms,
                     "int8_over_fp16": fp16_layer_ms / ms_per_step,
                     "fp16_chain": "torch.matmul x 7 + silu(gate) * up, CUDA graph, same rotation of weights",
                     "paper_context": "Table 3 of the paper: INT8 prefill 1.20x (batch 2) to 1.50x (batch 32) faster than FP16 on Atlas A2"}
        del xs16, ws16, ys16, gs16, h16
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
            W.run_layer(L)
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
    e2e_ms, _ = aggregate_over_ranks(f0.elapsed_time(f1), 0.0, world)

    status = pq.pq_device_status()
    if status != 0:
        raise SystemExit(f"bench.py: device status {status} after the timed region")

    # ---- the other benchmark configurations (single GPU only: a scaling run repeats the main workload)
    side = None
    if world == 1 and not args.no_side_workloads:
        del host_x, host_y
        side = []
        for name, m in SIDE_WORKLOADS:
            if name == wl.name and m == M:
                continue
            torch.cuda.empty_cache()
            side.append(side_workload(pq, torch, name, m, dev, stream, grouped, peaks, peak_kind))
        status = pq.pq_device_status()
        if status != 0:
            raise SystemExit(f"bench.py: device status {status} after the side workloads")

    if rank == 0:
        roof = W.roofline(gemm_avg_ms, gemm_launches_timed, peaks, peak_kind)
        metric, unit, value = W.value_of(ms_per_step, world)
        _, _, e2e_value = W.value_of(e2e_ms / e2e_steps, world)
        hbm = float(peaks["hbm_gbs"])
        out = {
            "metric": metric, "value": value, "unit": unit, "n_gpus": world, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": ms_per_step, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "int8", "data": "synthetic",
            "config": {"workload": wl.name, "M": M, "w_bits": wl.w_bits,
                       "linears": [[lin.name, lin.K, lin.N] for lin in wl.linears],
                       "step": f"{len(groups)} activation quantizations + {len(wl.linears)} quantized linears "
                               f"(one decoder layer) in {W.launches_per_step} kernel launches",
                       "grouped_calls": bool(grouped),
                       "cache": f"rotation over {n_layers} distinct layer buffer sets (> 2 x L2)",
                       "launch": "cuda_graph_per_layer" if W.graphs else "eager", "parallelism": "replicas",
                       "workspace_bytes": W.workspace_bytes},
            "timing": {"rounds": len(round_ms), "steps_per_round": args.steps, "timed_ms_total": sum(round_ms),
                       "ms_per_step_min": min(round_ms) / args.steps, "ms_per_step_max": max(round_ms) / args.steps,
                       "ms_per_step": "median over rounds"},
            "roofline": roof,
            "workloads": side,
            "fp16_context": fp16_ctx,
            "layer_chain": chain_ctx,
            "quantize": {"achieved_gbs": quant_gbs, "frac_of_hbm": quant_gbs / hbm,
                         "avg_launch_us": quant_avg_ms * 1e3, "launches_timed": quant_launches},
            "quantize_smooth": {"achieved_gbs": smooth_gbs, "frac_of_hbm": smooth_gbs / hbm,
                                "avg_launch_us": smooth_avg_ms * 1e3,
                                "what": "pq_quantize_act_smooth (Eq. 3: X S^-1) on the same inputs; not part of the step"},
            "quantize_hadamard": {"achieved_gbs": hadamard_gbs, "frac_of_hbm": hadamard_gbs / hbm,
                                  "avg_launch_us": hadamard_avg_ms * 1e3,
                                  "what": "pq_quantize_act_hadamard (Eq. 4: X H) on the same inputs; not part of the step"},
            "quantize_static": {"achieved_gbs": static_gbs, "frac_of_hbm": static_gbs / hbm,
                                "avg_launch_us": static_avg_ms * 1e3,
                                "what": "pq_quantize_act_static (one calibrated scale) on the same inputs; not part of the step"},
            "e2e": {"value": e2e_value, "unit": unit, "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h,
                    "steps": e2e_steps, "overlap": "copy-in, compute and copy-out on three streams"},
            "gpu_launches": W.launches_per_step * args.steps,
            "clocks": clocks,
        }
        if not args.no_cpu_baseline and world == 1:
            out["cpu_baseline"] = cpu_baseline(wl, M)
        print(json.dumps(out))
    if world > 1:
        dist.destroy_process_group()


# --------------------------------------------------------------------------- one operation (profilers, per-shape timing)

QUANT_OPS = ("quantize", "quantize_smooth", "quantize_hadamard", "quantize_static", "swiglu_quantize")
# linear_*: the one-call linear (quantizer + GEMM; one launch where the row kernel serves); quant_gemm_*: the
# same work as two calls (the time per PAIR of launches), for comparison
LINEAR_OPS = ("linear_w8a8", "linear_w4a8", "quant_gemm_w8a8", "quant_gemm_w4a8")
ONE_OPS = QUANT_OPS + ("gemm_w8a8", "gemm_w4a8") + LINEAR_OPS


def run_one_op(args):
    """ONE operation on one seeded shape.  --eager n: n plain launches and exit (for profilers);
    otherwise a CUDA graph of back-to-back launches rotating over buffer sets > 2 x L2, timed with events."""
    import torch

    import paper_2512_23367_b200 as pq

    op = args.one_op
    dims = [int(v) for v in args.shape.split(",")]
    M, K = dims[0], dims[1]
    N = dims[2] if len(dims) > 2 else 0
    G = max(args.members, 1)
    if op not in QUANT_OPS and N <= 0:
        raise SystemExit("bench.py --one-op gemm_*: --shape M,K,N")
    dev = torch.device("cuda", 0)
    torch.cuda.set_device(dev)
    per_set = (5 if op == "swiglu_quantize" else 3) * M * K + (G * N * K if op not in QUANT_OPS else 0)
    sets = args.sets or max(2, min(16, (2 * L2_BYTES) // max(per_set, 1) + 1))
    x = torch.from_numpy(synth.activations(M, K, 9000)).to(dev)
    packed = []
    for g in range(G if op not in QUANT_OPS else 0):
        w = torch.from_numpy(synth.weights(N, K, 9001 + g)).to(dev)
        packed.append(pq.pq_pack_w8(w) if op.endswith("w8a8") else pq.pq_pack_w4(w))
        del w
    need = pq.pq_workspace_bytes(M, [N] * G, K) if op.endswith("w8a8") else 0
    ws = pq.pq_workspace_init(torch.empty((need,), dtype=torch.uint8, device=dev)) if need else None
    bufs = []
    for _ in range(sets):
        xc = x.clone()
        q, s_tok = pq.pq_quantize_act(xc)
        b = {"x": xc, "q": q, "s_tok": s_tok, "up": (xc * 0.5).contiguous() if op == "swiglu_quantize" else None, "s_inv": torch.rand((K,), device=dev, dtype=torch.float32) + 0.5,
             "scale": torch.full((1,), 0.05, device=dev, dtype=torch.float32),
             "w": [tuple(t.clone() for t in p) for p in packed],
             "y": [torch.empty((M, N), device=dev, dtype=torch.float16) for _ in packed]}
        bufs.append(b)

    def launch(i):
        b = bufs[i % sets]
        if op == "quantize":
            pq.pq_quantize_act(b["x"], b["q"], b["s_tok"])
        elif op == "quantize_smooth":
            pq.pq_quantize_act_smooth(b["x"], b["s_inv"], b["q"], b["s_tok"])
        elif op == "quantize_hadamard":
            pq.pq_quantize_act_hadamard(b["x"], b["q"], b["s_tok"])
        elif op == "quantize_static":
            pq.pq_quantize_act_static(b["x"], b["scale"], b["q"], b["s_tok"])
        elif op == "swiglu_quantize":
            pq.pq_swiglu_quantize(b["x"], b["up"], b["q"], b["s_tok"])
        elif op == "linear_w8a8":
            pq.pq_linear_w8a8(b["x"], b["w"][0][0], b["w"][0][1], N, y=b["y"][0], q_tmp=b["q"], s_tok_tmp=b["s_tok"], workspace=ws)
        elif op == "linear_w4a8":
            pq.pq_linear_w4a8(b["x"], b["w"][0][0], b["w"][0][1], N, y=b["y"][0], q_tmp=b["q"], s_tok_tmp=b["s_tok"])
        elif op == "quant_gemm_w8a8":
            pq.pq_quantize_act(b["x"], b["q"], b["s_tok"])
            pq.pq_gemm_w8a8(b["q"], b["s_tok"], b["w"][0][0], b["w"][0][1], N, y=b["y"][0], workspace=ws)
        elif op == "quant_gemm_w4a8":
            pq.pq_quantize_act(b["x"], b["q"], b["s_tok"])
            pq.pq_gemm_w4a8(b["q"], b["s_tok"], b["w"][0][0], b["w"][0][1], N, y=b["y"][0])
        elif G > 1 and op == "gemm_w8a8":
            pq.pq_gemm_w8a8_group(b["q"], b["s_tok"], [(w[0], w[1], N) for w in b["w"]], b["y"], workspace=ws)
        elif G > 1:
            pq.pq_gemm_w4a8_group(b["q"], b["s_tok"], [(w[0], w[1], N) for w in b["w"]], b["y"])
        elif op == "gemm_w8a8":
            pq.pq_gemm_w8a8(b["q"], b["s_tok"], b["w"][0][0], b["w"][0][1], N, y=b["y"][0], workspace=ws)
        else:
            pq.pq_gemm_w4a8(b["q"], b["s_tok"], b["w"][0][0], b["w"][0][1], N, y=b["y"][0])

    base = {"op": op, "M": M, "K": K, "N": N, "members": G, "sets": sets}
    if args.eager:
        for i in range(args.eager):
            launch(i)
        torch.cuda.synchronize()
        print(json.dumps({**base, "eager_launches": args.eager, "status": pq.pq_device_status()}))
        return
    stream = torch.cuda.Stream()
    with torch.cuda.stream(stream):
        for i in range(sets):
            launch(i)
    stream.synchronize()
    n_launch = 16
    g = torch.cuda.CUDAGraph()
    with torch.cuda.graph(g, stream=stream):
        for i in range(n_launch):
            launch(i)
    times = []
    with torch.cuda.stream(stream):
        for _ in range(3):
            g.replay()
        for _ in range(20):
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record(stream)
            g.replay()
            e1.record(stream)
            times.append((e0, e1))
        stream.synchronize()
    us = sorted(e0.elapsed_time(e1) * 1e3 / n_launch for e0, e1 in times)
    med = us[len(us) // 2]
    out = {**base, "us_median": med, "us_min": us[0], "status": pq.pq_device_status()}
    if op in QUANT_OPS:
        out["GBps"] = ((5 if op == "swiglu_quantize" else 3) * M * K + 4 * M + (4 * K if op == "quantize_smooth" else 0)) / med / 1e3
    else:
        out["TOPS"] = 2 * M * G * N * K / med / 1e6
        wbytes = N * K + 4 * N if op.endswith("w8a8") else N * K // 2 + (K // 128) * N * 2
        out["GBps"] = (G * wbytes + M * K + 4 * M + 2 * M * G * N) / med / 1e3
    print(json.dumps(out))


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=200)
    ap.add_argument("--warmup", type=int, default=20)
    ap.add_argument("--impl", choices=["ours", "reference"], default="ours")
    ap.add_argument("--workload", default=DEFAULT_WORKLOAD, choices=sorted(synth.WORKLOADS))
    ap.add_argument("--M", type=int, default=None, help="token count (default: the workload's largest)")
    ap.add_argument("--no-graph", action="store_true", help="launch eagerly instead of replaying CUDA graphs")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-group", action="store_true",
                    help="one GEMM call per linear instead of grouped calls for linears that share their input")
    ap.add_argument("--no-fp16-context", action="store_true", help="skip the cuBLAS FP16 same-shape timing")
    ap.add_argument("--no-side-workloads", action="store_true", help="skip the `workloads` block (the other configurations)")
    ap.add_argument("--one-op", choices=ONE_OPS, default=None, help="run one operation on one shape instead of a workload")
    ap.add_argument("--shape", default="", help="--one-op: M,K[,N]")
    ap.add_argument("--members", type=int, default=1, help="--one-op gemm_*: this many linears of width N in one grouped call")
    ap.add_argument("--sets", type=int, default=0, help="--one-op: distinct buffer sets (0 = enough to exceed 2 x L2, max 16)")
    ap.add_argument("--eager", type=int, default=0, help="--one-op: run this many plain launches and exit (for profilers)")
    args = ap.parse_args()
    if args.one_op:
        return run_one_op(args)
    args.warmup = max(args.warmup, 3) if args.impl == "ours" else args.warmup
    wl = synth.WORKLOADS[args.workload]
    M = args.M if args.M is not None else max(wl.Ms)
    if args.impl == "reference":
        run_reference(args, wl, M)
    else:
        run_ours(args, wl, M)


if __name__ == "__main__":
    main()
