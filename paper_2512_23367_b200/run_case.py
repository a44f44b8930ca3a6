"""Runs ONE operation of the library on one shape, a few times, and prints its device time.

    python -m paper_2512_23367_b200.run_case --op gemm_w8a8 --M 4096 --K 4096 --N 4096

Meant for profilers (one kernel, few launches, bounded memory) and for per-shape timing.  Timing
replays a CUDA graph of `--launches` back-to-back launches that rotate over distinct buffer sets
(so that operands are not L2-resident) and divides the event time by the launch count.
"""
from __future__ import annotations

import argparse
import json

import torch

from . import binding as pq

QUANT_OPS = ("quantize", "quantize_smooth", "quantize_hadamard", "quantize_static")
OPS = QUANT_OPS + ("gemm_w8a8", "gemm_w4a8")


def main(argv=None):
    ap = argparse.ArgumentParser()
    ap.add_argument("--op", choices=OPS, required=True)
    ap.add_argument("--M", type=int, required=True)
    ap.add_argument("--K", type=int, required=True)
    ap.add_argument("--N", type=int, default=0)
    ap.add_argument("--group", type=int, default=1,
                    help="GEMM ops: this many linears of width N over the same tokens in one grouped call")
    ap.add_argument("--sets", type=int, default=0, help="distinct buffer sets (0 = enough to exceed 2 x L2, max 16)")
    ap.add_argument("--launches", type=int, default=16, help="launches per graph replay")
    ap.add_argument("--replays", type=int, default=20)
    ap.add_argument("--eager", type=int, default=0, help="run this many plain launches and exit (for profilers)")
    a = ap.parse_args(argv)
    dev = torch.device("cuda", 0)
    torch.manual_seed(0)
    M, K, N, G = a.M, a.K, a.N, max(a.group, 1)
    per_set = 2 * M * K + M * K + (G * N * K if a.op not in QUANT_OPS else 0)
    sets = a.sets or max(2, min(16, (2 * 126 * 2 ** 20) // max(per_set, 1) + 1))

    bufs = []
    for _ in range(sets):
        x = torch.randn((M, K), device=dev, dtype=torch.float16)
        x[:, :: max(K // 41, 1)] *= 50
        q, s_tok = pq.pq_quantize_act(x)
        entry = {"x": x, "q": q, "s_tok": s_tok,
                 "s_inv": torch.rand((K,), device=dev, dtype=torch.float32) + 0.5,
                 "scale": torch.full((1,), 0.05, device=dev, dtype=torch.float32)}
        if a.op not in QUANT_OPS:
            entry["w"], entry["y"] = [], []
            for _ in range(G):
                w = (torch.randn((N, K), device=dev, dtype=torch.float32) * 0.02).half()
                entry["w"].append(pq.pq_pack_w8(w) if a.op == "gemm_w8a8" else pq.pq_pack_w4(w))
                entry["y"].append(torch.empty((M, N), device=dev, dtype=torch.float16))
                del w
        bufs.append(entry)

    def launch(i):
        b = bufs[i % sets]
        if a.op == "quantize":
            pq.pq_quantize_act(b["x"], b["q"], b["s_tok"])
        elif a.op == "quantize_smooth":
            pq.pq_quantize_act_smooth(b["x"], b["s_inv"], b["q"], b["s_tok"])
        elif a.op == "quantize_hadamard":
            pq.pq_quantize_act_hadamard(b["x"], b["q"], b["s_tok"])
        elif a.op == "quantize_static":
            pq.pq_quantize_act_static(b["x"], b["scale"], b["q"], b["s_tok"])
        elif G > 1:
            call = pq.pq_gemm_w8a8_group if a.op == "gemm_w8a8" else pq.pq_gemm_w4a8_group
            call(b["q"], b["s_tok"], [(w[0], w[1], N) for w in b["w"]], b["y"])
        elif a.op == "gemm_w8a8":
            pq.pq_gemm_w8a8(b["q"], b["s_tok"], b["w"][0][0], b["w"][0][1], N, y=b["y"][0])
        else:
            pq.pq_gemm_w4a8(b["q"], b["s_tok"], b["w"][0][0], b["w"][0][1], N, y=b["y"][0])

    if a.eager:
        for i in range(a.eager):
            launch(i)
        torch.cuda.synchronize()
        print(json.dumps({"op": a.op, "M": M, "K": K, "N": N, "group": G, "eager_launches": a.eager,
                          "status": pq.pq_device_status()}))
        return

    stream = torch.cuda.Stream()
    with torch.cuda.stream(stream):
        for i in range(sets):
            launch(i)
    stream.synchronize()
    g = torch.cuda.CUDAGraph()
    with torch.cuda.graph(g, stream=stream):
        for i in range(a.launches):
            launch(i)
    times = []
    with torch.cuda.stream(stream):
        for _ in range(3):
            g.replay()
        for _ in range(a.replays):
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record(stream)
            g.replay()
            e1.record(stream)
            times.append((e0, e1))
        stream.synchronize()
    us = sorted(e0.elapsed_time(e1) * 1e3 / a.launches for e0, e1 in times)
    med, best = us[len(us) // 2], us[0]
    out = {"op": a.op, "M": M, "K": K, "N": N, "group": G, "sets": sets, "us_median": med, "us_min": best,
           "status": pq.pq_device_status()}
    if a.op in QUANT_OPS:
        out["GBps"] = (3 * M * K + 4 * M + (4 * K if a.op == "quantize_smooth" else 0)) / med / 1e3
    else:
        out["TOPS"] = 2 * M * G * N * K / med / 1e6
        wbytes = N * K if a.op == "gemm_w8a8" else N * K // 2 + (K // 128) * N * 2
        out["GBps"] = (G * wbytes + M * K + 2 * M * G * N) / med / 1e3
    print(json.dumps(out))


if __name__ == "__main__":
    main()
