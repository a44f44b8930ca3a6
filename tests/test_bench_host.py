"""Host-side logic of bench.py: step accounting and the multi-rank aggregation (gloo, 2 ranks)."""
import os
import subprocess
import sys
import textwrap

import bench
from paper_2512_23367_b200 import synth

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def test_layer_plan_shares_inputs_and_counts_ops():
    wl = synth.WORKLOADS["c2_w8a8_1b_prefill"]
    plan = bench.layer_plan(wl)
    assert [(K, idx) for K, idx in plan] == [(2048, [0, 1, 2]), (2048, [3]), (2048, [4, 5]), (6144, [6])]
    M = 2048
    assert bench.step_ops(wl, M) == 2 * M * (4 * 2048 * 2048 + 3 * 2048 * 6144)
    b = bench.step_bytes(wl, M)
    assert b["quantize"] == 3 * M * (3 * 2048 + 6144) + 4 * 4 * M
    wl5 = synth.WORKLOADS["c5_w4a8_7b_decode"]
    assert [idx for _, idx in bench.layer_plan(wl5)] == [[0], [1], [2]]
    assert bench.weight_bytes(wl5) == sum(l.N * l.K // 2 + (l.K // 128) * l.N * 2 for l in wl5.linears)
    n = bench.layers_for_rotation(wl, M)
    per = bench.weight_bytes(wl) + sum(2 * M * K for K, _ in plan)
    assert n * per > 2 * bench.L2_BYTES


def test_aggregate_over_two_gloo_ranks(tmp_path):
    script = textwrap.dedent("""
        import os, sys
        sys.path.insert(0, %r)
        import torch.distributed as dist
        import bench
        dist.init_process_group("gloo")
        r = dist.get_rank()
        ms, units = bench.aggregate_over_ranks(10.0 + 5.0 * r, 100.0 * (r + 1), dist.get_world_size())
        assert ms == 15.0 and units == 300.0, (ms, units)
        dist.destroy_process_group()
        print("rank", r, "ok")
    """ % ROOT)
    path = tmp_path / "ranks.py"
    path.write_text(script)
    env = dict(os.environ, MASTER_ADDR="127.0.0.1")
    out = subprocess.run([sys.executable, "-m", "torch.distributed.run", "--nnodes=1", "--nproc-per-node=2",
                          "--master-addr", "127.0.0.1", "--master-port", "29533", str(path)],
                         capture_output=True, text=True, env=env, timeout=240)
    assert out.returncode == 0, out.stdout + out.stderr
    assert out.stdout.count("ok") == 2
