"""The C-ABI library loads without a GPU and exports every symbol include/pq.h declares;
argument errors are reported before anything touches a device."""
import ctypes
import os
import re

import paper_2512_23367_b200 as pq
from paper_2512_23367_b200 import binding

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _declared():
    text = open(os.path.join(ROOT, "include", "pq.h")).read()
    return sorted(set(re.findall(r"PQ_API\s+[\w\s\*]+?\b(pq_\w+)\s*\(", text)))


def test_header_symbols_are_exported_and_bound():
    names = _declared()
    assert {"pq_quantize_act", "pq_pack_w8", "pq_pack_w4", "pq_gemm_w8a8", "pq_gemm_w4a8"} <= set(names)
    handle = ctypes.CDLL(pq.lib()._name)
    for n in names:
        assert hasattr(handle, n), n
    assert set(names) == set(binding.SIGNATURES), set(names) ^ set(binding.SIGNATURES)


def test_argument_errors_come_back_as_status_codes_without_a_device():
    L = pq.lib()
    PQ_ERR_NULL, PQ_ERR_SHAPE, PQ_ERR_ALIGN = 1, 2, 3
    assert L.pq_quantize_act(None, 4, 64, None, None, None) == PQ_ERR_NULL
    assert L.pq_quantize_act(16, 4, 60, 16, 16, None) == PQ_ERR_SHAPE      # K % 16
    assert L.pq_quantize_act(16, 0, 64, 16, 16, None) == PQ_ERR_SHAPE      # M < 1
    assert L.pq_quantize_act(8, 4, 64, 16, 16, None) == PQ_ERR_ALIGN
    assert L.pq_gemm_w8a8(16, 16, 16, 16, 4, 12, 64, 16, None, 0, None) == PQ_ERR_SHAPE   # N % 8
    assert L.pq_gemm_w8a8(16, 16, 16, 16, 4, 16, 131072, 16, None, 0, None) == PQ_ERR_SHAPE  # INT32 bound
    assert L.pq_gemm_w8a8(16, 16, 16, 16, 4, 16, 64, 16, 128, 1 << 20, None) == PQ_ERR_ALIGN   # workspace not 256-byte aligned
    assert L.pq_workspace_init(None, 1 << 20, None) == PQ_ERR_NULL
    assert L.pq_workspace_init(128, 1 << 20, None) == PQ_ERR_ALIGN
    assert L.pq_workspace_init(256, 1024, None) == PQ_ERR_SHAPE
    assert L.pq_gemm_w4a8(16, 16, 16, 16, 64, 4, 16, 256, 16, None) == PQ_ERR_SHAPE   # group != 128
    assert L.pq_gemm_w4a8(16, 16, 16, 16, 128, 4, 16, 192, 16, None) == PQ_ERR_SHAPE  # K % 128
    assert L.pq_pack_w4(16, 16, 256, 128, None, 16, None) == PQ_ERR_NULL
    # x, wq, s_ch, M, N, K, y, q_tmp, s_tok_tmp, workspace, bytes, stream
    assert L.pq_linear_w8a8(16, 16, 16, 4, 16, 64, 16, None, 16, None, 0, None) == PQ_ERR_NULL        # no q_tmp
    assert L.pq_linear_w8a8(16, 16, 16, 4, 12, 64, 16, 16, 16, None, 0, None) == PQ_ERR_SHAPE         # N % 8
    assert L.pq_linear_w8a8(8, 16, 16, 4, 16, 64, 16, 16, 16, None, 0, None) == PQ_ERR_ALIGN
    # x, wp, s_grp, group, M, N, K, y, q_tmp, s_tok_tmp, stream
    assert L.pq_linear_w4a8(16, 16, 16, 64, 4, 16, 256, 16, 16, 16, None) == PQ_ERR_SHAPE             # group != 128
    assert L.pq_linear_w4a8(16, 16, 16, 128, 4, 16, 256, 16, 16, None, None) == PQ_ERR_NULL           # no s_tok_tmp
    import ctypes
    ptrs = (ctypes.c_void_p * 2)(16, 16)
    holes = (ctypes.c_void_p * 2)(16, None)
    cols = (ctypes.c_int64 * 2)(16, 16)
    odd = (ctypes.c_int64 * 2)(16, 12)
    assert L.pq_gemm_w8a8_group(16, 16, 2, None, ptrs, cols, ptrs, 4, 64, None, 0, None) == PQ_ERR_NULL
    assert L.pq_gemm_w8a8_group(16, 16, 2, holes, ptrs, cols, ptrs, 4, 64, None, 0, None) == PQ_ERR_NULL   # a member's pointer
    assert L.pq_gemm_w8a8_group(16, 16, 0, ptrs, ptrs, cols, ptrs, 4, 64, None, 0, None) == PQ_ERR_SHAPE    # empty group
    assert L.pq_gemm_w8a8_group(16, 16, 5, ptrs, ptrs, cols, ptrs, 4, 64, None, 0, None) == PQ_ERR_SHAPE    # > PQ_MAX_GROUP
    assert L.pq_gemm_w8a8_group(16, 16, 2, ptrs, ptrs, odd, ptrs, 4, 64, None, 0, None) == PQ_ERR_SHAPE     # N[1] % 8
    assert L.pq_gemm_w4a8_group(16, 16, 2, ptrs, holes, 128, cols, ptrs, 4, 128, None) == PQ_ERR_NULL
    assert L.pq_gemm_w4a8_group(16, 16, 2, ptrs, ptrs, 64, cols, ptrs, 4, 128, None) == PQ_ERR_SHAPE    # group != 128
    assert L.pq_gemm_w4a8_group(16, 16, 5, ptrs, ptrs, 128, cols, ptrs, 4, 128, None) == PQ_ERR_SHAPE   # > PQ_MAX_GROUP
    assert L.pq_quantize_act_smooth(16, None, 4, 64, 16, 16, None) == PQ_ERR_NULL
    assert L.pq_quantize_act_smooth(16, 8, 4, 64, 16, 16, None) == PQ_ERR_ALIGN     # factor vector
    assert L.pq_pack_w8_smooth(16, None, 16, 64, 16, 16, None) == PQ_ERR_NULL
    assert L.pq_pack_w4_smooth(16, 16, 16, 256, 64, 16, 16, None) == PQ_ERR_SHAPE   # group != 128
    assert L.pq_col_absmax(16, 0, 64, 16, None) == PQ_ERR_SHAPE
    assert L.pq_smooth_scales(16, 16, 0, 16, 16, None) == PQ_ERR_SHAPE
    assert L.pq_smooth_scales_alpha(16, 16, 64, 5, 16, 16, None) == PQ_ERR_SHAPE      # alpha beyond 4/4
    assert L.pq_quantize_act_hadamard(16, 4, 16400, 16, 16, None) == PQ_ERR_SHAPE   # row does not fit the registers
    assert L.pq_pack_w4_hadamard(16, 16, 192, 128, 16, 16, None) == PQ_ERR_SHAPE     # K % 128
    assert [L.pq_hadamard_block(K) for K in (16, 48, 208, 2048, 4096, 11008, 20)] == [16, 16, 16, 2048, 4096, 256, 0]
    assert L.pq_quantize_act_static(16, None, 4, 64, 16, 16, None) == PQ_ERR_NULL
    assert L.pq_quantize_act_static(16, 16, 4, 60, 16, 16, None) == PQ_ERR_SHAPE
    assert L.pq_packed_w8_bytes(8, 256) == 2048 and L.pq_packed_w4_bytes(8, 256) == 1024
    assert L.pq_status_str(0) == b"ok" and b"wait" in L.pq_status_str(6)


def test_schedule_choice_for_the_benchmark_shapes():
    """Host logic of the W8A8 pair GEMM: tile width and K parts, on a 148-SM device."""
    ws = 64 << 20
    # many tiles: wide tiles, no split, with or without scratch
    assert pq.pq_plan_w8a8(4096, 11008, 4096, 148, ws) == (256, 1)
    assert pq.pq_plan_w8a8(2048, 2048, 2048, 148, ws) == (256, 1)
    assert pq.pq_plan_w8a8(2048, 2048, 6144, 148, ws) == (256, 1)
    # 32 tiles and 86 K blocks: two K parts fill the machine -- but only with room for the partials
    assert pq.pq_plan_w8a8(512, 4096, 11008, 148, ws) == (256, 2)
    assert pq.pq_plan_w8a8(512, 4096, 11008, 148, 0) == (256, 1)
    assert pq.pq_plan_w8a8(512, 4096, 11008, 148, 8 << 20)[1] == 1      # 16 MiB needed
    # short K: the scratch round trip costs more than it saves
    assert pq.pq_plan_w8a8(512, 4096, 4096, 148, ws) == (256, 1)
    # a single narrow tile column
    assert pq.pq_plan_w8a8(300, 128, 2048, 148, ws)[0] == 128
    # a few tiles with a very long K: up to four parts
    assert pq.pq_plan_w8a8(257, 264, 8192, 148, ws)[1] == 4


def test_workspace_size_query_agrees_with_the_planner():
    """pq_workspace_bytes = header + partial sums of the schedule chosen with unlimited room; with that
    much the planner picks that schedule, with one byte less it does not split as far."""
    for M, N, K in [(512, 4096, 11008), (257, 264, 8192), (300, 520, 11008), (512, 1024, 11008)]:
        need = pq.pq_workspace_bytes(M, N, K)
        bn, parts = pq.pq_plan_w8a8(M, N, K, 148, 1 << 40)
        assert parts > 1
        tiles = -(-M // 256) * -(-N // bn)
        assert need == 65536 + tiles * 2 * parts * 128 * bn * 4
        assert pq.pq_plan_w8a8(M, N, K, 148, need) == (bn, parts)
        assert pq.pq_plan_w8a8(M, N, K, 148, need - 1) != (bn, parts)
    # shapes that never split need nothing: many tiles, short K, decode-shaped
    for M, N, K in [(4096, 11008, 4096), (2048, 2048, 2048), (512, 4096, 4096), (64, 4096, 11008), (128, 4096, 11008)]:
        assert pq.pq_workspace_bytes(M, N, K) == 0
    # a group is sized as one launch over all members' tiles
    assert pq.pq_workspace_bytes(512, [512, 512], 11008) > pq.pq_workspace_bytes(512, [512], 11008) > 0
    assert pq.pq_workspace_bytes(512, [12], 11008) == 0            # invalid width


def test_binding_measures_every_operand_before_the_call():
    """A wrong N or a short buffer must become a Python exception, never a launch: the C calls trust the
    sizes they are given.  (Sizes are checked before devices, so CPU tensors are enough to show it.)"""
    import pytest
    import torch
    M, K, N = 4, 64, 16
    q, st = torch.zeros((M, K), dtype=torch.int8), torch.ones(M)
    wq, sc = torch.zeros(N * K, dtype=torch.uint8), torch.ones(N)
    wp, sg = torch.zeros(N * K // 2, dtype=torch.uint8), torch.ones((K // 128 or 1) * N, dtype=torch.float16)
    y = torch.zeros((M, N), dtype=torch.float16)
    with pytest.raises(ValueError, match="wq: expected 2048 elements"):
        pq.pq_gemm_w8a8(q, st, wq, sc, 2 * N, y)
    with pytest.raises(ValueError, match="s_ch: expected"):
        pq.pq_gemm_w8a8(q, st, wq, sc[:-1], N, y)
    with pytest.raises(ValueError, match="s_tok: expected"):
        pq.pq_gemm_w8a8(q, st[:-1], wq, sc, N, y)
    with pytest.raises(ValueError, match="y: expected"):
        pq.pq_gemm_w8a8(q, st, wq, sc, N, y[:-1])
    with pytest.raises(ValueError, match="y: expected"):
        pq.pq_gemm_w8a8_noalloc(q, st, wq, sc, N, y[:-1])
    with pytest.raises(ValueError, match="wq: expected"):
        pq.pq_gemm_w8a8_noalloc(q, st, wq[:-1], sc, N, y)
    q2, st2 = torch.zeros((M, 128), dtype=torch.int8), torch.ones(M)
    wp, sg = torch.zeros(N * 64, dtype=torch.uint8), torch.ones(N, dtype=torch.float16)
    with pytest.raises(ValueError, match="wp: expected"):
        pq.pq_gemm_w4a8(q2, st2, wp[:-1], sg, N)
    with pytest.raises(ValueError, match="s_grp: expected"):
        pq.pq_gemm_w4a8(q2, st2, wp, sg[:-1], N)
    with pytest.raises(ValueError, match="wq: expected"):
        pq.pq_acc_w8a8(q, wq[:-1], N)
    with pytest.raises(ValueError, match="wp: expected"):
        pq.pq_acc_w4a8(q2, wp[:-1], N)
    with pytest.raises(ValueError, match=r"members\[1\] weights: expected"):
        pq.pq_gemm_w8a8_group(q, st, [(wq, sc, N), (wq[:-1], sc, N)])
    with pytest.raises(ValueError, match=r"ys\[0\]: expected"):
        pq.pq_gemm_w8a8_group(q, st, [(wq, sc, N)], [y[:-1]])
    with pytest.raises(ValueError, match=r"members\[0\] scales: expected"):
        pq.pq_gemm_w4a8_group(q2, st2, [(wp, sg[:-1], N)])
    with pytest.raises(ValueError, match="q: expected"):
        pq.pq_quantize_act(torch.zeros((M, K), dtype=torch.float16), q=torch.zeros((M, K - 1), dtype=torch.int8))
    x, x2 = torch.zeros((M, K), dtype=torch.float16), torch.zeros((M, 128), dtype=torch.float16)
    with pytest.raises(ValueError, match="wq: expected"):
        pq.pq_linear_w8a8(x, wq[:-1], sc, N)
    with pytest.raises(ValueError, match="q_tmp: expected"):
        pq.pq_linear_w8a8(x, wq, sc, N, q_tmp=torch.zeros((M, K - 1), dtype=torch.int8))
    with pytest.raises(ValueError, match="y: expected"):
        pq.pq_linear_w8a8(x, wq, sc, N, y=y[:-1])
    with pytest.raises(ValueError, match="s_grp: expected"):
        pq.pq_linear_w4a8(x2, wp, sg[:-1], N)
    with pytest.raises(ValueError, match="s_tok_tmp: expected"):
        pq.pq_linear_w4a8(x2, wp, sg, N, s_tok_tmp=torch.ones(M - 1))
    with pytest.raises(TypeError):
        pq.pq_gemm_w8a8(q, st, wq.to(torch.int8), sc, N, y)
    with pytest.raises(ValueError, match="CUDA"):          # right sizes, wrong memory: there is no CPU path
        pq.pq_gemm_w8a8(q, st, wq, sc, N, y)
