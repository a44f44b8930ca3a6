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
    assert L.pq_gemm_w8a8(16, 16, 16, 16, 4, 12, 64, 16, None) == PQ_ERR_SHAPE   # N % 8
    assert L.pq_gemm_w8a8(16, 16, 16, 16, 4, 16, 131072, 16, None) == PQ_ERR_SHAPE  # INT32 bound
    assert L.pq_gemm_w4a8(16, 16, 16, 16, 64, 4, 16, 256, 16, None) == PQ_ERR_SHAPE   # group != 128
    assert L.pq_gemm_w4a8(16, 16, 16, 16, 128, 4, 16, 192, 16, None) == PQ_ERR_SHAPE  # K % 128
    assert L.pq_pack_w4(16, 16, 256, 128, None, 16, None) == PQ_ERR_NULL
    import ctypes
    ptrs = (ctypes.c_void_p * 2)(16, 16)
    holes = (ctypes.c_void_p * 2)(16, None)
    cols = (ctypes.c_int64 * 2)(16, 16)
    odd = (ctypes.c_int64 * 2)(16, 12)
    assert L.pq_gemm_w8a8_group(16, 16, 2, None, ptrs, cols, ptrs, 4, 64, None) == PQ_ERR_NULL
    assert L.pq_gemm_w8a8_group(16, 16, 2, holes, ptrs, cols, ptrs, 4, 64, None) == PQ_ERR_NULL   # a member's pointer
    assert L.pq_gemm_w8a8_group(16, 16, 0, ptrs, ptrs, cols, ptrs, 4, 64, None) == PQ_ERR_SHAPE    # empty group
    assert L.pq_gemm_w8a8_group(16, 16, 5, ptrs, ptrs, cols, ptrs, 4, 64, None) == PQ_ERR_SHAPE    # > PQ_MAX_GROUP
    assert L.pq_gemm_w8a8_group(16, 16, 2, ptrs, ptrs, odd, ptrs, 4, 64, None) == PQ_ERR_SHAPE     # N[1] % 8
    assert L.pq_gemm_w4a8_group(16, 16, 2, ptrs, holes, 128, cols, ptrs, 4, 128, None) == PQ_ERR_NULL
    assert L.pq_gemm_w4a8_group(16, 16, 2, ptrs, ptrs, 64, cols, ptrs, 4, 128, None) == PQ_ERR_SHAPE    # group != 128
    assert L.pq_gemm_w4a8_group(16, 16, 5, ptrs, ptrs, 128, cols, ptrs, 4, 128, None) == PQ_ERR_SHAPE   # > PQ_MAX_GROUP
    assert L.pq_quantize_act_smooth(16, None, 4, 64, 16, 16, None) == PQ_ERR_NULL
    assert L.pq_quantize_act_smooth(16, 8, 4, 64, 16, 16, None) == PQ_ERR_ALIGN     # factor vector
    assert L.pq_pack_w8_smooth(16, None, 16, 64, 16, 16, None) == PQ_ERR_NULL
    assert L.pq_pack_w4_smooth(16, 16, 16, 256, 64, 16, 16, None) == PQ_ERR_SHAPE   # group != 128
    assert L.pq_col_absmax(16, 0, 64, 16, None) == PQ_ERR_SHAPE
    assert L.pq_smooth_scales(16, 16, 0, 16, 16, None) == PQ_ERR_SHAPE
    assert L.pq_quantize_act_hadamard(16, 4, 16400, 16, 16, None) == PQ_ERR_SHAPE   # row does not fit the registers
    assert L.pq_pack_w4_hadamard(16, 16, 192, 128, 16, 16, None) == PQ_ERR_SHAPE     # K % 128
    assert [L.pq_hadamard_block(K) for K in (16, 48, 208, 2048, 4096, 11008, 20)] == [16, 16, 16, 256, 256, 256, 0]
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
