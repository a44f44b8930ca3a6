"""pq_gemm_w8a8_noalloc -- the W8A8 linear for callers that may not allocate device memory.

Who needs it: a plug-in whose host passes only input and output buffers, a serving loop or capture
region where cudaMalloc (which synchronizes the device) is forbidden, a program that fixed its
device-memory budget at start-up.  The call takes its split-K scratch from a fixed array inside the
library instead of a workspace somebody allocated, so it must give exactly what pq_gemm_w8a8 gives.

The array is shared by every call and keeps the previous call's contents, so each case runs the new
entry point twice in a row: a stale counter or partial sum left by the first call would show up in
the second.  This file sorts last on purpose; it must also pass when run alone.
"""
import numpy as np
import pytest
import torch

import paper_2512_23367_b200 as pq
from paper_2512_23367_b200 import synth

pytestmark = pytest.mark.gpu
DEV = "cuda:0"
REL, ABS = 2.0 ** -10, 1e-3      # the tolerance of the other W8A8 parity tests


def _inputs(M, K, N, seed):
    x = synth.activations(M, K, seed)
    w = synth.weights(N, K, seed + 1)
    q, s_tok = pq.pq_quantize_act(torch.from_numpy(x).to(DEV))
    wq, s_ch = pq.pq_pack_w8(torch.from_numpy(w).to(DEV))
    return q, s_tok, wq, s_ch


STATIC_SCRATCH_BYTES = (32 << 20) + (64 << 10)      # the array inside the library


# shapes on which the kernel really splits K (few tiles, long K), one that does not, and decode-shaped
# token counts (no scratch at all) whose padded output is beyond the array's limit
@pytest.mark.parametrize("M,K,N,split", [(512, 11008, 1024, True), (300, 11008, 520, True), (257, 8192, 264, True),
                                         (512, 2048, 1000, False), (96, 4096, 512, False),
                                         (1, 4096, 11008, False), (128, 4096, 11008, False)])
def test_matches_the_allocating_entry_point_on_two_calls_in_a_row(M, K, N, split):
    # the comparison is only worth something where the scratch array is really used: K must be split
    # (token counts up to 128 run on the schedule that reduces inside the SMs, whatever the plan would say)
    assert (M > 128 and pq.pq_plan_w8a8(M, N, K, 148, STATIC_SCRATCH_BYTES)[1] > 1) == split
    q, s_tok, wq, s_ch = _inputs(M, K, N, seed=900 + M)
    need = pq.pq_workspace_bytes(M, N, K)
    ws = pq.pq_workspace_init(torch.empty((need,), dtype=torch.uint8, device=DEV)) if need else None
    y_ref = pq.pq_gemm_w8a8(q, s_tok, wq, s_ch, N, workspace=ws)   # existing entry point (caller's workspace)
    pad = 1024
    for _ in range(2):
        buf = torch.full((pad + M * N + pad,), 7.0, dtype=torch.float16, device=DEV)
        y = buf[pad:pad + M * N].view(M, N)
        pq.pq_gemm_w8a8_noalloc(q, s_tok, wq, s_ch, N, y)     # through the C ABI; creates no tensor
        torch.cuda.synchronize()
        g, r = y.double(), y_ref.double()
        assert torch.isfinite(g).all()
        assert ((g - r).abs() <= REL * r.abs() + ABS).all()
        assert torch.equal(y, y_ref)                          # integer partial sums: in fact bit-identical
        assert (buf[:pad] == 7.0).all() and (buf[pad + M * N:] == 7.0).all()
    assert pq.pq_device_status() == 0


def test_sizes_beyond_the_fixed_array_are_refused_before_anything_runs():
    M, K, N = 4096, 256, 4096                                  # 16 Mi padded outputs > 2 Mi
    q = torch.zeros((M, K), dtype=torch.int8, device=DEV)
    s_tok = torch.ones((M,), dtype=torch.float32, device=DEV)
    wq = torch.zeros((N * K,), dtype=torch.uint8, device=DEV)
    s_ch = torch.ones((N,), dtype=torch.float32, device=DEV)
    y = torch.full((M, N), 3.0, dtype=torch.float16, device=DEV)
    with pytest.raises(pq.PQError) as err:
        pq.pq_gemm_w8a8_noalloc(q, s_tok, wq, s_ch, N, y)
    assert err.value.status == 7                               # PQ_ERR_LIMIT
    torch.cuda.synchronize()
    assert (y == 3.0).all()                                    # nothing was launched
    assert np.isclose(float(y[0, 0]), 3.0)
