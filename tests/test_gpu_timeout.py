"""The give-up path of the kernels: every wait on a barrier is bounded, and a wait that runs out makes the
kernel record PQ_ERR_TIMEOUT in the device status word, let the copies and MMAs it has in flight finish, and
return.  Nothing is broken here to provoke it: the poll bound itself is lowered (pq_set_wait_limit), to
"no polls at all" -- every role gives up at its first wait, so the status MUST be PQ_ERR_TIMEOUT -- and to a
few polls, where some wait in the middle of the kernel may or may not run out.  Afterwards the default bound
is restored and the same call must give the oracle-checked result again: the context, the barriers, tensor
memory and the scratch are all usable."""
import numpy as np
import pytest
import torch

import oracle
import paper_2512_23367_b200 as pq
from paper_2512_23367_b200 import synth

pytestmark = pytest.mark.gpu
DEV = "cuda:0"
PQ_ERR_TIMEOUT = 6
WAIT_NONE = 0xFFFFFFFF


def _case(kind):
    """-> (call() -> y, reinit(), check(y)) on one small shape per kernel; check compares a few token rows
    with the oracle."""
    M, K, N = {"w8a8_pair": (300, 1024, 520), "w8a8_pair_split_k": (512, 11008, 1024), "w8a8_noalloc": (512, 11008, 1024),
               "w8a8_small_m": (16, 2048, 1024), "w8a8_small_m_blocks": (200, 2048, 1024), "w4a8_pair": (300, 1024, 520), "w4a8_small_m": (16, 2048, 1024), "w4a8_small_m_128": (100, 2048, 1024), "w4a8_small_m_blocks": (200, 2048, 1024),
               "w8a8_rows": (3, 2048, 1024), "w4a8_rows": (2, 2048, 1024), "w4a8_linear_rows": (2, 2048, 1024)}[kind]
    x, w = synth.activations(M, K, 31), synth.weights(N, K, 32)
    q, s_tok = pq.pq_quantize_act(torch.from_numpy(x).to(DEV))
    y = torch.empty((M, N), dtype=torch.float16, device=DEV)
    rows = np.unique(np.concatenate([[0, M - 1], np.arange(0, M, 61)]))
    qo, so = oracle.quantize_act(x[rows])

    def check(y_gpu):
        if kind.startswith("w4a8"):
            _, ref = oracle.gemm_w4a8(qo, so, *oracle.pack_w4(w, 128), 128, want_acc=False)
        else:
            _, ref = oracle.gemm_w8a8(qo, so, *oracle.pack_w8(w), want_acc=False)
        g, ref = y_gpu.cpu().numpy()[rows].astype(np.float64), ref.astype(np.float64)
        assert np.all(np.abs(g - ref) <= 2.0 ** -10 * np.abs(ref) + 1e-3)

    if kind == "w4a8_linear_rows":     # the row kernel quantizing its own tokens
        wp, sg = pq.pq_pack_w4(torch.from_numpy(w).to(DEV))
        xd = torch.from_numpy(x).to(DEV)
        return (lambda: pq.pq_linear_w4a8(xd, wp, sg, N, y=y, q_tmp=q, s_tok_tmp=s_tok)), (lambda: None), check
    if kind.startswith("w4a8"):
        wp, sg = pq.pq_pack_w4(torch.from_numpy(w).to(DEV))
        return (lambda: pq.pq_gemm_w4a8(q, s_tok, wp, sg, N, y=y)), (lambda: None), check
    wq, s_ch = pq.pq_pack_w8(torch.from_numpy(w).to(DEV))
    if kind == "w8a8_noalloc":
        return (lambda: pq.pq_gemm_w8a8_noalloc(q, s_tok, wq, s_ch, N, y)), (lambda: None), check
    ws = None
    if kind == "w8a8_pair_split_k":
        need = pq.pq_workspace_bytes(M, N, K)
        assert pq.pq_plan_w8a8(M, N, K, 148, need)[1] > 1
        ws = torch.empty((need,), dtype=torch.uint8, device=DEV)
    return ((lambda: pq.pq_gemm_w8a8(q, s_tok, wq, s_ch, N, y=y, workspace=ws)),
            (lambda: ws is not None and pq.pq_workspace_init(ws)), check)


@pytest.mark.parametrize("kind", ["w8a8_pair", "w8a8_pair_split_k", "w8a8_noalloc", "w8a8_small_m", "w8a8_small_m_blocks", "w4a8_pair", "w4a8_small_m", "w4a8_small_m_128", "w4a8_small_m_blocks",
                                  "w8a8_rows", "w4a8_rows", "w4a8_linear_rows"])
def test_a_wait_that_runs_out_is_reported_and_leaves_everything_usable(kind):
    call, reinit, check = _case(kind)
    reinit()
    good = call().clone()
    assert pq.pq_device_status() == 0
    check(good)
    for limit in (WAIT_NONE, 1, 16, 256):
        pq.pq_set_wait_limit(limit)
        try:
            got = call().clone()
            status = pq.pq_device_status()        # synchronizes
        finally:
            pq.pq_set_wait_limit(0)
        if limit == WAIT_NONE:
            assert status == PQ_ERR_TIMEOUT
        else:
            assert status in (0, PQ_ERR_TIMEOUT)
            if status == 0:
                assert torch.equal(got, good)     # nothing ran out: the result is the normal one
        reinit()                                   # a caller's workspace is prepared again after a give-up
        assert torch.equal(call(), good)
        assert pq.pq_device_status() == 0
