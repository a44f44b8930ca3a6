"""pq_gemm_w8a8_group / pq_gemm_w4a8_group: several linears over the same quantized tokens in one call.

The contract is "exactly what one pq_gemm_w8a8 call per member gives", so every case checks bit
equality with those calls, and parity with the CPU oracle (INT32 accumulators are exact, the FP16
result within the tolerance of the other W8A8 tests) independently of them.
"""
import numpy as np
import pytest
import torch

import oracle
import paper_2512_23367_b200 as pq
from paper_2512_23367_b200 import synth

pytestmark = pytest.mark.gpu
DEV = "cuda:0"
REL, ABS = 2.0 ** -10, 1e-3


def _members(K, Ns, seed):
    ws = [synth.weights(N, K, seed + 1 + i) for i, N in enumerate(Ns)]
    packed = [pq.pq_pack_w8(torch.from_numpy(w).to(DEV)) for w in ws]
    return ws, [(wq, s_ch, N) for (wq, s_ch), N in zip(packed, Ns)]


# q/k/v-like (equal widths), gate/up-like, ragged widths that end inside a tile, one member wider
# than the others, four members, M with a ragged last row block, K long enough to split
@pytest.mark.parametrize("M,K,Ns", [
    (512, 512, (512, 512, 512)),
    (300, 256, (520, 264)),
    (257, 384, (1000, 136, 8)),
    (2048, 512, (2048, 2048, 2048)),
    (600, 1024, (256, 768, 264, 128)),
    (512, 8192, (264, 520)),
    (129, 128, (16, 24)),
])
def test_group_equals_one_call_per_member_and_the_oracle(M, K, Ns):
    x = synth.activations(M, K, 4000 + M)
    ws, members = _members(K, Ns, 4100 + M)
    q, s_tok = pq.pq_quantize_act(torch.from_numpy(x).to(DEV))
    pad = 512
    bufs = [torch.full((pad + M * N + pad,), 5.0, dtype=torch.float16, device=DEV) for N in Ns]
    ys = [b[pad:pad + M * N].view(M, N) for b, N in zip(bufs, Ns)]
    need = pq.pq_workspace_bytes(M, Ns, K)
    scratch = pq.pq_workspace_init(torch.empty((need,), dtype=torch.uint8, device=DEV)) if need else None
    out = pq.pq_gemm_w8a8_group(q, s_tok, members, ys, workspace=scratch)
    torch.cuda.synchronize()
    assert pq.pq_device_status() == 0
    qo, so = oracle.quantize_act(x)
    assert np.array_equal(q.cpu().numpy(), qo)
    for (wq, s_ch, N), w, y, b in zip(members, ws, out, bufs):
        single = pq.pq_gemm_w8a8(q, s_tok, wq, s_ch, N)
        assert torch.equal(y, single)
        wqo, sco = oracle.pack_w8(w)
        _, ref = oracle.gemm_w8a8(qo, so, wqo, sco, want_acc=False)
        g, ref = y.cpu().numpy().astype(np.float64), ref.astype(np.float64)
        assert np.all(np.abs(g - ref) <= REL * np.abs(ref) + ABS)
        assert (b[:pad] == 5.0).all() and (b[pad + M * N:] == 5.0).all()   # nothing outside the member's output


@pytest.mark.parametrize("M,K,Ns", [(1, 512, (256, 520)), (16, 512, (256, 520)), (64, 512, (256, 520)),
                                    (100, 512, (256, 520)), (3, 4224, (2376, 136, 8)), (33, 1024, (128, 128, 128, 264)),
                                    (128, 2048, (1000, 520)), (7, 4096, (4096, 4096, 4096))])
def test_small_token_counts_group_on_the_weight_streaming_kernel(M, K, Ns):
    x = synth.activations(M, K, 4300 + M)
    _, members = _members(K, Ns, 4400 + M)
    q, s_tok = pq.pq_quantize_act(torch.from_numpy(x).to(DEV))
    out = pq.pq_gemm_w8a8_group(q, s_tok, members)
    for (wq, s_ch, N), y in zip(members, out):
        assert torch.equal(y, pq.pq_gemm_w8a8(q, s_tok, wq, s_ch, N))


def test_two_group_calls_in_a_row_leave_the_split_k_scratch_clean():
    M, K, Ns = 512, 11008, (512, 512)
    x = synth.activations(M, K, 4500)
    _, members = _members(K, Ns, 4501)
    q, s_tok = pq.pq_quantize_act(torch.from_numpy(x).to(DEV))
    need = pq.pq_workspace_bytes(M, Ns, K)
    assert need > 0                                                     # this group splits K
    scratch = pq.pq_workspace_init(torch.empty((need,), dtype=torch.uint8, device=DEV))
    first = [y.clone() for y in pq.pq_gemm_w8a8_group(q, s_tok, members, workspace=scratch)]
    second = pq.pq_gemm_w8a8_group(q, s_tok, members, workspace=scratch)
    for a, b, (wq, s_ch, N) in zip(first, second, members):
        assert torch.equal(a, b)
        assert torch.equal(a, pq.pq_gemm_w8a8(q, s_tok, wq, s_ch, N))
    assert pq.pq_device_status() == 0


# ---------------------------------------------------------------------------- W4A8

def _members_w4(K, Ns, seed):
    ws = [synth.weights(N, K, seed + 1 + i) for i, N in enumerate(Ns)]
    packed = [pq.pq_pack_w4(torch.from_numpy(w).to(DEV)) for w in ws]
    return ws, [(wp, sg, N) for (wp, sg), N in zip(packed, Ns)]


@pytest.mark.parametrize("M,K,Ns", [
    (512, 512, (512, 512, 512)),
    (300, 256, (520, 264)),
    (257, 384, (1000, 136, 8)),
    (2048, 512, (2048, 2048, 2048)),
    (600, 1024, (256, 768, 264, 128)),
    (129, 128, (16, 24)),
])
def test_w4a8_group_equals_one_call_per_member_and_the_oracle(M, K, Ns):
    x = synth.activations(M, K, 5000 + M)
    ws, members = _members_w4(K, Ns, 5100 + M)
    q, s_tok = pq.pq_quantize_act(torch.from_numpy(x).to(DEV))
    pad = 512
    bufs = [torch.full((pad + M * N + pad,), 5.0, dtype=torch.float16, device=DEV) for N in Ns]
    ys = [b[pad:pad + M * N].view(M, N) for b, N in zip(bufs, Ns)]
    out = pq.pq_gemm_w4a8_group(q, s_tok, members, ys)
    torch.cuda.synchronize()
    assert pq.pq_device_status() == 0
    qo, so = oracle.quantize_act(x)
    for (wp, sg, N), w, y, b in zip(members, ws, out, bufs):
        assert torch.equal(y, pq.pq_gemm_w4a8(q, s_tok, wp, sg, N))
        codes, sgo = oracle.pack_w4(w)
        _, ref = oracle.gemm_w4a8(qo, so, codes, sgo, want_acc=False)
        g, ref = y.cpu().numpy().astype(np.float64), ref.astype(np.float64)
        assert np.all(np.abs(g - ref) <= REL * np.abs(ref) + ABS)
        assert (b[:pad] == 5.0).all() and (b[pad + M * N:] == 5.0).all()


@pytest.mark.parametrize("M,K,Ns", [(1, 512, (256, 520)), (16, 512, (256, 520)), (64, 512, (256, 520)),
                                    (3, 4224, (2376, 136, 8)), (33, 1024, (128, 128, 128, 264)),
                                    (7, 4096, (4096, 4096, 4096)), (65, 128, (16, 24)), (100, 1024, (1408, 520)),
                                    (128, 4096, (4096, 4096, 4096)), (200, 1024, (1408, 520)), (256, 4096, (4096, 4096))])
def test_w4a8_small_token_counts_group_on_the_weight_streaming_kernel(M, K, Ns):
    """Decode-shaped W4A8 sums its K parts in FP32 in a fixed order, but the number of parts depends on
    how many tiles the launch holds: the grouped result may differ from the per-member call in the last
    FP32 bit, so it is held to the oracle tolerance (and to the per-member result within the same)."""
    x = synth.activations(M, K, 5300 + M)
    ws, members = _members_w4(K, Ns, 5400 + M)
    q, s_tok = pq.pq_quantize_act(torch.from_numpy(x).to(DEV))
    out = pq.pq_gemm_w4a8_group(q, s_tok, members)
    torch.cuda.synchronize()
    assert pq.pq_device_status() == 0
    qo, so = oracle.quantize_act(x)
    for (wp, sg, N), w, y in zip(members, ws, out):
        _, ref = oracle.gemm_w4a8(qo, so, *oracle.pack_w4(w, 128), 128, want_acc=False)
        g, ref = y.cpu().numpy().astype(np.float64), ref.astype(np.float64)
        assert np.all(np.abs(g - ref) <= REL * np.abs(ref) + ABS)
        single = pq.pq_gemm_w4a8(q, s_tok, wp, sg, N).cpu().numpy().astype(np.float64)
        assert np.all(np.abs(g - single) <= REL * np.abs(single) + ABS)


# ---------------------------------------------------------------------------- the benchmark's grouped launches

@pytest.mark.parametrize("bits,M,K,Ns", [
    (8, 2048, 2048, (2048, 2048, 2048)),      # 1B-class q/k/v
    (8, 2048, 2048, (6144, 6144)),            # 1B-class gate/up
    (8, 4096, 4096, (4096, 4096, 4096)),      # 7B-class q/k/v
    (8, 512, 4096, (11008, 11008)),           # 7B-class gate/up at M = 512
    (4, 2048, 4096, (4096, 4096, 4096)),      # W4A8 q/k/v
    (4, 2048, 4096, (11008, 11008)),          # W4A8 gate/up
])
def test_benchmark_groups_at_full_size_touch_every_tile(bits, M, K, Ns):
    """The grouped launches exactly as bench.py issues them.  The oracle checks a token row out of every
    block of 128 x all channels of every member, and all token rows x a channel out of every block of 64
    of every member: every output tile of the launch is compared."""
    rng = np.random.default_rng(4600 + M + len(Ns))
    starts = np.arange(0, M, 128)
    rows = np.unique(np.concatenate([[0, 127, 128, 255, 256, M - 1], np.minimum(starts + rng.integers(0, 128, len(starts)), M - 1)]))
    x = synth.activations(M, K, 4700 + M)
    ws = [synth.weights(N, K, 4800 + i) for i, N in enumerate(Ns)]
    q, s_tok = pq.pq_quantize_act(torch.from_numpy(x).to(DEV))
    qo, so = oracle.quantize_act(x)
    assert np.array_equal(q.cpu().numpy(), qo)
    if bits == 8:
        members = [(*pq.pq_pack_w8(torch.from_numpy(w).to(DEV)), N) for w, N in zip(ws, Ns)]
        need = pq.pq_workspace_bytes(M, Ns, K)
        scratch = pq.pq_workspace_init(torch.empty((need,), dtype=torch.uint8, device=DEV)) if need else None
        out = pq.pq_gemm_w8a8_group(q, s_tok, members, workspace=scratch)
    else:
        members = [(*pq.pq_pack_w4(torch.from_numpy(w).to(DEV)), N) for w, N in zip(ws, Ns)]
        out = pq.pq_gemm_w4a8_group(q, s_tok, members)
    torch.cuda.synchronize()
    assert pq.pq_device_status() == 0

    def close(g, ref):
        g, ref = g.astype(np.float64), ref.astype(np.float64)
        return np.isfinite(g).all() and np.all(np.abs(g - ref) <= REL * np.abs(ref) + ABS)

    for w, y, N in zip(ws, out, Ns):
        cstarts = np.arange(0, N, 64)
        cols = np.unique(np.concatenate([[0, N - 1], np.minimum(cstarts + rng.integers(0, 64, len(cstarts)), N - 1)]))
        yh = y.cpu().numpy()
        if bits == 8:
            wq, sc = oracle.pack_w8(w)
            _, ref_r = oracle.gemm_w8a8(qo[rows], so[rows], wq, sc, want_acc=False)
            _, ref_c = oracle.gemm_w8a8(qo, so, wq[cols], sc[cols], want_acc=False)
        else:
            codes, sg = oracle.pack_w4(w, 128)
            _, ref_r = oracle.gemm_w4a8(qo[rows], so[rows], codes, sg, 128, want_acc=False)
            _, ref_c = oracle.gemm_w4a8(qo, so, codes[cols], sg[cols], 128, want_acc=False)
        assert close(yh[rows], ref_r)
        assert close(yh[:, cols], ref_c)
