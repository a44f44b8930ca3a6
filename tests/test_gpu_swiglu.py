"""GPU parity of pq_swiglu_quantize: the MLP's gated activation h = silu(gate) * up fused with the down
projection's per-token quantizer.  h decides integer codes, so both sides evaluate it as the same fixed
sequence of binary32 operations: codes and token scales must match the CPU oracle bit for bit."""
import numpy as np
import pytest
import torch

import oracle
import paper_2512_23367_b200 as pq
from paper_2512_23367_b200 import synth

pytestmark = pytest.mark.gpu
DEV = "cuda:0"
REL, ABS = 2.0 ** -10, 1e-3


def _gate_up(M, I, seed):
    """Operands shaped like the outputs of the gate and up linears: roughly normal, a few large values,
    exact zeros, and values where e^-g saturates on either side."""
    rng = np.random.default_rng(seed)
    gate = (rng.standard_normal((M, I)) * 2.5).astype(np.float16)
    up = (rng.standard_normal((M, I)) * 4.0).astype(np.float16)
    gate[:, ::97] = 0
    up[:, 5::131] = 0
    gate[0, : min(I, 8)] = np.array([30, -30, 90, -90, 120, -120, 65504, -65504], np.float16)[: min(I, 8)]
    if M > 2:
        gate[2] = 0                       # a token whose gate is closed: zero row, scale 0
    return gate, up


def _run(gate, up):
    q, s = pq.pq_swiglu_quantize(torch.from_numpy(gate).to(DEV), torch.from_numpy(up).to(DEV))
    assert pq.pq_device_status() == 0
    q_ref, s_ref = oracle.swiglu_quantize(gate, up)
    assert np.array_equal(s.cpu().numpy().view(np.uint32), s_ref.view(np.uint32))
    assert np.array_equal(q.cpu().numpy(), q_ref)


@pytest.mark.parametrize("M,I", [(16, 256), (1, 16), (33, 48), (300, 1536), (130, 11008), (64, 6144), (5, 16384),
                                 (257, 2048), (7, 4096), (3, 8192), (2, 12288), (2048, 11008)])
def test_codes_and_scales_bit_exact(M, I):
    _run(*_gate_up(M, I, seed=M + I))


def test_every_finite_fp16_gate_value():
    g = np.arange(65536, dtype=np.uint16).view(np.float16)
    g = g[np.isfinite(g)]
    rows = 4
    I = (len(g) + rows - 1) // rows // 16 * 16 + 16
    gate = np.zeros((rows, I), np.float16)
    gate.reshape(-1)[: len(g)] = g
    for u in (1.0, -3.0, 0.0078125):
        _run(gate, np.full_like(gate, u))


def test_row_longer_than_the_kernel_serves_is_refused():
    g = torch.zeros((2, 16400 // 16 * 16 + 16), dtype=torch.float16, device=DEV)
    with pytest.raises(pq.PQError) as err:
        pq.pq_swiglu_quantize(g, g)
    assert err.value.status == 2


def test_mlp_chain_gate_up_swiglu_down_against_the_oracle():
    """gate/up linears (one grouped launch) -> SwiGLU + quantize -> down linear, every stage compared."""
    M, H, I = 300, 512, 1536
    x = synth.activations(M, H, 81)
    wg, wu, wd = synth.weights(I, H, 82), synth.weights(I, H, 83), synth.weights(H, I, 84)
    q, s_tok = pq.pq_quantize_act(torch.from_numpy(x).to(DEV))
    pg, pu, pd = (pq.pq_pack_w8(torch.from_numpy(w).to(DEV)) for w in (wg, wu, wd))
    g, u = pq.pq_gemm_w8a8_group(q, s_tok, [(pg[0], pg[1], I), (pu[0], pu[1], I)])
    qh, sh = pq.pq_swiglu_quantize(g, u)
    y = pq.pq_gemm_w8a8(qh, sh, pd[0], pd[1], H)
    assert pq.pq_device_status() == 0
    # The oracle's gate/up outputs may differ from the GPU's in the last FP16 bit (binary64 against FP32
    # dequantization), so the fused stage is checked on the GPU's own gate/up values, where it is exact...
    qh_ref, sh_ref = oracle.swiglu_quantize(g.cpu().numpy(), u.cpu().numpy())
    assert np.array_equal(qh.cpu().numpy(), qh_ref) and np.array_equal(sh.cpu().numpy(), sh_ref)
    _, y_ref = oracle.gemm_w8a8(qh_ref, sh_ref, *oracle.pack_w8(wd), want_acc=False)
    gy, ry = y.cpu().numpy().astype(np.float64), y_ref.astype(np.float64)
    assert np.all(np.abs(gy - ry) <= REL * np.abs(ry) + ABS)
    # ... and the whole chain against the oracle's own chain: the two differ by quantization noise only
    qo, so = oracle.quantize_act(x)
    _, go = oracle.gemm_w8a8(qo, so, *oracle.pack_w8(wg), want_acc=False)
    _, uo = oracle.gemm_w8a8(qo, so, *oracle.pack_w8(wu), want_acc=False)
    assert np.all(np.abs(g.cpu().numpy().astype(np.float64) - go) <= REL * np.abs(go) + ABS)
    _, yo = oracle.gemm_w8a8(*oracle.swiglu_quantize(go, uo), *oracle.pack_w8(wd), want_acc=False)
    yo = yo.astype(np.float64)
    assert np.abs(gy - yo).max() <= 0.02 * np.abs(yo).max()
