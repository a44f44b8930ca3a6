"""GPU parity of the static-scale activation quantizer against the CPU oracle (bit-exact codes), and the
quantized linears fed by it."""
import numpy as np
import pytest
import torch

import oracle
import paper_2512_23367_b200 as pq
from paper_2512_23367_b200 import synth

pytestmark = pytest.mark.gpu
DEV = "cuda:0"
REL, ABS = 2.0 ** -10, 1e-3


@pytest.mark.parametrize("M,K", [(1, 16), (16, 256), (33, 2048), (300, 4096), (70, 11008), (2048, 2048)])
def test_static_quantizer_bit_exact(M, K):
    x = synth.activations(M, K, 8000 + M)
    for s in (np.float32(np.abs(x.astype(np.float32)).max() / 127.5), np.float32(0.037), np.float32(2.0 ** -3)):
        q, s_tok = pq.pq_quantize_act_static(torch.from_numpy(x).to(DEV), torch.tensor([s], device=DEV))
        qo, so = oracle.quantize_act_static(x, s)
        assert np.array_equal(q.cpu().numpy(), qo)
        assert np.array_equal(s_tok.cpu().numpy(), so)
    if M * K >= 4096:                                                            # (the 1 x 16 case has no outlier channel)
        assert (np.abs(qo.astype(np.int16)) == 128).any() or (qo == 127).any()  # the small scales saturate


def test_non_positive_scale_gives_zero_codes():
    x = synth.activations(4, 256, 8100)
    for s in (0.0, -1.0):
        q, s_tok = pq.pq_quantize_act_static(torch.from_numpy(x).to(DEV), torch.tensor([s], device=DEV))
        assert (q == 0).all() and (s_tok == 0).all()


def test_linears_on_statically_quantized_activations():
    M, K, N = 200, 1024, 264
    x, w = synth.activations(M, K, 8200), synth.weights(N, K, 8200)
    s = np.float32(np.abs(x.astype(np.float32)).max() / 127.5)
    q, s_tok = pq.pq_quantize_act_static(torch.from_numpy(x).to(DEV), torch.tensor([s], device=DEV))
    qo, so = oracle.quantize_act_static(x, s)
    wd = torch.from_numpy(w).to(DEV)
    y8 = pq.pq_gemm_w8a8(q, s_tok, *pq.pq_pack_w8(wd), N).cpu().numpy().astype(np.float64)
    _, r8 = oracle.gemm_w8a8(qo, so, *oracle.pack_w8(w), want_acc=False)
    r8 = r8.astype(np.float64)
    assert np.all(np.abs(y8 - r8) <= REL * np.abs(r8) + ABS)
    y4 = pq.pq_gemm_w4a8(q, s_tok, *pq.pq_pack_w4(wd), N).cpu().numpy().astype(np.float64)
    _, r4 = oracle.gemm_w4a8(qo, so, *oracle.pack_w4(w, 128), 128, want_acc=False)
    r4 = r4.astype(np.float64)
    assert np.all(np.abs(y4 - r4) <= REL * np.abs(r4) + ABS)
    assert pq.pq_device_status() == 0


@pytest.mark.parametrize("M,K", [(1, 16), (37, 272), (300, 4096), (64, 11008)])
def test_static_channel_scales_bit_exact(M, K):
    x = synth.activations(M, K, 8300 + M)
    rng = np.random.default_rng(M + K)
    a = np.abs(synth.activations(64, K, 8400 + M).astype(np.float32)).max(axis=0)     # "calibration" maxima per channel
    inv_s = (np.float32(127.5) / np.maximum(a, np.float32(1e-3))).astype(np.float32)
    inv_s[rng.integers(0, K, 3)] = 0.0                                               # dead channels
    inv_s[rng.integers(0, K, 2)] = -1.0
    q, s_tok = pq.pq_quantize_act_static_channel(torch.from_numpy(x).to(DEV), torch.from_numpy(inv_s).to(DEV))
    qo, so = oracle.quantize_act_static_channel(x, inv_s)
    assert np.array_equal(q.cpu().numpy(), qo)
    assert np.array_equal(s_tok.cpu().numpy(), so) and (so == 1.0).all()


def test_linear_on_channel_scaled_activations_with_the_scales_folded_into_the_weights():
    M, K, N = 200, 1024, 264
    x, w = synth.activations(M, K, 8500), synth.weights(N, K, 8500)
    a = np.abs(x.astype(np.float32)).max(axis=0)
    s = (np.maximum(a, np.float32(1e-3)) / np.float32(127.5)).astype(np.float32)
    inv_s = (np.float32(1.0) / s).astype(np.float32)
    q, s_tok = pq.pq_quantize_act_static_channel(torch.from_numpy(x).to(DEV), torch.from_numpy(inv_s).to(DEV))
    wq, s_ch = pq.pq_pack_w8(torch.from_numpy(w).to(DEV), smooth=torch.from_numpy(s).to(DEV))
    y = pq.pq_gemm_w8a8(q, s_tok, wq, s_ch, N).cpu().numpy().astype(np.float64)
    qo, so = oracle.quantize_act_static_channel(x, inv_s)
    _, yo = oracle.gemm_w8a8(qo, so, *oracle.pack_w8(w, smooth=s), want_acc=False)
    yo = yo.astype(np.float64)
    assert np.all(np.abs(y - yo) <= 2.0 ** -10 * np.abs(yo) + 1e-3)
    # sanity: still the product X W^T up to quantization noise (folding the activation scales into the
    # weights moves the outlier channels' range onto the weight side, as Eq. 3 with alpha = 1 would)
    exact = x.astype(np.float64) @ w.astype(np.float64).T
    assert np.linalg.norm(y - exact) < 0.1 * np.linalg.norm(exact)
