"""GPU parity for decode-shaped calls (M <= 128): the weight-streaming schedule must give the same
INT32 accumulators (bit-exact) and FP16 outputs (within tolerance) as the CPU oracle."""
import numpy as np
import pytest
import torch

import oracle
import paper_2512_23367_b200 as pq
from paper_2512_23367_b200 import synth

pytestmark = pytest.mark.gpu
DEV = "cuda:0"
REL, ABS = 2.0 ** -10, 1e-3


def _np(t):
    return t.cpu().numpy()


def assert_y_close(y_gpu, y_ref):
    g, r = y_gpu.astype(np.float64), y_ref.astype(np.float64)
    assert np.isfinite(g).all()
    bad = np.abs(g - r) > REL * np.abs(r) + ABS
    assert not bad.any(), (int(bad.sum()), np.argwhere(bad)[:5], g[bad][:5], r[bad][:5])


def run_w8(M, N, K, seed):
    x, w = synth.activations(M, K, seed), synth.weights(N, K, seed)
    q, s_tok = pq.pq_quantize_act(torch.from_numpy(x).to(DEV))
    wq, s_ch = pq.pq_pack_w8(torch.from_numpy(w).to(DEV))
    pad = 1024
    buf = torch.full((pad + M * N + pad,), 7.0, dtype=torch.float16, device=DEV)
    y = buf[pad:pad + M * N].view(M, N)
    pq.pq_gemm_w8a8(q, s_tok, wq, s_ch, N, y=y)
    acc = pq.pq_acc_w8a8(q, wq, N)
    assert pq.pq_device_status() == 0
    q_ref, st_ref = oracle.quantize_act(x)
    wq_ref, sc_ref = oracle.pack_w8(w)
    acc_ref, y_ref = oracle.gemm_w8a8(q_ref, st_ref, wq_ref, sc_ref)
    assert np.array_equal(_np(q), q_ref)
    assert np.array_equal(_np(acc), acc_ref)
    assert_y_close(_np(y), y_ref)
    assert (buf[:pad] == 7.0).all() and (buf[pad + M * N:] == 7.0).all()


def run_w4(M, N, K, seed):
    x, w = synth.activations(M, K, seed), synth.weights(N, K, seed)
    q, s_tok = pq.pq_quantize_act(torch.from_numpy(x).to(DEV))
    wp, s_grp = pq.pq_pack_w4(torch.from_numpy(w).to(DEV))
    y = pq.pq_gemm_w4a8(q, s_tok, wp, s_grp, N)
    acc = pq.pq_acc_w4a8(q, wp, N)
    assert pq.pq_device_status() == 0
    q_ref, st_ref = oracle.quantize_act(x)
    codes_ref, sg_ref = oracle.pack_w4(w, 128)
    acc_ref, y_ref = oracle.gemm_w4a8(q_ref, st_ref, codes_ref, sg_ref, 128)
    assert np.array_equal(_np(acc), np.transpose(acc_ref, (2, 0, 1)))
    assert_y_close(_np(y), y_ref)


SMALL = [(1, 256, 256), (4, 136, 384), (16, 520, 1024), (17, 128, 128), (33, 264, 2048), (64, 1024, 1152),
         (3, 8, 128), (48, 4096, 256),
         # one to four tokens may take the CUDA-core row kernel: row sets not a multiple of the grid, shares
         # that fit the ring and shares that need refills, K with a short last 128-block, every token count
         (2, 1000, 640), (3, 2376, 4224), (4, 152, 11008), (1, 4744, 128), (2, 8, 8192)]


@pytest.mark.parametrize("M,N,K", SMALL + [(5, 264, 144), (64, 8, 16)])
def test_w8a8_small_m(M, N, K):
    run_w8(M, N, K, seed=M * 3 + N + K)


@pytest.mark.parametrize("M,N,K", SMALL + [(65, 264, 2048), (128, 520, 1152), (100, 136, 4224), (127, 1408, 384)])
def test_w4a8_small_m(M, N, K):
    run_w4(M, N, K, seed=M * 5 + N + K)


@pytest.mark.parametrize("M", [1, 4, 16, 64])
@pytest.mark.parametrize("K,N", [(4096, 4096), (4096, 11008), (11008, 4096)])
def test_decode_sweep_7b_shapes_every_element(M, K, N):
    run_w8(M, N, K, seed=5000 + M)
    run_w4(M, N, K, seed=6000 + M)
