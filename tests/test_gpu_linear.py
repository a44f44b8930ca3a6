"""GPU parity for the one-call linear (quantizer + GEMM): where the CUDA-core row kernel serves the shape it
quantizes its own tokens, and the result must be bit for bit that of pq_quantize_act followed by pq_gemm_*,
and within the FP16 tolerance of the oracle's quantizer + GEMM; elsewhere the call runs the two kernels."""
import numpy as np
import pytest
import torch

import oracle
import paper_2512_23367_b200 as pq
from paper_2512_23367_b200 import synth

pytestmark = pytest.mark.gpu
DEV = "cuda:0"
REL, ABS = 2.0 ** -10, 1e-3

# one to four tokens on the row kernel (shares that fit the ring and shares that need refills, K with a short
# last 128-block, N not a multiple of the grid), then shapes that take the two-kernel route
SHAPES = [(1, 4096, 4096), (2, 1000, 640), (3, 2376, 4224), (4, 152, 11008), (1, 4744, 128), (4, 4096, 4096),
          (1, 4096, 11008), (16, 520, 1024), (200, 384, 2048), (300, 1024, 1152)]


def _close(y, ref):
    g, r = y.cpu().numpy().astype(np.float64), ref.astype(np.float64)
    assert np.all(np.abs(g - r) <= REL * np.abs(r) + ABS)


@pytest.mark.parametrize("M,N,K", SHAPES)
def test_linear_w8a8_equals_quantizer_then_gemm_and_the_oracle(M, N, K):
    x, w = synth.activations(M, K, 900 + M), synth.weights(N, K, 910 + M)
    xd = torch.from_numpy(x).to(DEV)
    wq, s_ch = pq.pq_pack_w8(torch.from_numpy(w).to(DEV))
    pad = 256
    buf = torch.full((pad + M * N + pad,), 3.0, dtype=torch.float16, device=DEV)
    y = pq.pq_linear_w8a8(xd, wq, s_ch, N, y=buf[pad:pad + M * N].view(M, N))
    again = pq.pq_linear_w8a8(xd, wq, s_ch, N)
    q, s_tok = pq.pq_quantize_act(xd)
    two = pq.pq_gemm_w8a8(q, s_tok, wq, s_ch, N)
    assert pq.pq_device_status() == 0
    assert torch.equal(y, two) and torch.equal(again, two)
    assert (buf[:pad] == 3.0).all() and (buf[pad + M * N:] == 3.0).all()
    qo, so = oracle.quantize_act(x)
    _, ref = oracle.gemm_w8a8(qo, so, *oracle.pack_w8(w), want_acc=False)
    _close(y, ref)


@pytest.mark.parametrize("M,N,K", [(m, n, k) for (m, n, k) in SHAPES if k % 128 == 0])
def test_linear_w4a8_equals_quantizer_then_gemm_and_the_oracle(M, N, K):
    x, w = synth.activations(M, K, 920 + M), synth.weights(N, K, 930 + M)
    xd = torch.from_numpy(x).to(DEV)
    wp, sg = pq.pq_pack_w4(torch.from_numpy(w).to(DEV))
    y = pq.pq_linear_w4a8(xd, wp, sg, N)
    q, s_tok = pq.pq_quantize_act(xd)
    two = pq.pq_gemm_w4a8(q, s_tok, wp, sg, N)
    assert pq.pq_device_status() == 0
    assert torch.equal(y, two)
    qo, so = oracle.quantize_act(x)
    _, ref = oracle.gemm_w4a8(qo, so, *oracle.pack_w4(w, 128), 128, want_acc=False)
    _close(y, ref)


def test_rows_of_zeros_and_extreme_values():
    """An all-zero token (scale 0, codes 0, output 0) next to one whose largest magnitude is the FP16 maximum."""
    M, N, K = 3, 256, 512
    x = np.zeros((M, K), dtype=np.float16)
    x[1, :] = synth.activations(1, K, 5)[0]
    x[2, 7] = np.float16(65504.0)
    x[2, 100] = np.float16(-65504.0)
    w = synth.weights(N, K, 6)
    xd = torch.from_numpy(x).to(DEV)
    wq, s_ch = pq.pq_pack_w8(torch.from_numpy(w).to(DEV))
    y = pq.pq_linear_w8a8(xd, wq, s_ch, N)
    q, s_tok = pq.pq_quantize_act(xd)
    assert torch.equal(y, pq.pq_gemm_w8a8(q, s_tok, wq, s_ch, N))
    assert (y[0] == 0).all()
    qo, so = oracle.quantize_act(x)
    _, ref = oracle.gemm_w8a8(qo, so, *oracle.pack_w8(w), want_acc=False)
    _close(y, ref)
