"""GPU parity of the Hadamard variant (Eq. 4): the quantizers of X H and W H and the quantized linears
built from them, against the CPU oracle.  The rotation is the same butterfly in the same order in both,
so codes and scales are compared bit for bit; the FP16 output within 2^-10 relative + 1e-3 absolute."""
import numpy as np
import pytest
import torch

import oracle
import paper_2512_23367_b200 as pq
from paper_2512_23367_b200 import synth

pytestmark = pytest.mark.gpu
DEV = "cuda:0"
REL, ABS = 2.0 ** -10, 1e-3


def _t(a):
    return torch.from_numpy(a).to(DEV)


def _np(t):
    return t.cpu().numpy()


# block orders 16 / 32 / 64 / 128 / 256 and whole rows of 512 ... 16384 (K a power of two); row teams of
# 32 / 64 / 128 / 256 threads; ragged last row blocks; the benchmark widths 2048, 4096, 6144, 11008
@pytest.mark.parametrize("M,K", [(1, 16), (3, 48), (5, 96), (7, 192), (9, 384), (16, 256), (33, 2048), (130, 4096),
                                 (20, 6144), (70, 11008), (4, 16384), (6, 512), (11, 1024), (3, 8192), (5, 768),
                                 (2, 12288), (300, 128), (9, 64), (5, 32)])
def test_quantize_act_hadamard_bit_exact(M, K):
    assert pq.pq_hadamard_block(K) == oracle.hadamard_block(K)
    x = synth.activations(M, K, 7000 + M)
    q, s_tok = pq.pq_quantize_act_hadamard(_t(x))
    qo, so = oracle.quantize_act_hadamard(x)
    assert np.array_equal(_np(q), qo)
    assert np.array_equal(_np(s_tok).view(np.uint32), so.view(np.uint32))


def test_spike_and_zero_rows():
    x = np.zeros((3, 768), np.float16)
    x[0, 300] = 48.0                      # -> +-3 over the second block of 256, token scale 3 / 127.5
    q, s_tok = pq.pq_quantize_act_hadamard(_t(x))
    q, s_tok = _np(q), _np(s_tok)
    assert (q[0, :256] == 0).all() and (q[0, 512:] == 0).all() and (np.abs(q[0, 256:512].astype(np.int16)) >= 127).all()
    assert s_tok[0] == np.float32(3.0) / np.float32(127.5)
    assert (q[1:] == 0).all() and (s_tok[1:] == 0).all()


@pytest.mark.parametrize("N,K", [(8, 128), (24, 384), (264, 640), (96, 4096), (16, 11008), (40, 512), (24, 2048), (8, 16384),
                                 (16, 256), (16, 768)])
def test_weight_packers_of_WH_bit_exact(N, K):
    w = synth.weights(N, K, 7100 + N)
    wq, s_ch = pq.pq_pack_w8_hadamard(_t(w))
    wqo, s_cho = oracle.pack_w8_hadamard(w)
    assert np.array_equal(_np(pq.pq_unpack_w8(wq, N, K)), wqo)
    assert np.array_equal(_np(s_ch).view(np.uint32), s_cho.view(np.uint32))
    wp, sg = pq.pq_pack_w4_hadamard(_t(w))
    codes, sgo = oracle.pack_w4_hadamard(w, 128)
    assert np.array_equal(_np(pq.pq_unpack_w4(wp, N, K)), codes)
    assert np.array_equal(_np(sg).T.view(np.uint16), sgo.view(np.uint16))       # device layout is [K/128, N]


@pytest.mark.parametrize("M,K,N", [(16, 512, 256), (200, 1024, 264), (300, 4096, 520)])
def test_rotated_linears_end_to_end(M, K, N):
    x, w = synth.activations(M, K, 7200 + M), synth.weights(N, K, 7200 + M)
    xd, wd = _t(x), _t(w)
    q, s_tok = pq.pq_quantize_act_hadamard(xd)
    qo, s_toko = oracle.quantize_act_hadamard(x)
    exact = x.astype(np.float64) @ w.astype(np.float64).T

    wq, s_ch = pq.pq_pack_w8_hadamard(wd)
    y8 = _np(pq.pq_gemm_w8a8(q, s_tok, wq, s_ch, N)).astype(np.float64)
    _, r8 = oracle.gemm_w8a8(qo, s_toko, *oracle.pack_w8_hadamard(w), want_acc=False)
    r8 = r8.astype(np.float64)
    assert np.all(np.abs(y8 - r8) <= REL * np.abs(r8) + ABS)

    wp, sg = pq.pq_pack_w4_hadamard(wd)
    y4 = _np(pq.pq_gemm_w4a8(q, s_tok, wp, sg, N)).astype(np.float64)
    _, r4 = oracle.gemm_w4a8(qo, s_toko, *oracle.pack_w4_hadamard(w, 128), 128, want_acc=False)
    r4 = r4.astype(np.float64)
    assert np.all(np.abs(y4 - r4) <= REL * np.abs(r4) + ABS)
    # what the variant is for: the INT8 x INT8 product gets much closer to X W^T on outlier channels
    qp, stp = pq.pq_quantize_act(xd)
    wqp, scp = pq.pq_pack_w8(wd)
    plain = _np(pq.pq_gemm_w8a8(qp, stp, wqp, scp, N)).astype(np.float64)
    assert np.linalg.norm(y8 - exact) < 0.5 * np.linalg.norm(plain - exact)
    assert pq.pq_device_status() == 0
