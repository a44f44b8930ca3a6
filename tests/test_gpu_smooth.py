"""GPU parity of the SmoothQuant variant (Eq. 3): column maxima, the scale vector, the quantizers of
X S^-1 and S W, and the quantized linears built from them, against the CPU oracle.  Integer codes and
every stored scale are compared bit for bit; the FP16 output within 2^-10 relative + 1e-3 absolute."""
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


@pytest.mark.parametrize("R,K", [(1, 16), (37, 208), (64, 256), (65, 4096), (300, 11008)])
def test_col_absmax_bit_exact(R, K):
    a = synth.activations(R, K, 6000 + R)
    a[R // 2, K // 3] = -30000.0
    assert np.array_equal(_np(pq.pq_col_absmax(_t(a))), oracle.col_absmax(a))


def test_smooth_scales_bit_exact_including_dead_channels():
    rng = np.random.default_rng(61)
    xa = rng.uniform(0.01, 80.0, 4096).astype(np.float32)
    wa = rng.uniform(0.001, 0.3, 4096).astype(np.float32)
    xa[5], wa[9] = 0.0, 0.0
    s, s_inv = pq.pq_smooth_scales(_t(xa), _t(wa))
    so, sio = oracle.smooth_scales(xa, wa)
    assert np.array_equal(_np(s).view(np.uint32), so.view(np.uint32))
    assert np.array_equal(_np(s_inv).view(np.uint32), sio.view(np.uint32))
    assert _np(s)[5] == 1.0 and _np(s)[9] == 1.0


@pytest.mark.parametrize("alpha_quarters", [0, 1, 2, 3, 4])
def test_smooth_scales_for_quarter_alphas_bit_exact(alpha_quarters):
    rng = np.random.default_rng(63)
    xa = rng.uniform(0.01, 80.0, 11008).astype(np.float32)
    wa = rng.uniform(0.001, 0.3, 11008).astype(np.float32)
    xa[5], wa[9] = 0.0, 0.0
    s, s_inv = pq.pq_smooth_scales(_t(xa), _t(wa), alpha_quarters)
    so, sio = oracle.smooth_scales_alpha(xa, wa, alpha_quarters)
    assert np.array_equal(_np(s).view(np.uint32), so.view(np.uint32))
    assert np.array_equal(_np(s_inv).view(np.uint32), sio.view(np.uint32))


def test_alpha_outside_the_quarters_is_refused():
    v = _t(np.ones(64, np.float32))
    with pytest.raises(pq.PQError) as err:
        pq.pq_smooth_scales(v, v, 5)
    assert err.value.status == 2


# row teams of 32 / 64 / 128 / 256 threads, ragged row blocks, K beyond the register-cached part
@pytest.mark.parametrize("M,K", [(1, 16), (16, 256), (9, 2048), (130, 4096), (33, 6144), (70, 11008), (5, 20480)])
def test_quantize_act_smooth_bit_exact(M, K):
    x = synth.activations(M, K, 6100 + M)
    s_inv = np.random.default_rng(62 + M).uniform(0.01, 4.0, K).astype(np.float32)
    q, s_tok = pq.pq_quantize_act_smooth(_t(x), _t(s_inv))
    qo, so = oracle.quantize_act(x, s_inv)
    assert np.array_equal(_np(q), qo)
    assert np.array_equal(_np(s_tok).view(np.uint32), so.view(np.uint32))
    assert not np.array_equal(qo, oracle.quantize_act(x)[0])


def test_zero_rows_and_zero_factors_give_zero_codes_and_scale():
    x = synth.activations(4, 256, 6200)
    x[1] = 0
    s_inv = np.ones(256, np.float32)
    s_inv[::2] = 0.0
    q, s_tok = pq.pq_quantize_act_smooth(_t(x), _t(s_inv))
    qo, so = oracle.quantize_act(x, s_inv)
    assert np.array_equal(_np(q), qo) and np.array_equal(_np(s_tok), so)
    assert (qo[1] == 0).all() and so[1] == 0.0 and (qo[:, ::2] == 0).all()
    q0, s0 = pq.pq_quantize_act_smooth(_t(x), _t(np.zeros(256, np.float32)))
    assert (_np(q0) == 0).all() and (_np(s0) == 0).all()


@pytest.mark.parametrize("N,K", [(8, 128), (264, 384), (96, 4096), (24, 11008)])
def test_weight_packers_of_SW_bit_exact(N, K):
    w = synth.weights(N, K, 6300 + N)
    s = np.random.default_rng(63 + N).uniform(0.2, 30.0, K).astype(np.float32)
    wq, s_ch = pq.pq_pack_w8(_t(w), _t(s))
    wqo, s_cho = oracle.pack_w8(w, s)
    assert np.array_equal(_np(pq.pq_unpack_w8(wq, N, K)), wqo)
    assert np.array_equal(_np(s_ch).view(np.uint32), s_cho.view(np.uint32))
    wp, sg = pq.pq_pack_w4(_t(w), 128, _t(s))
    codes, sgo = oracle.pack_w4(w, 128, s)
    assert np.array_equal(_np(pq.pq_unpack_w4(wp, N, K)), codes)
    assert np.array_equal(_np(sg).T.view(np.uint16), sgo.view(np.uint16))       # device layout is [K/128, N]


@pytest.mark.parametrize("M,K,N", [(16, 512, 256), (200, 1024, 264), (300, 4096, 520)])
def test_smoothed_linears_end_to_end(M, K, N):
    """Calibrate on the activations themselves, smooth both sides, run the unchanged GEMMs."""
    x, w = synth.activations(M, K, 6400 + M), synth.weights(N, K, 6400 + M)
    xd, wd = _t(x), _t(w)
    s, s_inv = pq.pq_smooth_scales(pq.pq_col_absmax(xd), pq.pq_col_absmax(wd))
    so, sio = oracle.smooth_scales(oracle.col_absmax(x), oracle.col_absmax(w))
    assert np.array_equal(_np(s), so) and np.array_equal(_np(s_inv), sio)
    q, s_tok = pq.pq_quantize_act_smooth(xd, s_inv)
    qo, s_toko = oracle.quantize_act(x, sio)
    assert np.array_equal(_np(q), qo)
    exact = x.astype(np.float64) @ w.astype(np.float64).T

    wq, s_ch = pq.pq_pack_w8(wd, s)
    y8 = _np(pq.pq_gemm_w8a8(q, s_tok, wq, s_ch, N)).astype(np.float64)
    _, r8 = oracle.gemm_w8a8(qo, s_toko, *oracle.pack_w8(w, so), want_acc=False)
    r8 = r8.astype(np.float64)
    assert np.all(np.abs(y8 - r8) <= REL * np.abs(r8) + ABS)

    wp, sg = pq.pq_pack_w4(wd, 128, s)
    y4 = _np(pq.pq_gemm_w4a8(q, s_tok, wp, sg, N)).astype(np.float64)
    _, r4 = oracle.gemm_w4a8(qo, s_toko, *oracle.pack_w4(w, 128, so), 128, want_acc=False)
    r4 = r4.astype(np.float64)
    assert np.all(np.abs(y4 - r4) <= REL * np.abs(r4) + ABS)
    # what the variant is for: closer to the unquantized product than plain W4A8 on outlier channels
    qp, stp = pq.pq_quantize_act(xd)
    wpp, sgp = pq.pq_pack_w4(wd)
    plain = _np(pq.pq_gemm_w4a8(qp, stp, wpp, sgp, N)).astype(np.float64)
    assert np.linalg.norm(y4 - exact) < 0.8 * np.linalg.norm(plain - exact)
    assert pq.pq_device_status() == 0
