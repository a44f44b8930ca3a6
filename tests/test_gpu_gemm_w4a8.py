"""GPU parity: W4A8 linear (INT4 weights widened in-kernel, per-group dequantization) against the
CPU oracle.  Per-group INT32 accumulators bit-exact, FP16 output within 2^-10 relative + 1e-3."""
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


def stratified(n, block, rng, extra=()):
    """Sorted sample of range(n): one seeded index in every block of `block`, the edges, and `extra`."""
    starts = np.arange(0, n, block)
    picks = np.minimum(starts + rng.integers(0, block, len(starts)), n - 1)
    return np.unique(np.concatenate([picks, [0, n - 1], np.asarray(extra, dtype=np.int64)])).astype(np.int64)


def run_case(M, N, K, seed, n_out=None, rows=None, cols=None):
    """rows: compare these token rows x all N; cols (with rows): also all M rows x these output channels.
    Without either, every element is compared.  The per-group INT32 accumulators are always compared."""
    x = synth.activations(M, K, seed, n_out)
    w = synth.weights(N, K, seed)
    if N > 2 and K >= 256:
        w[1, 128:256] = 0                  # an all-zero group: scale 0, contributes exactly 0
    q, s_tok = pq.pq_quantize_act(torch.from_numpy(x).to(DEV))
    wp, s_grp = pq.pq_pack_w4(torch.from_numpy(w).to(DEV))
    y = pq.pq_gemm_w4a8(q, s_tok, wp, s_grp, N)
    acc = pq.pq_acc_w4a8(q, wp, N)
    assert pq.pq_device_status() == 0
    q_ref, s_tok_ref = oracle.quantize_act(x)
    codes_ref, sg_ref = oracle.pack_w4(w, 128)
    assert np.array_equal(_np(q), q_ref)
    assert np.array_equal(_np(pq.pq_unpack_w4(wp, N, K)), codes_ref)
    assert np.array_equal(_np(s_grp).view(np.uint16), np.ascontiguousarray(sg_ref.T).view(np.uint16))   # device layout [K/128, N]
    sel = np.arange(M) if rows is None else rows
    sel_d = torch.from_numpy(sel).to(DEV)
    acc_ref, y_ref = oracle.gemm_w4a8(q_ref[sel], s_tok_ref[sel], codes_ref, sg_ref, 128)
    assert np.array_equal(_np(acc[:, sel_d, :]), np.transpose(acc_ref, (2, 0, 1)))
    assert_y_close(_np(y[sel_d]), y_ref)
    if cols is not None:
        cols_d = torch.from_numpy(cols).to(DEV)
        acc_ref, y_ref = oracle.gemm_w4a8(q_ref, s_tok_ref, codes_ref[cols], sg_ref[cols], 128)
        assert np.array_equal(_np(acc[:, :, cols_d]), np.transpose(acc_ref, (2, 0, 1)))
        assert_y_close(_np(y[:, cols_d]), y_ref)


@pytest.mark.parametrize("M", [16, 200])
def test_tiny_linear_every_element(M):
    run_case(M, 256, 256, seed=0, n_out=4)


@pytest.mark.parametrize("M,N,K", [
    (128, 128, 128), (130, 264, 256), (257, 520, 1024), (65, 8, 128), (300, 1024, 4096),
    (129, 136, 11008), (512, 256, 384), (96, 4096, 512), (1, 256, 512), (64, 384, 1280),
    (128, 4096, 4096), (100, 11008, 1024), (65, 1000, 11008), (113, 4096, 11008),
    # 129..256 tokens: narrow linears stream their weights in two token blocks, wide ones stay on the pair kernel
    (200, 4096, 1024), (256, 1152, 4224), (129, 4096, 384), (130, 9608, 256), (200, 9736, 384),
])
def test_shapes_spanning_tiles_and_ragged_tails(M, N, K):
    run_case(M, N, K, seed=M + N + K)


def test_extreme_codes_minus128_times_minus8():
    M, N, K = 130, 136, 1024
    q = torch.full((M, K), -128, dtype=torch.int8, device=DEV)
    wp = torch.full((N * K // 2,), 0x88, dtype=torch.uint8, device=DEV)     # code -8 in both nibbles
    acc = pq.pq_acc_w4a8(q, wp, N)
    assert pq.pq_device_status() == 0
    assert acc.shape == (K // 128, M, N) and (acc == 128 * 128 * 8).all()
    wp7 = torch.full((N * K // 2,), 0x77, dtype=torch.uint8, device=DEV)    # code +7
    assert (pq.pq_acc_w4a8(q, wp7, N) == -128 * 128 * 7).all()


def test_equal_power_of_two_group_scales_reduce_to_integer_sum():
    # with every group scale equal to 2^-3 and token scale 1 the result is exactly acc / 8
    M, N, K = 140, 128, 512
    rng = np.random.default_rng(5)
    q = torch.from_numpy(rng.integers(-20, 21, (M, K)).astype(np.int8)).to(DEV)
    w = torch.from_numpy((rng.integers(-7, 8, (N, K)) * 0.125).astype(np.float16))
    w[:, ::128] = 7.5 * 0.125              # pins every group's max so that each scale is exactly 0.125
    wp, s_grp = pq.pq_pack_w4(w.to(DEV))
    assert (s_grp == 0.125).all()
    ones = torch.ones((M,), dtype=torch.float32, device=DEV)
    y = pq.pq_gemm_w4a8(q, ones, wp, s_grp, N)
    acc = pq.pq_acc_w4a8(q, wp, N).sum(dim=0)
    want = (acc.double() * 0.125).to(torch.float16)
    assert torch.equal(y, want)


@pytest.mark.parametrize("M,K,N", [(2048, 4096, 11008), (2048, 11008, 4096), (2048, 4096, 4096)])
def test_full_size_layers_touch_every_tile(M, K, N):
    """The benchmarked shapes: a token row out of every block of 128 x all N channels, and all M rows x a
    channel out of every block of 64 (at least 256 channels): every output tile is compared, the per-group
    INT32 accumulators bit for bit."""
    rng = np.random.default_rng(M + K + N)
    rows = stratified(M, 128, rng, extra=[127, 128, M - 129])
    cols = stratified(N, 64, rng, extra=rng.integers(0, N, max(0, 256 - N // 64)))
    run_case(M, N, K, seed=4000 + N % 97, rows=rows, cols=cols)
