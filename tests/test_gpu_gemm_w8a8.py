"""GPU parity: W8A8 linear against the CPU oracle.  INT32 accumulators bit-exact, FP16 output
within 2^-10 relative + 1e-3 absolute."""
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
    picks = starts + rng.integers(0, block, len(starts))
    picks = np.minimum(picks, n - 1)
    return np.unique(np.concatenate([picks, [0, n - 1], np.asarray(extra, dtype=np.int64)])).astype(np.int64)


def run_case(M, N, K, seed, n_out=None, rows=None, cols=None):
    """rows: compare these token rows x all N; cols (with rows): also all M rows x these output channels.
    Without either, every element is compared."""
    x = synth.activations(M, K, seed, n_out)
    w = synth.weights(N, K, seed)
    xd, wd = torch.from_numpy(x).to(DEV), torch.from_numpy(w).to(DEV)
    q, s_tok = pq.pq_quantize_act(xd)
    wq, s_ch = pq.pq_pack_w8(wd)
    acc = pq.pq_acc_w8a8(q, wq, N)
    y = pq.pq_gemm_w8a8(q, s_tok, wq, s_ch, N)
    assert pq.pq_device_status() == 0
    q_ref, s_tok_ref = oracle.quantize_act(x)
    wq_ref, s_ch_ref = oracle.pack_w8(w)
    assert np.array_equal(_np(q), q_ref)
    assert np.array_equal(_np(s_tok), s_tok_ref)
    assert np.array_equal(_np(pq.pq_unpack_w8(wq, N, K)), wq_ref)
    sel = np.arange(M) if rows is None else rows
    acc_ref, y_ref = oracle.gemm_w8a8(q_ref[sel], s_tok_ref[sel], wq_ref, s_ch_ref)
    sel_d = torch.from_numpy(sel).to(DEV)
    assert np.array_equal(_np(acc[sel_d]), acc_ref)
    assert_y_close(_np(y[sel_d]), y_ref)
    if cols is not None:
        acc_ref, y_ref = oracle.gemm_w8a8(q_ref, s_tok_ref, wq_ref[cols], s_ch_ref[cols])
        cols_d = torch.from_numpy(cols).to(DEV)
        assert np.array_equal(_np(acc[:, cols_d]), acc_ref)
        assert_y_close(_np(y[:, cols_d]), y_ref)


def test_config1_tiny_linear_every_element():
    run_case(16, 256, 256, seed=0, n_out=4)


@pytest.mark.parametrize("M,N,K", [
    (128, 256, 128), (130, 264, 144), (257, 520, 1040), (200, 384, 2048), (65, 8, 16),
    (300, 1024, 4096), (129, 136, 11008), (512, 256, 256), (96, 4096, 512),
    # 129..256 tokens: narrow linears stream their weights in two token blocks, wide ones stay on the pair kernel
    (256, 4096, 1024), (200, 1152, 4224), (130, 9608, 256), (200, 9736, 384),
])
def test_shapes_spanning_tiles_and_ragged_tails(M, N, K):
    run_case(M, N, K, seed=M + N + K)


def test_extreme_codes_minus128_times_minus128():
    M, N, K = 130, 264, 11008
    q = torch.full((M, K), -128, dtype=torch.int8, device=DEV)
    wq = torch.full((N * K,), 0x80, dtype=torch.uint8, device=DEV)      # code -128 everywhere
    acc = pq.pq_acc_w8a8(q, wq, N)
    assert pq.pq_device_status() == 0
    assert (acc == K * 16384).all()
    q[1::2] = 127
    acc = _np(pq.pq_acc_w8a8(q, wq, N))
    assert (acc[0::2] == K * 16384).all() and (acc[1::2] == -K * 127 * 128).all()


def test_identity_weights_return_the_codes():
    M, K = 140, 256
    x = synth.activations(M, K, seed=3)
    q, s_tok = pq.pq_quantize_act(torch.from_numpy(x).to(DEV))
    eye = torch.eye(K, dtype=torch.float16, device=DEV) * 0.75
    wq, s_ch = pq.pq_pack_w8(eye)
    assert np.array_equal(_np(pq.pq_unpack_w8(wq, K, K)), oracle.pack_w8(_np(eye))[0])
    acc = pq.pq_acc_w8a8(q, wq, K)
    assert torch.equal(acc, 127 * q.to(torch.int32))       # +max -> 127.5 -> 128 -> clamped to 127
    wqn, _ = pq.pq_pack_w8(-eye)
    assert np.array_equal(_np(pq.pq_unpack_w8(wqn, K, K)), oracle.pack_w8(_np(-eye))[0])
    assert torch.equal(pq.pq_acc_w8a8(q, wqn, K), -128 * q.to(torch.int32))


def test_output_guard_bands_stay_untouched():
    M, N, K = 130, 264, 256
    x = synth.activations(M, K, seed=9)
    w = synth.weights(N, K, seed=9)
    q, s_tok = pq.pq_quantize_act(torch.from_numpy(x).to(DEV))
    wq, s_ch = pq.pq_pack_w8(torch.from_numpy(w).to(DEV))
    pad = 4096
    buf = torch.full((pad + M * N + pad,), 7.0, dtype=torch.float16, device=DEV)
    y = buf[pad:pad + M * N].view(M, N)
    pq.pq_gemm_w8a8(q, s_tok, wq, s_ch, N, y=y)
    assert pq.pq_device_status() == 0
    assert (buf[:pad] == 7.0).all() and (buf[pad + M * N:] == 7.0).all()


# every (K, N) of the 1B-class layer at M = 2048 and of the 7B-class layer at M = 512 and M = 4096
@pytest.mark.parametrize("M,K,N", [(2048, 2048, 2048), (2048, 2048, 6144), (2048, 6144, 2048),
                                   (512, 4096, 4096), (512, 4096, 11008), (512, 11008, 4096),
                                   (4096, 4096, 4096), (4096, 4096, 11008), (4096, 11008, 4096)])
def test_full_size_layers_touch_every_tile(M, K, N):
    """The benchmarked shapes: a token row out of every block of 128 rows x all N channels, and all M rows
    x a channel out of every block of 64 (at least 256 channels) -- every output tile of every tiling the
    kernel may choose is compared, the INT32 accumulators bit for bit."""
    rng = np.random.default_rng(M + K + N)
    rows = stratified(M, 128, rng, extra=[127, 128, M - 129])
    cols = stratified(N, 64, rng, extra=rng.integers(0, N, max(0, 256 - N // 64)))
    assert len(cols) >= min(N, 200)
    run_case(M, N, K, seed=2000 + N % 97, rows=rows, cols=cols)


@pytest.mark.parametrize("M,K,N", [(512, 11008, 1024), (300, 11008, 520), (260, 6144, 136), (257, 8192, 264)])
def test_split_k_through_scratch_matches_the_unsplit_result_bit_for_bit(M, K, N):
    """Few tiles and a long K: given a workspace the GEMM cuts K into parts and sums the INT32 partials
    exactly, so the FP16 output must equal the one computed without a workspace, twice in a row (the
    arrival counters go back to zero), and must match the oracle."""
    need = pq.pq_workspace_bytes(M, N, K)
    assert need > 0 and pq.pq_plan_w8a8(M, N, K, 148, need)[1] > 1      # K really is split
    x = synth.activations(M, K, seed=77)
    w = synth.weights(N, K, seed=78)
    q, s_tok = pq.pq_quantize_act(torch.from_numpy(x).to(DEV))
    wq, s_ch = pq.pq_pack_w8(torch.from_numpy(w).to(DEV))
    ws = pq.pq_workspace_init(torch.full((need,), 0xAB, dtype=torch.uint8, device=DEV))
    pad = 2048
    buf = torch.full((pad + M * N + pad,), 7.0, dtype=torch.float16, device=DEV)
    y_split = buf[pad:pad + M * N].view(M, N)
    pq.pq_gemm_w8a8(q, s_tok, wq, s_ch, N, y=y_split, workspace=ws)
    y_again = pq.pq_gemm_w8a8(q, s_tok, wq, s_ch, N, workspace=ws)
    y_plain = pq.pq_gemm_w8a8(q, s_tok, wq, s_ch, N)                    # no workspace: no split
    assert pq.pq_device_status() == 0
    assert torch.equal(y_split, y_plain) and torch.equal(y_again, y_plain)
    assert (buf[:pad] == 7.0).all() and (buf[pad + M * N:] == 7.0).all()
    q_ref, st_ref = oracle.quantize_act(x)
    wq_ref, sc_ref = oracle.pack_w8(w)
    rows = np.unique(np.concatenate([[0, 127, 128, M - 1], np.arange(0, M, 37)]))
    _, y_ref = oracle.gemm_w8a8(q_ref[rows], st_ref[rows], wq_ref, sc_ref)
    assert_y_close(_np(y_split)[rows], y_ref)


def test_two_streams_with_their_own_workspaces_run_split_k_concurrently():
    """Calls that may overlap on the GPU get separate workspaces: two streams each issue a chain of
    split-K GEMMs (different inputs) with nothing ordering one chain against the other; every result
    must equal the one computed serially, bit for bit."""
    M, K, N = 512, 11008, 1024
    need = pq.pq_workspace_bytes(M, N, K)
    assert pq.pq_plan_w8a8(M, N, K, 148, need)[1] > 1
    cases = []
    for i in range(2):
        x = synth.activations(M, K, seed=300 + i)
        w = synth.weights(N, K, seed=310 + i)
        q, s_tok = pq.pq_quantize_act(torch.from_numpy(x).to(DEV))
        wq, s_ch = pq.pq_pack_w8(torch.from_numpy(w).to(DEV))
        ws = pq.pq_workspace_init(torch.empty((need,), dtype=torch.uint8, device=DEV))
        serial = pq.pq_gemm_w8a8(q, s_tok, wq, s_ch, N)                 # unsplit, default stream
        cases.append((q, s_tok, wq, s_ch, ws, serial))
    torch.cuda.synchronize()
    streams = [torch.cuda.Stream(device=DEV) for _ in cases]
    reps = 12
    outs = [[torch.empty((M, N), dtype=torch.float16, device=DEV) for _ in range(reps)] for _ in cases]
    for r in range(reps):                                              # interleaved issue: the chains overlap
        for (q, s_tok, wq, s_ch, ws, _), st, ys in zip(cases, streams, outs):
            with torch.cuda.stream(st):
                pq.pq_gemm_w8a8(q, s_tok, wq, s_ch, N, y=ys[r], workspace=ws)
    torch.cuda.synchronize()
    assert pq.pq_device_status() == 0
    for (_, _, _, _, _, serial), ys in zip(cases, outs):
        for y in ys:
            assert torch.equal(y, serial)


def test_host_threads_call_concurrently_on_their_own_streams():
    """The library keeps no per-call host state: four host threads, each with its own stream, inputs and
    workspace, issue split-K and unsplit GEMMs at the same time (ctypes drops the GIL inside the calls); every
    result equals the one computed serially."""
    import threading
    shapes = [(512, 11008, 1024), (300, 1024, 520), (512, 11008, 1024), (140, 6144, 136)]
    cases = []
    for i, (M, K, N) in enumerate(shapes):
        x, w = synth.activations(M, K, seed=500 + i), synth.weights(N, K, seed=510 + i)
        q, s_tok = pq.pq_quantize_act(torch.from_numpy(x).to(DEV))
        wq, s_ch = pq.pq_pack_w8(torch.from_numpy(w).to(DEV))
        need = pq.pq_workspace_bytes(M, N, K)
        ws = pq.pq_workspace_init(torch.empty((need,), dtype=torch.uint8, device=DEV)) if need else None
        serial = pq.pq_gemm_w8a8(q, s_tok, wq, s_ch, N)
        cases.append((q, s_tok, wq, s_ch, N, ws, serial))
    torch.cuda.synchronize()
    results, errors = [None] * len(cases), []

    def work(i):
        try:
            q, s_tok, wq, s_ch, N, ws, _ = cases[i]
            st = torch.cuda.Stream(device=DEV)
            outs = []
            with torch.cuda.stream(st):
                for _ in range(20):
                    outs.append(pq.pq_gemm_w8a8(q, s_tok, wq, s_ch, N, workspace=ws))
            st.synchronize()
            results[i] = outs
        except Exception as e:      # surfaced below: an exception in a thread must fail the test
            errors.append(e)

    threads = [threading.Thread(target=work, args=(i,)) for i in range(len(cases))]
    for t in threads:
        t.start()
    for t in threads:
        t.join()
    assert not errors, errors
    assert pq.pq_device_status() == 0
    for (_, _, _, _, _, _, serial), outs in zip(cases, results):
        for y in outs:
            assert torch.equal(y, serial)


@pytest.mark.parametrize("M", [1, 16, 130])
def test_longest_k_the_int32_accumulator_allows(M):
    """K = 131056 is the largest K the shape rule admits (K * 128 * 128 < 2^31): with every code at -128 the
    accumulator reaches 131056 * 16384 = 2 147 221 504, 262 144 below the INT32 limit, on every schedule."""
    K, N = 131056, 264
    q = torch.full((M, K), -128, dtype=torch.int8, device=DEV)
    wq = torch.full((N * K,), 0x80, dtype=torch.uint8, device=DEV)
    acc = pq.pq_acc_w8a8(q, wq, N)
    assert pq.pq_device_status() == 0
    assert (acc == K * 16384).all() and K * 16384 < 2 ** 31
    q[:, 1::2] = 127                                   # alternate signs: the sum stays small, every product is extreme
    acc = _np(pq.pq_acc_w8a8(q, wq, N))
    assert (acc == (K // 2) * (16384 - 127 * 128)).all()
    with pytest.raises(pq.PQError) as err:             # one step further is refused before anything runs
        pq.pq_acc_w8a8(torch.zeros((M, 131072), dtype=torch.int8, device=DEV),
                       torch.zeros((N * 131072,), dtype=torch.uint8, device=DEV), N)
    assert err.value.status == 2
