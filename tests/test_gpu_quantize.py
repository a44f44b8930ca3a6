"""GPU parity: activation quantizer and weight packers against the CPU oracle (bit-exact)."""
import numpy as np
import pytest
import torch

import oracle
import paper_2512_23367_b200 as pq
from paper_2512_23367_b200 import synth

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def _np(t):
    return t.cpu().numpy()


@pytest.mark.parametrize("M,K,n_out", [(16, 256, 4), (1, 4096, None), (37, 2048, None), (64, 11008, None),
                                       (300, 4096, None), (5, 16, 1), (9, 1040, 3), (3, 32768, 10),
                                       (2, 66000 // 16 * 16, 5)])
def test_quantize_act_codes_and_scales_bit_exact(M, K, n_out):
    x = synth.activations(M, K, seed=M * 7 + K, n_outlier=n_out)
    if M > 4:
        x[2] = 0                       # all-zero token
        x[3] = np.float16(-3.0)        # every element is -max: all codes -128
    if M > 8:
        x[4, ::2] = np.float16(127.5) * np.float16(2.0 ** -3)   # +max and planted ties
        x[4, 1::2] = (np.arange(K // 2) % 255 - 127).astype(np.float16) * np.float16(2.0 ** -3) + np.float16(0.0625)
    q_ref, s_ref = oracle.quantize_act(x)
    q, s = pq.pq_quantize_act(torch.from_numpy(x).to(DEV))
    assert pq.pq_device_status() == 0
    assert np.array_equal(_np(s).view(np.uint32), s_ref.view(np.uint32))
    assert np.array_equal(_np(q), q_ref)


@pytest.mark.parametrize("N,K", [(256, 256), (64, 4096), (40, 11008), (8, 16), (24, 2064)])
def test_pack_w8_bit_exact(N, K):
    w = synth.weights(N, K, seed=N + K)
    w[1] = 0
    wq_ref, s_ref = oracle.pack_w8(w)
    wq, s_ch = pq.pq_pack_w8(torch.from_numpy(w).to(DEV))
    codes = pq.pq_unpack_w8(wq, N, K)
    assert np.array_equal(_np(s_ch).view(np.uint32), s_ref.view(np.uint32))
    assert np.array_equal(_np(codes), wq_ref)


@pytest.mark.parametrize("N,K", [(256, 256), (64, 4096), (40, 11008), (8, 128)])
def test_pack_w4_bit_exact_and_round_trip(N, K):
    w = synth.weights(N, K, seed=N + K + 1)
    w[1, :128] = 0                     # an all-zero group
    w[2, 5] = np.float16(0.3)          # a large value: other codes of its group collapse towards 0
    codes_ref, sg_ref = oracle.pack_w4(w, 128)
    wp, s_grp = pq.pq_pack_w4(torch.from_numpy(w).to(DEV))
    assert s_grp.shape == (K // 128, N)
    assert np.array_equal(_np(s_grp).T.copy().view(np.uint16), sg_ref.view(np.uint16))
    codes = pq.pq_unpack_w4(wp, N, K)
    assert np.array_equal(_np(codes), codes_ref)
    assert wp.numel() == N * K // 2


def test_entry_points_reject_bad_arguments_on_device():
    x = torch.zeros((4, 64), dtype=torch.float16, device=DEV)
    with pytest.raises(ValueError):
        pq.pq_quantize_act(torch.zeros((4, 64), dtype=torch.float16))      # CPU tensor: no CPU path
    with pytest.raises(pq.PQError) as e:
        pq.pq_quantize_act(x[:, :40].contiguous())                          # K % 16 != 0
    assert e.value.status == 2
    with pytest.raises(pq.PQError) as e:
        pq.pq_pack_w4(torch.zeros((8, 256), dtype=torch.float16, device=DEV), group=64)
    assert e.value.status == 2
