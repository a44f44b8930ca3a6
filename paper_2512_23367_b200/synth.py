"""Seeded synthetic inputs for the quantized linear layer.

Holds no arithmetic of the method itself: only the random draws and the workload
shapes.  Both the CUDA path and the CPU oracle are fed from here, so that they see
identical bits.

Recipe (stands in for the paper's openPangu-Embedded prefill activations and weights,
which are not available): activations are i.i.d. N(0,1) with a fixed random subset of
K-channels multiplied by 50 -- the heavy-tailed outlier channels the paper's
channel-wise |value| figure shows -- and weights are i.i.d. N(0, 0.02); both are cast
to FP16 (round to nearest even).  The generator is numpy's counter-based Philox stream
keyed by the seed.
"""
from __future__ import annotations

from dataclasses import dataclass

import numpy as np

OUTLIER_GAIN = 50.0
WEIGHT_SIGMA = 0.02
GROUP = 128


def _rng(seed: int, stream: int) -> np.random.Generator:
    return np.random.Generator(np.random.Philox(key=[int(seed), int(stream)]))


def outlier_channels(K: int, seed: int, n_outlier: int | None = None) -> np.ndarray:
    """Indices of the K-channels that carry the x50 gain (sorted)."""
    if n_outlier is None:
        n_outlier = int(round(0.01 * K))
    n_outlier = min(max(int(n_outlier), 0), K)
    idx = _rng(seed, 2).choice(K, size=n_outlier, replace=False)
    return np.sort(idx)


def activations(M: int, K: int, seed: int, n_outlier: int | None = None) -> np.ndarray:
    """FP16 [M,K]: N(0,1) with `n_outlier` channels (default round(0.01*K)) scaled x50."""
    x = _rng(seed, 0).standard_normal((M, K), dtype=np.float32)
    ch = outlier_channels(K, seed, n_outlier)
    x[:, ch] *= np.float32(OUTLIER_GAIN)
    return x.astype(np.float16)


def weights(N: int, K: int, seed: int) -> np.ndarray:
    """FP16 [N,K] (one output channel per row): N(0, 0.02)."""
    w = _rng(seed, 1).standard_normal((N, K), dtype=np.float32)
    w *= np.float32(WEIGHT_SIGMA)
    return w.astype(np.float16)


@dataclass(frozen=True)
class Linear:
    name: str
    K: int
    N: int


def _layer(hidden: int, inter: int) -> tuple[Linear, ...]:
    return (
        Linear("q_proj", hidden, hidden),
        Linear("k_proj", hidden, hidden),
        Linear("v_proj", hidden, hidden),
        Linear("o_proj", hidden, hidden),
        Linear("gate_proj", hidden, inter),
        Linear("up_proj", hidden, inter),
        Linear("down_proj", inter, hidden),
    )


LAYER_1B = _layer(2048, 6144)
LAYER_7B = _layer(4096, 11008)
# The three distinct (K, N) shapes of the 7B-class layer, used by the decode sweep.
SHAPES_7B = (Linear("attn", 4096, 4096), Linear("gate_up", 4096, 11008), Linear("down", 11008, 4096))


@dataclass(frozen=True)
class Workload:
    """One benchmark configuration: a list of linears, the token counts and the weight format."""
    config: int
    name: str
    w_bits: int
    Ms: tuple[int, ...]
    linears: tuple[Linear, ...]
    n_outlier: int | None = None  # None -> round(0.01*K)
    chain: bool = False           # the down projection's input is SwiGLU(gate output, up output), not its own draw

    def seed(self, linear_index: int) -> int:
        return 1000 * self.config + linear_index if self.config else 0


WORKLOADS = {
    "c1_w8a8_tiny": Workload(0, "c1_w8a8_tiny", 8, (16,), (Linear("lin", 256, 256),), n_outlier=4),
    "c2_w8a8_1b_prefill": Workload(2, "c2_w8a8_1b_prefill", 8, (2048,), LAYER_1B),
    "c3_w8a8_7b_prefill": Workload(3, "c3_w8a8_7b_prefill", 8, (512, 4096), LAYER_7B),
    "c4_w4a8_7b_prefill": Workload(4, "c4_w4a8_7b_prefill", 4, (2048,), LAYER_7B),
    "c5_w8a8_7b_decode": Workload(5, "c5_w8a8_7b_decode", 8, (1, 4, 16, 64), SHAPES_7B),
    "c5_w4a8_7b_decode": Workload(6, "c5_w4a8_7b_decode", 4, (1, 4, 16, 64), SHAPES_7B),
    # The whole 7B-class layer at decode-shaped token counts (q/k/v and gate/up share their inputs, so the
    # grouped calls apply): the same seven linears as c3, the token counts of c5.
    "c5l_w8a8_7b_decode_layer": Workload(7, "c5l_w8a8_7b_decode_layer", 8, (1, 4, 16, 64), LAYER_7B),
    "c5l_w4a8_7b_decode_layer": Workload(8, "c5l_w4a8_7b_decode_layer", 4, (1, 4, 16, 64), LAYER_7B),
    # The 7B-class layer as a chain: the MLP's down projection consumes SwiGLU(gate, up) of the step's own
    # gate/up outputs, re-quantized in the same pass (token counts of the prefill sweep).
    "c3l_w8a8_7b_layer_chain": Workload(9, "c3l_w8a8_7b_layer_chain", 8, (128, 256, 512, 1024, 2048, 4096), LAYER_7B,
                                        chain=True),
    "c4l_w4a8_7b_layer_chain": Workload(10, "c4l_w4a8_7b_layer_chain", 4, (128, 256, 512, 1024, 2048, 4096), LAYER_7B,
                                        chain=True),
}


def linear_inputs(wl: Workload, linear_index: int, M: int):
    """(x f16 [M,K], w f16 [N,K]) for one linear of a workload."""
    lin = wl.linears[linear_index]
    s = wl.seed(linear_index)
    return activations(M, lin.K, s, wl.n_outlier), weights(lin.N, lin.K, s)
