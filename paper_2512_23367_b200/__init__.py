"""B200 (sm_100a) quantized linear layer: per-token INT8 activations times INT8 / packed-INT4
weights on the tcgen05 tensor cores, dequantized to FP16.

The compute lives in ``libpq.so`` (CUDA, C ABI declared in ``include/pq.h``); this package is
the argument-marshalling binding with the same call names.  ``synth`` holds the seeded input
generators.  Importing the package does not load the CUDA library; the first call does, and
raises if it cannot be loaded -- there is no CPU or library fallback.
"""
from . import synth  # noqa: F401
from .binding import (  # noqa: F401
    PQError,
    lib,
    pq_acc_w4a8,
    pq_acc_w8a8,
    pq_col_absmax,
    pq_device_status,
    pq_gemm_w4a8,
    pq_gemm_w4a8_group,
    pq_gemm_w8a8,
    pq_gemm_w8a8_group,
    pq_gemm_w8a8_noalloc,
    pq_hadamard_block,
    pq_pack_w4,
    pq_pack_w4_hadamard,
    pq_linear_w4a8,
    pq_linear_w8a8,
    pq_pack_w8,
    pq_pack_w8_hadamard,
    pq_plan_w8a8,
    pq_quantize_act,
    pq_quantize_act_hadamard,
    pq_quantize_act_smooth,
    pq_quantize_act_static,
    pq_quantize_act_static_channel,
    pq_set_wait_limit,
    pq_smooth_scales,
    pq_swiglu_quantize,
    pq_unpack_w4,
    pq_unpack_w8,
    pq_workspace_bytes,
    pq_workspace_init,
)
