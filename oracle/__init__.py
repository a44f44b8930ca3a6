"""CPU oracle for the quantized linear layer -- TEST INFRASTRUCTURE ONLY.

Thin numpy/ctypes wrapper around ``pq_oracle.c`` (plain C, compiled with gcc).  Only
tests, the smoke check and the benchmark's CPU-baseline leg may import this package;
the CUDA library and its Python binding never do, and this package never imports them.

Every function takes and returns numpy arrays; FP16 tensors are ``np.float16`` arrays
(passed to C as their 16-bit patterns).
"""
from __future__ import annotations

import ctypes
import os
import subprocess

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "pq_oracle.c")
_SO = os.path.join(_HERE, "libpq_oracle.so")

CFLAGS = ["-O2", "-std=c11", "-fPIC", "-shared", "-fopenmp", "-ffp-contract=off", "-fno-fast-math",
          "-Wall", "-Wextra"]


def build(force: bool = False) -> str:
    """Compile the oracle with gcc if the shared object is missing or stale."""
    if force or not os.path.exists(_SO) or os.path.getmtime(_SO) < os.path.getmtime(_SRC):
        tmp = _SO + f".tmp{os.getpid()}"
        subprocess.check_call(["gcc", *CFLAGS, "-o", tmp, _SRC, "-lm"])
        os.replace(tmp, _SO)
    return _SO


_lib = None


def _load():
    global _lib
    if _lib is None:
        lib = ctypes.CDLL(build())
        i64, vp = ctypes.c_int64, ctypes.c_void_p
        lib.pqo_half_to_float.restype = ctypes.c_float
        lib.pqo_half_to_float.argtypes = [ctypes.c_uint16]
        lib.pqo_double_to_half_rne.restype = ctypes.c_uint16
        lib.pqo_double_to_half_rne.argtypes = [ctypes.c_double]
        lib.pqo_float_to_half_rne.restype = ctypes.c_uint16
        lib.pqo_float_to_half_rne.argtypes = [ctypes.c_float]
        lib.pqo_quantize_act.argtypes = [vp, i64, i64, vp, vp]
        lib.pqo_pack_w8.argtypes = [vp, i64, i64, vp, vp]
        lib.pqo_pack_w4.argtypes = [vp, i64, i64, i64, vp, vp]
        lib.pqo_nibble_pack.argtypes = [vp, i64, i64, vp]
        lib.pqo_nibble_unpack.argtypes = [vp, i64, i64, vp]
        lib.pqo_gemm_w8a8.argtypes = [vp, vp, vp, vp, i64, i64, i64, vp, vp]
        lib.pqo_gemm_w4a8.argtypes = [vp, vp, vp, vp, i64, i64, i64, i64, vp, vp]
        lib.pqo_num_threads.restype = ctypes.c_int
        _lib = lib
    return _lib


class OracleError(RuntimeError):
    pass


def _check(rc: int, what: str) -> None:
    if rc == 1:
        raise OverflowError(f"{what}: an integer accumulator left the int32 range")
    if rc != 0:
        raise OracleError(f"{what}: bad argument (code {rc})")


def _c(a: np.ndarray, dtype) -> np.ndarray:
    a = np.ascontiguousarray(a)
    if a.dtype != np.dtype(dtype):
        raise TypeError(f"expected {np.dtype(dtype)}, got {a.dtype}")
    return a


def _p(a):
    return None if a is None else a.ctypes.data_as(ctypes.c_void_p)


def num_threads() -> int:
    return int(_load().pqo_num_threads())


def half_to_float(bits: int) -> float:
    return float(_load().pqo_half_to_float(int(bits) & 0xFFFF))


def double_to_half_bits(v: float) -> int:
    return int(_load().pqo_double_to_half_rne(float(v)))


def float_to_half_bits(v: float) -> int:
    return int(_load().pqo_float_to_half_rne(float(np.float32(v))))


def quantize_act(x: np.ndarray):
    """x f16 [M,K] -> (q int8 [M,K], s_tok f32 [M]).  Eq. 1-2, n = 8, per token."""
    x = _c(x, np.float16)
    M, K = x.shape
    q = np.empty((M, K), np.int8)
    s = np.empty((M,), np.float32)
    _check(_load().pqo_quantize_act(_p(x), M, K, _p(q), _p(s)), "quantize_act")
    return q, s


def pack_w8(w: np.ndarray):
    """w f16 [N,K] -> (wq int8 [N,K], s_ch f32 [N]).  Eq. 2, n = 8, per output channel."""
    w = _c(w, np.float16)
    N, K = w.shape
    wq = np.empty((N, K), np.int8)
    s = np.empty((N,), np.float32)
    _check(_load().pqo_pack_w8(_p(w), N, K, _p(wq), _p(s)), "pack_w8")
    return wq, s


def pack_w4(w: np.ndarray, group: int = 128):
    """w f16 [N,K] -> (codes int8 [N,K] in [-8,7], s_grp f16 [N,K/group]).  Eq. 2, n = 4."""
    w = _c(w, np.float16)
    N, K = w.shape
    if K % group:
        raise OracleError("pack_w4: K must be a multiple of the group size")
    codes = np.empty((N, K), np.int8)
    s = np.empty((N, K // group), np.float16)
    _check(_load().pqo_pack_w4(_p(w), N, K, group, _p(codes), _p(s)), "pack_w4")
    return codes, s


def nibble_pack(codes: np.ndarray) -> np.ndarray:
    codes = _c(codes, np.int8)
    N, K = codes.shape
    out = np.empty((N, K // 2), np.uint8)
    _check(_load().pqo_nibble_pack(_p(codes), N, K, _p(out)), "nibble_pack")
    return out


def nibble_unpack(b: np.ndarray) -> np.ndarray:
    b = _c(b, np.uint8)
    N, K2 = b.shape
    out = np.empty((N, 2 * K2), np.int8)
    _check(_load().pqo_nibble_unpack(_p(b), N, 2 * K2, _p(out)), "nibble_unpack")
    return out


def gemm_w8a8(q, s_tok, wq, s_ch, want_acc: bool = True, want_y: bool = True):
    """-> (acc int32 [M,N] or None, y f16 [M,N] or None)."""
    q, wq = _c(q, np.int8), _c(wq, np.int8)
    s_tok, s_ch = _c(s_tok, np.float32), _c(s_ch, np.float32)
    M, K = q.shape
    N, K2 = wq.shape
    if K != K2 or s_tok.shape != (M,) or s_ch.shape != (N,):
        raise OracleError("gemm_w8a8: shape mismatch")
    acc = np.empty((M, N), np.int32) if want_acc else None
    y = np.empty((M, N), np.float16) if want_y else None
    _check(_load().pqo_gemm_w8a8(_p(q), _p(s_tok), _p(wq), _p(s_ch), M, N, K, _p(acc), _p(y)),
           "gemm_w8a8")
    return acc, y


def gemm_w4a8(q, s_tok, codes, s_grp, group: int = 128, want_acc: bool = True, want_y: bool = True):
    """-> (acc_g int32 [M,N,K/group] or None, y f16 [M,N] or None)."""
    q, codes = _c(q, np.int8), _c(codes, np.int8)
    s_tok, s_grp = _c(s_tok, np.float32), _c(s_grp, np.float16)
    M, K = q.shape
    N, K2 = codes.shape
    if K != K2 or K % group or s_tok.shape != (M,) or s_grp.shape != (N, K // group):
        raise OracleError("gemm_w4a8: shape mismatch")
    acc = np.empty((M, N, K // group), np.int32) if want_acc else None
    y = np.empty((M, N), np.float16) if want_y else None
    _check(_load().pqo_gemm_w4a8(_p(q), _p(s_tok), _p(codes), _p(s_grp), group, M, N, K,
                                 _p(acc), _p(y)), "gemm_w4a8")
    return acc, y
