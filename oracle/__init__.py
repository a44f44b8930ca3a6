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
        lib.pqo_quantize_act_smooth.argtypes = [vp, vp, i64, i64, vp, vp]
        lib.pqo_pack_w8_smooth.argtypes = [vp, vp, i64, i64, vp, vp]
        lib.pqo_pack_w4_smooth.argtypes = [vp, vp, i64, i64, i64, vp, vp]
        lib.pqo_quantize_act_static.argtypes = [vp, ctypes.c_float, i64, i64, vp, vp]
        lib.pqo_quantize_act_static_channel.argtypes = [vp, vp, i64, i64, vp, vp]
        lib.pqo_col_absmax.argtypes = [vp, i64, i64, vp]
        lib.pqo_hadamard_block.restype = i64
        lib.pqo_hadamard_block.argtypes = [i64]
        lib.pqo_rotate_rows.argtypes = [vp, i64, i64, vp]
        lib.pqo_quantize_act_hadamard.argtypes = [vp, i64, i64, vp, vp]
        lib.pqo_pack_w8_hadamard.argtypes = [vp, i64, i64, vp, vp]
        lib.pqo_pack_w4_hadamard.argtypes = [vp, i64, i64, i64, vp, vp]
        lib.pqo_smooth_scales.argtypes = [vp, vp, i64, vp, vp]
        lib.pqo_smooth_scales_alpha.argtypes = [vp, vp, i64, ctypes.c_int, vp, vp]
        lib.pqo_swiglu_quantize.argtypes = [vp, vp, i64, i64, vp, vp, vp]
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


def _col(col, K: int):
    col = _c(col, np.float32)
    if col.shape != (K,):
        raise OracleError("column factors must have shape [K]")
    return col


def quantize_act(x: np.ndarray, s_inv: np.ndarray | None = None):
    """x f16 [M,K] -> (q int8 [M,K], s_tok f32 [M]).  Eq. 1-2, n = 8, per token.
    With s_inv f32 [K]: quantizes X S^-1 (Eq. 3)."""
    x = _c(x, np.float16)
    M, K = x.shape
    q = np.empty((M, K), np.int8)
    s = np.empty((M,), np.float32)
    if s_inv is None:
        _check(_load().pqo_quantize_act(_p(x), M, K, _p(q), _p(s)), "quantize_act")
    else:
        s_inv = _col(s_inv, K)
        _check(_load().pqo_quantize_act_smooth(_p(x), _p(s_inv), M, K, _p(q), _p(s)), "quantize_act_smooth")
    return q, s


def quantize_act_static(x: np.ndarray, scale: float):
    """INT8 codes of x against ONE calibrated scale (static quantization): (q int8 [M,K], s_tok f32 [M] = scale)."""
    x = _c(x, np.float16)
    M, K = x.shape
    q = np.empty((M, K), np.int8)
    s = np.empty((M,), np.float32)
    _check(_load().pqo_quantize_act_static(_p(x), float(np.float32(scale)), M, K, _p(q), _p(s)), "quantize_act_static")
    return q, s


def quantize_act_static_channel(x: np.ndarray, inv_s: np.ndarray):
    """INT8 codes of x against one calibrated scale PER FEATURE CHANNEL, given as reciprocals inv_s f32 [K]:
    (q int8 [M,K], s_tok f32 [M] = 1; the channel scales are the caller's to fold into the weights)."""
    x = _c(x, np.float16)
    M, K = x.shape
    inv_s = _col(inv_s, K)
    q = np.empty((M, K), np.int8)
    s = np.empty((M,), np.float32)
    _check(_load().pqo_quantize_act_static_channel(_p(x), _p(inv_s), M, K, _p(q), _p(s)), "quantize_act_static_channel")
    return q, s


def hadamard_block(K: int) -> int:
    """Order B of the Hadamard blocks used for rows of length K (Eq. 4): largest power of two dividing K, <= 256."""
    return int(_load().pqo_hadamard_block(int(K)))


def rotate_rows(a: np.ndarray) -> np.ndarray:
    """a f16 [R,K] -> a H in binary32 [R,K], H = I (x) H_B / sqrt(B) (Eq. 4)."""
    a = _c(a, np.float16)
    R, K = a.shape
    out = np.empty((R, K), np.float32)
    _check(_load().pqo_rotate_rows(_p(a), R, K, _p(out)), "rotate_rows")
    return out


def quantize_act_hadamard(x: np.ndarray):
    """Per-token INT8 quantization of X H (Eq. 4): x f16 [M,K] -> (q int8 [M,K], s_tok f32 [M])."""
    x = _c(x, np.float16)
    M, K = x.shape
    q = np.empty((M, K), np.int8)
    s = np.empty((M,), np.float32)
    _check(_load().pqo_quantize_act_hadamard(_p(x), M, K, _p(q), _p(s)), "quantize_act_hadamard")
    return q, s


def pack_w8_hadamard(w: np.ndarray):
    """Per-channel INT8 quantization of W H (rows of W rotated, Eq. 4)."""
    w = _c(w, np.float16)
    N, K = w.shape
    wq = np.empty((N, K), np.int8)
    s = np.empty((N,), np.float32)
    _check(_load().pqo_pack_w8_hadamard(_p(w), N, K, _p(wq), _p(s)), "pack_w8_hadamard")
    return wq, s


def pack_w4_hadamard(w: np.ndarray, group: int = 128):
    """Group-wise INT4 quantization of W H (Eq. 4): (codes int8 [N,K], s_grp f16 [N,K/group])."""
    w = _c(w, np.float16)
    N, K = w.shape
    if K % group:
        raise OracleError("pack_w4_hadamard: K must be a multiple of the group size")
    codes = np.empty((N, K), np.int8)
    s = np.empty((N, K // group), np.float16)
    _check(_load().pqo_pack_w4_hadamard(_p(w), N, K, group, _p(codes), _p(s)), "pack_w4_hadamard")
    return codes, s


def swiglu_quantize(gate: np.ndarray, up: np.ndarray, want_h: bool = False):
    """gate, up f16 [M,I] -> (q int8 [M,I], s_tok f32 [M]) of h = silu(gate) * up (binary32), quantized per
    token by Eq. 1-2; with want_h also h f32 [M,I] as a third result."""
    gate, up = _c(gate, np.float16), _c(up, np.float16)
    if gate.shape != up.shape or gate.ndim != 2:
        raise OracleError("swiglu_quantize: gate and up must be [M,I]")
    M, I = gate.shape
    q = np.empty((M, I), np.int8)
    s = np.empty((M,), np.float32)
    h = np.empty((M, I), np.float32) if want_h else None
    _check(_load().pqo_swiglu_quantize(_p(gate), _p(up), M, I, _p(h), _p(q), _p(s)), "swiglu_quantize")
    return (q, s, h) if want_h else (q, s)


def col_absmax(a: np.ndarray) -> np.ndarray:
    """a f16 [R,K] -> f32 [K]: max over rows of |a[r,k]| (calibration statistic of Eq. 3)."""
    a = _c(a, np.float16)
    R, K = a.shape
    out = np.empty((K,), np.float32)
    _check(_load().pqo_col_absmax(_p(a), R, K, _p(out)), "col_absmax")
    return out


def smooth_scales(x_absmax: np.ndarray, w_absmax: np.ndarray):
    """Eq. 3 with alpha = 0.5: (s, s_inv) f32 [K] from the column maxima of X and W."""
    xa, wa = _c(x_absmax, np.float32), _c(w_absmax, np.float32)
    if xa.shape != wa.shape or xa.ndim != 1:
        raise OracleError("smooth_scales: two vectors of the same length")
    s, s_inv = np.empty_like(xa), np.empty_like(xa)
    _check(_load().pqo_smooth_scales(_p(xa), _p(wa), xa.shape[0], _p(s), _p(s_inv)), "smooth_scales")
    return s, s_inv


def smooth_scales_alpha(x_absmax: np.ndarray, w_absmax: np.ndarray, alpha_quarters: int):
    """Eq. 3 with alpha = alpha_quarters / 4 (0 ... 4): (s, s_inv) f32 [K]."""
    xa, wa = _c(x_absmax, np.float32), _c(w_absmax, np.float32)
    if xa.shape != wa.shape or xa.ndim != 1:
        raise OracleError("smooth_scales_alpha: two vectors of the same length")
    s, s_inv = np.empty_like(xa), np.empty_like(xa)
    _check(_load().pqo_smooth_scales_alpha(_p(xa), _p(wa), xa.shape[0], int(alpha_quarters), _p(s), _p(s_inv)),
           "smooth_scales_alpha")
    return s, s_inv


def pack_w8(w: np.ndarray, smooth: np.ndarray | None = None):
    """w f16 [N,K] -> (wq int8 [N,K], s_ch f32 [N]).  Eq. 2, n = 8, per output channel.
    With smooth f32 [K]: quantizes S W (Eq. 3)."""
    w = _c(w, np.float16)
    N, K = w.shape
    wq = np.empty((N, K), np.int8)
    s = np.empty((N,), np.float32)
    if smooth is None:
        _check(_load().pqo_pack_w8(_p(w), N, K, _p(wq), _p(s)), "pack_w8")
    else:
        smooth = _col(smooth, K)
        _check(_load().pqo_pack_w8_smooth(_p(w), _p(smooth), N, K, _p(wq), _p(s)), "pack_w8_smooth")
    return wq, s


def pack_w4(w: np.ndarray, group: int = 128, smooth: np.ndarray | None = None):
    """w f16 [N,K] -> (codes int8 [N,K] in [-8,7], s_grp f16 [N,K/group]).  Eq. 2, n = 4.
    With smooth f32 [K]: quantizes S W (Eq. 3)."""
    w = _c(w, np.float16)
    N, K = w.shape
    if K % group:
        raise OracleError("pack_w4: K must be a multiple of the group size")
    codes = np.empty((N, K), np.int8)
    s = np.empty((N, K // group), np.float16)
    if smooth is None:
        _check(_load().pqo_pack_w4(_p(w), N, K, group, _p(codes), _p(s)), "pack_w4")
    else:
        smooth = _col(smooth, K)
        _check(_load().pqo_pack_w4_smooth(_p(w), _p(smooth), N, K, group, _p(codes), _p(s)), "pack_w4_smooth")
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
