"""ctypes binding of libpq.so.  Marshals torch CUDA tensors (device pointers, sizes, the current
stream) into the C calls of ``include/pq.h``; every step of the computation runs in the library's
kernels.  torch is used for device memory and streams only."""
from __future__ import annotations

import ctypes
import os

import torch

from . import build as _build

GROUP = 128

_lib = None

_i64, _i32, _vp = ctypes.c_int64, ctypes.c_int32, ctypes.c_void_p

# name -> (restype, argtypes); mirrors include/pq.h
SIGNATURES = {
    "pq_status_str": (ctypes.c_char_p, [ctypes.c_int]),
    "pq_packed_w8_bytes": (ctypes.c_size_t, [_i64, _i64]),
    "pq_packed_w4_bytes": (ctypes.c_size_t, [_i64, _i64]),
    "pq_quantize_act": (ctypes.c_int, [_vp, _i64, _i64, _vp, _vp, _vp]),
    "pq_pack_w8": (ctypes.c_int, [_vp, _i64, _i64, _vp, _vp, _vp]),
    "pq_pack_w4": (ctypes.c_int, [_vp, _i64, _i64, _i32, _vp, _vp, _vp]),
    "pq_unpack_w8": (ctypes.c_int, [_vp, _i64, _i64, _vp, _vp]),
    "pq_unpack_w4": (ctypes.c_int, [_vp, _i64, _i64, _vp, _vp]),
    "pq_gemm_w8a8": (ctypes.c_int, [_vp, _vp, _vp, _vp, _i64, _i64, _i64, _vp, _vp]),
    "pq_gemm_w4a8": (ctypes.c_int, [_vp, _vp, _vp, _vp, _i32, _i64, _i64, _i64, _vp, _vp]),
    "pq_acc_w8a8": (ctypes.c_int, [_vp, _vp, _i64, _i64, _i64, _vp, _vp]),
    "pq_acc_w4a8": (ctypes.c_int, [_vp, _vp, _i32, _i64, _i64, _i64, _vp, _vp]),
    "pq_device_status": (ctypes.c_int, [ctypes.POINTER(ctypes.c_int)]),
    "pq_set_workspace": (ctypes.c_int, [_vp, ctypes.c_size_t, _vp]),
    "pq_plan_w8a8": (ctypes.c_int, [_i64, _i64, _i64, _i32, ctypes.c_size_t, ctypes.POINTER(_i32), ctypes.POINTER(_i32)]),
    "pq_gemm_w8a8_noalloc": (ctypes.c_int, [_vp, _vp, _vp, _vp, _i64, _i64, _i64, _vp, _vp]),
    "pq_gemm_w8a8_group": (ctypes.c_int, [_vp, _vp, _i32, ctypes.POINTER(_vp), ctypes.POINTER(_vp),
                                          ctypes.POINTER(_i64), ctypes.POINTER(_vp), _i64, _i64, _vp]),
    "pq_quantize_act_static": (ctypes.c_int, [_vp, _vp, _i64, _i64, _vp, _vp, _vp]),
    "pq_hadamard_block": (_i32, [_i64]),
    "pq_quantize_act_hadamard": (ctypes.c_int, [_vp, _i64, _i64, _vp, _vp, _vp]),
    "pq_pack_w8_hadamard": (ctypes.c_int, [_vp, _i64, _i64, _vp, _vp, _vp]),
    "pq_pack_w4_hadamard": (ctypes.c_int, [_vp, _i64, _i64, _i32, _vp, _vp, _vp]),
    "pq_col_absmax": (ctypes.c_int, [_vp, _i64, _i64, _vp, _vp]),
    "pq_smooth_scales": (ctypes.c_int, [_vp, _vp, _i64, _vp, _vp, _vp]),
    "pq_quantize_act_smooth": (ctypes.c_int, [_vp, _vp, _i64, _i64, _vp, _vp, _vp]),
    "pq_pack_w8_smooth": (ctypes.c_int, [_vp, _vp, _i64, _i64, _vp, _vp, _vp]),
    "pq_pack_w4_smooth": (ctypes.c_int, [_vp, _vp, _i64, _i64, _i32, _vp, _vp, _vp]),
    "pq_gemm_w4a8_group": (ctypes.c_int, [_vp, _vp, _i32, ctypes.POINTER(_vp), ctypes.POINTER(_vp), _i32,
                                          ctypes.POINTER(_i64), ctypes.POINTER(_vp), _i64, _i64, _vp]),
}
MAX_GROUP = 4


class PQError(RuntimeError):
    def __init__(self, call: str, status: int):
        self.status = status
        msg = lib().pq_status_str(status).decode() if _lib is not None else "?"
        super().__init__(f"{call} failed: status {status} ({msg})")


def lib() -> ctypes.CDLL:
    """Load (building first if missing or stale) libpq.so.  Raises if that is impossible."""
    global _lib
    if _lib is None:
        path = _build.LIB
        if _build.stale():
            path = _build.build()
        if not os.path.exists(path):
            raise RuntimeError(f"CUDA library {path} is missing and could not be built")
        handle = ctypes.CDLL(path)
        for name, (res, args) in SIGNATURES.items():
            fn = getattr(handle, name)  # AttributeError if the library lacks a declared symbol
            fn.restype, fn.argtypes = res, args
        _lib = handle
    return _lib


def _stream() -> int:
    return torch.cuda.current_stream().cuda_stream


def _dev(t: torch.Tensor, dtype: torch.dtype, what: str) -> torch.Tensor:
    if not t.is_cuda:
        raise ValueError(f"{what}: expected a CUDA tensor (this library has no CPU path)")
    if t.dtype != dtype:
        raise TypeError(f"{what}: expected {dtype}, got {t.dtype}")
    if not t.is_contiguous():
        raise ValueError(f"{what}: expected a contiguous tensor")
    return t


def _check(call: str, status: int) -> None:
    if status != 0:
        raise PQError(call, status)


def _factors(v: torch.Tensor, K: int, name: str) -> torch.Tensor:
    v = _dev(v, torch.float32, name)
    if tuple(v.shape) != (K,):
        raise ValueError(f"{name}: expected shape [{K}]")
    return v


def pq_quantize_act(x: torch.Tensor, q: torch.Tensor | None = None, s_tok: torch.Tensor | None = None):
    """x f16 [M,K] -> (q int8 [M,K], s_tok f32 [M])."""
    x = _dev(x, torch.float16, "x")
    M, K = x.shape
    if q is None:
        q = torch.empty((M, K), dtype=torch.int8, device=x.device)
    if s_tok is None:
        s_tok = torch.empty((M,), dtype=torch.float32, device=x.device)
    _check("pq_quantize_act", lib().pq_quantize_act(x.data_ptr(), M, K, q.data_ptr(), s_tok.data_ptr(), _stream()))
    return q, s_tok


def pq_quantize_act_smooth(x: torch.Tensor, s_inv: torch.Tensor, q: torch.Tensor | None = None,
                           s_tok: torch.Tensor | None = None):
    """Quantizes X S^-1 (Eq. 3): x f16 [M,K], s_inv f32 [K] -> (q int8 [M,K], s_tok f32 [M])."""
    x = _dev(x, torch.float16, "x")
    M, K = x.shape
    s_inv = _factors(s_inv, K, "s_inv")
    if q is None:
        q = torch.empty((M, K), dtype=torch.int8, device=x.device)
    if s_tok is None:
        s_tok = torch.empty((M,), dtype=torch.float32, device=x.device)
    _check("pq_quantize_act_smooth", lib().pq_quantize_act_smooth(x.data_ptr(), s_inv.data_ptr(), M, K, q.data_ptr(),
                                                                  s_tok.data_ptr(), _stream()))
    return q, s_tok


def pq_quantize_act_static(x: torch.Tensor, scale: torch.Tensor, q: torch.Tensor | None = None,
                           s_tok: torch.Tensor | None = None):
    """INT8 codes against one calibrated scale: x f16 [M,K], scale f32 device tensor with one element
    -> (q int8 [M,K], s_tok f32 [M] filled with the scale)."""
    x = _dev(x, torch.float16, "x")
    M, K = x.shape
    scale = _dev(scale, torch.float32, "scale")
    if scale.numel() != 1:
        raise ValueError("scale: one element")
    if q is None:
        q = torch.empty((M, K), dtype=torch.int8, device=x.device)
    if s_tok is None:
        s_tok = torch.empty((M,), dtype=torch.float32, device=x.device)
    _check("pq_quantize_act_static", lib().pq_quantize_act_static(x.data_ptr(), scale.data_ptr(), M, K, q.data_ptr(),
                                                                  s_tok.data_ptr(), _stream()))
    return q, s_tok


def pq_hadamard_block(K: int) -> int:
    """Order of the Hadamard blocks the Eq. 4 calls use for rows of length K (host-only query)."""
    return int(lib().pq_hadamard_block(int(K)))


def pq_quantize_act_hadamard(x: torch.Tensor, q: torch.Tensor | None = None, s_tok: torch.Tensor | None = None):
    """Quantizes X H (Eq. 4): x f16 [M,K] -> (q int8 [M,K], s_tok f32 [M])."""
    x = _dev(x, torch.float16, "x")
    M, K = x.shape
    if q is None:
        q = torch.empty((M, K), dtype=torch.int8, device=x.device)
    if s_tok is None:
        s_tok = torch.empty((M,), dtype=torch.float32, device=x.device)
    _check("pq_quantize_act_hadamard", lib().pq_quantize_act_hadamard(x.data_ptr(), M, K, q.data_ptr(),
                                                                      s_tok.data_ptr(), _stream()))
    return q, s_tok


def pq_pack_w8_hadamard(w: torch.Tensor):
    """Packs W H (Eq. 4): w f16 [N,K] -> (wq opaque uint8 buffer, s_ch f32 [N])."""
    w = _dev(w, torch.float16, "w")
    N, K = w.shape
    wq = torch.empty((lib().pq_packed_w8_bytes(N, K),), dtype=torch.uint8, device=w.device)
    s_ch = torch.empty((N,), dtype=torch.float32, device=w.device)
    _check("pq_pack_w8_hadamard", lib().pq_pack_w8_hadamard(w.data_ptr(), N, K, wq.data_ptr(), s_ch.data_ptr(), _stream()))
    return wq, s_ch


def pq_pack_w4_hadamard(w: torch.Tensor, group: int = GROUP):
    """Packs W H (Eq. 4): w f16 [N,K] -> (wp opaque uint8 buffer, s_grp f16 [K/group, N])."""
    w = _dev(w, torch.float16, "w")
    N, K = w.shape
    wp = torch.empty((lib().pq_packed_w4_bytes(N, K),), dtype=torch.uint8, device=w.device)
    s_grp = torch.empty((max(K // max(group, 1), 1), N), dtype=torch.float16, device=w.device)
    _check("pq_pack_w4_hadamard", lib().pq_pack_w4_hadamard(w.data_ptr(), N, K, group, wp.data_ptr(), s_grp.data_ptr(),
                                                            _stream()))
    return wp, s_grp


def pq_col_absmax(a: torch.Tensor) -> torch.Tensor:
    """a f16 [R,K] -> f32 [K]: column maxima of |a| (calibration statistic of Eq. 3)."""
    a = _dev(a, torch.float16, "a")
    R, K = a.shape
    out = torch.empty((K,), dtype=torch.float32, device=a.device)
    _check("pq_col_absmax", lib().pq_col_absmax(a.data_ptr(), R, K, out.data_ptr(), _stream()))
    return out


def pq_smooth_scales(x_absmax: torch.Tensor, w_absmax: torch.Tensor):
    """Eq. 3 with alpha = 0.5: (s, s_inv) f32 [K] from the column maxima of X and of W."""
    xa = _dev(x_absmax, torch.float32, "x_absmax")
    wa = _factors(w_absmax, xa.shape[0], "w_absmax")
    s, s_inv = torch.empty_like(xa), torch.empty_like(xa)
    _check("pq_smooth_scales", lib().pq_smooth_scales(xa.data_ptr(), wa.data_ptr(), xa.shape[0], s.data_ptr(),
                                                      s_inv.data_ptr(), _stream()))
    return s, s_inv


def pq_pack_w8(w: torch.Tensor, smooth: torch.Tensor | None = None):
    """w f16 [N,K] -> (wq opaque uint8 buffer, s_ch f32 [N]).  With smooth f32 [K]: packs S W (Eq. 3)."""
    w = _dev(w, torch.float16, "w")
    N, K = w.shape
    wq = torch.empty((lib().pq_packed_w8_bytes(N, K),), dtype=torch.uint8, device=w.device)
    s_ch = torch.empty((N,), dtype=torch.float32, device=w.device)
    if smooth is None:
        _check("pq_pack_w8", lib().pq_pack_w8(w.data_ptr(), N, K, wq.data_ptr(), s_ch.data_ptr(), _stream()))
    else:
        smooth = _factors(smooth, K, "smooth")
        _check("pq_pack_w8_smooth", lib().pq_pack_w8_smooth(w.data_ptr(), smooth.data_ptr(), N, K, wq.data_ptr(),
                                                            s_ch.data_ptr(), _stream()))
    return wq, s_ch


def pq_pack_w4(w: torch.Tensor, group: int = GROUP, smooth: torch.Tensor | None = None):
    """w f16 [N,K] -> (wp opaque uint8 buffer, s_grp f16 [K/group, N]).  With smooth f32 [K]: packs S W (Eq. 3)."""
    w = _dev(w, torch.float16, "w")
    N, K = w.shape
    wp = torch.empty((lib().pq_packed_w4_bytes(N, K),), dtype=torch.uint8, device=w.device)
    s_grp = torch.empty((max(K // max(group, 1), 1), N), dtype=torch.float16, device=w.device)
    if smooth is None:
        _check("pq_pack_w4", lib().pq_pack_w4(w.data_ptr(), N, K, group, wp.data_ptr(), s_grp.data_ptr(), _stream()))
    else:
        smooth = _factors(smooth, K, "smooth")
        _check("pq_pack_w4_smooth", lib().pq_pack_w4_smooth(w.data_ptr(), smooth.data_ptr(), N, K, group, wp.data_ptr(),
                                                            s_grp.data_ptr(), _stream()))
    return wp, s_grp


def pq_unpack_w8(wq: torch.Tensor, N: int, K: int) -> torch.Tensor:
    wq = _dev(wq, torch.uint8, "wq")
    codes = torch.empty((N, K), dtype=torch.int8, device=wq.device)
    _check("pq_unpack_w8", lib().pq_unpack_w8(wq.data_ptr(), N, K, codes.data_ptr(), _stream()))
    return codes


def pq_unpack_w4(wp: torch.Tensor, N: int, K: int) -> torch.Tensor:
    wp = _dev(wp, torch.uint8, "wp")
    codes = torch.empty((N, K), dtype=torch.int8, device=wp.device)
    _check("pq_unpack_w4", lib().pq_unpack_w4(wp.data_ptr(), N, K, codes.data_ptr(), _stream()))
    return codes


def pq_plan_w8a8(M: int, N: int, K: int, sms: int = 148, scratch_bytes: int = 0) -> tuple[int, int]:
    """(tile width, number of K parts) the W8A8 GEMM would choose; host-only, needs no GPU."""
    bn, sp = _i32(0), _i32(0)
    _check("pq_plan_w8a8", lib().pq_plan_w8a8(M, N, K, sms, scratch_bytes, ctypes.byref(bn), ctypes.byref(sp)))
    return int(bn.value), int(sp.value)


_workspaces: dict[int, torch.Tensor] = {}
WORKSPACE_BYTES = int(os.environ.get("PQ_WORKSPACE_MB", "64")) << 20


def pq_set_workspace(workspace: torch.Tensor | None) -> None:
    """Registers (or, with None, unregisters) scratch memory for the current device: a uint8 CUDA
    tensor the caller keeps alive.  The W8A8 GEMM uses it to split K on shapes with few tiles."""
    if workspace is None:
        _check("pq_set_workspace", lib().pq_set_workspace(None, 0, _stream()))
        return
    workspace = _dev(workspace, torch.uint8, "workspace")
    _check("pq_set_workspace", lib().pq_set_workspace(workspace.data_ptr(), workspace.numel(), _stream()))


def _ensure_workspace(device: torch.device) -> None:
    """Gives each device one scratch buffer on first use (torch owns the memory; the library never
    allocates).  PQ_WORKSPACE_MB=0 turns this off."""
    idx = device.index if device.index is not None else torch.cuda.current_device()
    if idx in _workspaces or WORKSPACE_BYTES <= 0:
        return
    with torch.cuda.device(idx):
        buf = torch.empty((WORKSPACE_BYTES,), dtype=torch.uint8, device=device)
        pq_set_workspace(buf)
    _workspaces[idx] = buf


def pq_gemm_w8a8(q, s_tok, wq, s_ch, N: int, y: torch.Tensor | None = None) -> torch.Tensor:
    """q int8 [M,K], s_tok f32 [M], wq/s_ch from pq_pack_w8 -> y f16 [M,N]."""
    q = _dev(q, torch.int8, "q")
    _ensure_workspace(q.device)
    M, K = q.shape
    _dev(s_tok, torch.float32, "s_tok"), _dev(wq, torch.uint8, "wq"), _dev(s_ch, torch.float32, "s_ch")
    if y is None:
        y = torch.empty((M, N), dtype=torch.float16, device=q.device)
    _check("pq_gemm_w8a8", lib().pq_gemm_w8a8(q.data_ptr(), s_tok.data_ptr(), wq.data_ptr(), s_ch.data_ptr(),
                                              M, N, K, y.data_ptr(), _stream()))
    return y


def pq_gemm_w8a8_group(q, s_tok, members, ys=None) -> list[torch.Tensor]:
    """Several W8A8 linears over the same quantized tokens as one call (one kernel launch).  members: sequence of (wq, s_ch, N) from pq_pack_w8; ys: optional outputs f16 [M,N_g].
    Returns the outputs; each equals pq_gemm_w8a8(q, s_tok, wq, s_ch, N) bit for bit."""
    q = _dev(q, torch.int8, "q")
    _ensure_workspace(q.device)
    M, K = q.shape
    _dev(s_tok, torch.float32, "s_tok")
    n = len(members)
    if ys is None:
        ys = [torch.empty((M, int(N)), dtype=torch.float16, device=q.device) for (_, _, N) in members]
    if len(ys) != n:
        raise ValueError("one output per member")
    for (wq, s_ch, _), y in zip(members, ys):
        _dev(wq, torch.uint8, "wq"), _dev(s_ch, torch.float32, "s_ch"), _dev(y, torch.float16, "y")
    wq_arr = (_vp * max(n, 1))(*[m[0].data_ptr() for m in members])
    sc_arr = (_vp * max(n, 1))(*[m[1].data_ptr() for m in members])
    n_arr = (_i64 * max(n, 1))(*[int(m[2]) for m in members])
    y_arr = (_vp * max(n, 1))(*[y.data_ptr() for y in ys])
    _check("pq_gemm_w8a8_group", lib().pq_gemm_w8a8_group(q.data_ptr(), s_tok.data_ptr(), n, wq_arr, sc_arr, n_arr,
                                                          y_arr, M, K, _stream()))
    return list(ys)


def pq_gemm_w4a8_group(q, s_tok, members, ys=None, group: int = GROUP) -> list[torch.Tensor]:
    """Several W4A8 linears over the same quantized tokens as one call (one kernel launch).  members: sequence of (wp, s_grp, N) from pq_pack_w4; ys: optional outputs f16 [M,N_g].
    Each output equals pq_gemm_w4a8(q, s_tok, wp, s_grp, N) bit for bit."""
    q = _dev(q, torch.int8, "q")
    M, K = q.shape
    _dev(s_tok, torch.float32, "s_tok")
    n = len(members)
    if ys is None:
        ys = [torch.empty((M, int(N)), dtype=torch.float16, device=q.device) for (_, _, N) in members]
    if len(ys) != n:
        raise ValueError("one output per member")
    for (wp, s_grp, _), y in zip(members, ys):
        _dev(wp, torch.uint8, "wp"), _dev(s_grp, torch.float16, "s_grp"), _dev(y, torch.float16, "y")
    wp_arr = (_vp * max(n, 1))(*[m[0].data_ptr() for m in members])
    sg_arr = (_vp * max(n, 1))(*[m[1].data_ptr() for m in members])
    n_arr = (_i64 * max(n, 1))(*[int(m[2]) for m in members])
    y_arr = (_vp * max(n, 1))(*[y.data_ptr() for y in ys])
    _check("pq_gemm_w4a8_group", lib().pq_gemm_w4a8_group(q.data_ptr(), s_tok.data_ptr(), n, wp_arr, sg_arr, group,
                                                          n_arr, y_arr, M, K, _stream()))
    return list(ys)


def pq_gemm_w8a8_noalloc(q, s_tok, wq, s_ch, N: int, y: torch.Tensor) -> torch.Tensor:
    """Same product as pq_gemm_w8a8, for callers that may not allocate: the output tensor is
    required (this wrapper creates none) and the library's built-in scratch array is used instead of
    a registered workspace.  Raises PQError with status 7 when the padded output exceeds 2 Mi
    elements.  Calls on one device must not overlap on the GPU."""
    q = _dev(q, torch.int8, "q")
    M, K = q.shape
    _dev(s_tok, torch.float32, "s_tok"), _dev(wq, torch.uint8, "wq"), _dev(s_ch, torch.float32, "s_ch")
    _dev(y, torch.float16, "y")
    _check("pq_gemm_w8a8_noalloc", lib().pq_gemm_w8a8_noalloc(q.data_ptr(), s_tok.data_ptr(), wq.data_ptr(),
                                                              s_ch.data_ptr(), M, N, K, y.data_ptr(), _stream()))
    return y


def pq_gemm_w4a8(q, s_tok, wp, s_grp, N: int, group: int = GROUP, y: torch.Tensor | None = None) -> torch.Tensor:
    """q int8 [M,K], s_tok f32 [M], wp/s_grp from pq_pack_w4 -> y f16 [M,N]."""
    q = _dev(q, torch.int8, "q")
    M, K = q.shape
    _dev(s_tok, torch.float32, "s_tok"), _dev(wp, torch.uint8, "wp"), _dev(s_grp, torch.float16, "s_grp")
    if y is None:
        y = torch.empty((M, N), dtype=torch.float16, device=q.device)
    _check("pq_gemm_w4a8", lib().pq_gemm_w4a8(q.data_ptr(), s_tok.data_ptr(), wp.data_ptr(), s_grp.data_ptr(),
                                              group, M, N, K, y.data_ptr(), _stream()))
    return y


def pq_acc_w8a8(q, wq, N: int) -> torch.Tensor:
    """Exact INT32 accumulators [M,N] of the W8A8 product."""
    q = _dev(q, torch.int8, "q")
    M, K = q.shape
    _dev(wq, torch.uint8, "wq")
    acc = torch.empty((M, N), dtype=torch.int32, device=q.device)
    _check("pq_acc_w8a8", lib().pq_acc_w8a8(q.data_ptr(), wq.data_ptr(), M, N, K, acc.data_ptr(), _stream()))
    return acc


def pq_acc_w4a8(q, wp, N: int, group: int = GROUP) -> torch.Tensor:
    """Exact INT32 per-group accumulators [K/group, M, N] of the W4A8 product."""
    q = _dev(q, torch.int8, "q")
    M, K = q.shape
    _dev(wp, torch.uint8, "wp")
    acc = torch.empty((K // group, M, N), dtype=torch.int32, device=q.device)
    _check("pq_acc_w4a8", lib().pq_acc_w4a8(q.data_ptr(), wp.data_ptr(), group, M, N, K, acc.data_ptr(), _stream()))
    return acc


def pq_device_status() -> int:
    """Synchronizes; returns and clears the device status word (0 = ok, 6 = a bounded wait expired)."""
    v = ctypes.c_int(0)
    _check("pq_device_status", lib().pq_device_status(ctypes.byref(v)))
    return int(v.value)
