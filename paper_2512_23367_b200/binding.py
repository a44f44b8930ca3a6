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
    "pq_last_cuda_error": (ctypes.c_char_p, []),
    "pq_packed_w8_bytes": (ctypes.c_size_t, [_i64, _i64]),
    "pq_packed_w4_bytes": (ctypes.c_size_t, [_i64, _i64]),
    "pq_quantize_act": (ctypes.c_int, [_vp, _i64, _i64, _vp, _vp, _vp]),
    "pq_pack_w8": (ctypes.c_int, [_vp, _i64, _i64, _vp, _vp, _vp]),
    "pq_pack_w4": (ctypes.c_int, [_vp, _i64, _i64, _i32, _vp, _vp, _vp]),
    "pq_unpack_w8": (ctypes.c_int, [_vp, _i64, _i64, _vp, _vp]),
    "pq_unpack_w4": (ctypes.c_int, [_vp, _i64, _i64, _vp, _vp]),
    "pq_gemm_w8a8": (ctypes.c_int, [_vp, _vp, _vp, _vp, _i64, _i64, _i64, _vp, _vp, ctypes.c_size_t, _vp]),
    "pq_gemm_w4a8": (ctypes.c_int, [_vp, _vp, _vp, _vp, _i32, _i64, _i64, _i64, _vp, _vp]),
    "pq_acc_w8a8": (ctypes.c_int, [_vp, _vp, _i64, _i64, _i64, _vp, _vp]),
    "pq_acc_w4a8": (ctypes.c_int, [_vp, _vp, _i32, _i64, _i64, _i64, _vp, _vp]),
    "pq_device_status": (ctypes.c_int, [ctypes.POINTER(ctypes.c_int)]),
    "pq_workspace_bytes": (ctypes.c_size_t, [_i64, ctypes.POINTER(_i64), _i32, _i64, _i32]),
    "pq_workspace_init": (ctypes.c_int, [_vp, ctypes.c_size_t, _vp]),
    "pq_set_wait_limit": (ctypes.c_int, [ctypes.c_uint32]),
    "pq_plan_w8a8": (ctypes.c_int, [_i64, _i64, _i64, _i32, ctypes.c_size_t, ctypes.POINTER(_i32), ctypes.POINTER(_i32)]),
    "pq_gemm_w8a8_noalloc": (ctypes.c_int, [_vp, _vp, _vp, _vp, _i64, _i64, _i64, _vp, _vp]),
    "pq_gemm_w8a8_group": (ctypes.c_int, [_vp, _vp, _i32, ctypes.POINTER(_vp), ctypes.POINTER(_vp),
                                          ctypes.POINTER(_i64), ctypes.POINTER(_vp), _i64, _i64, _vp,
                                          ctypes.c_size_t, _vp]),
    "pq_quantize_act_static": (ctypes.c_int, [_vp, _vp, _i64, _i64, _vp, _vp, _vp]),
    "pq_swiglu_quantize": (ctypes.c_int, [_vp, _vp, _i64, _i64, _vp, _vp, _vp]),
    "pq_linear_w8a8": (ctypes.c_int, [_vp, _vp, _vp, _i64, _i64, _i64, _vp, _vp, _vp, _vp, ctypes.c_size_t, _vp]),
    "pq_linear_w4a8": (ctypes.c_int, [_vp, _vp, _vp, _i32, _i64, _i64, _i64, _vp, _vp, _vp, _vp]),
    "pq_quantize_act_static_channel": (ctypes.c_int, [_vp, _vp, _i64, _i64, _vp, _vp, _vp]),
    "pq_hadamard_block": (_i32, [_i64]),
    "pq_quantize_act_hadamard": (ctypes.c_int, [_vp, _i64, _i64, _vp, _vp, _vp]),
    "pq_pack_w8_hadamard": (ctypes.c_int, [_vp, _i64, _i64, _vp, _vp, _vp]),
    "pq_pack_w4_hadamard": (ctypes.c_int, [_vp, _i64, _i64, _i32, _vp, _vp, _vp]),
    "pq_col_absmax": (ctypes.c_int, [_vp, _i64, _i64, _vp, _vp]),
    "pq_smooth_scales": (ctypes.c_int, [_vp, _vp, _i64, _vp, _vp, _vp]),
    "pq_smooth_scales_alpha": (ctypes.c_int, [_vp, _vp, _i64, _i32, _vp, _vp, _vp]),
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
        if status == 5 and _lib is not None:
            msg += ": " + lib().pq_last_cuda_error().decode()
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


def _sized(t: torch.Tensor, dtype: torch.dtype, numel: int, what: str) -> torch.Tensor:
    """A contiguous tensor of `dtype` with exactly `numel` elements.  The C calls take raw pointers and trust
    the sizes they are given, so a short buffer would become an out-of-bounds device access: every operand is
    measured here, before anything is launched (and before the devices are looked at, so that a wrong size is
    reported as such wherever the tensor lives)."""
    if t.dtype != dtype:
        raise TypeError(f"{what}: expected {dtype}, got {t.dtype}")
    if t.numel() != int(numel):
        raise ValueError(f"{what}: expected {int(numel)} elements, got {t.numel()}")
    if not t.is_contiguous():
        raise ValueError(f"{what}: expected a contiguous tensor")
    return t


def _together(first: torch.Tensor, *others: torch.Tensor | None) -> None:
    """All operands of a call live on one CUDA device."""
    if not first.is_cuda:
        raise ValueError("expected CUDA tensors (this library has no CPU path)")
    for t in others:
        if t is not None and t.device != first.device:
            raise ValueError(f"operands on different devices: {t.device} and {first.device}")


def _tokens(q: torch.Tensor, s_tok: torch.Tensor) -> tuple[int, int]:
    """Measures the quantized tokens (q int8 [M,K], s_tok f32 [M]); returns (M, K)."""
    if q.dim() != 2:
        raise ValueError("q: expected a 2-D tensor [M,K]")
    M, K = q.shape
    _sized(q, torch.int8, M * K, "q")
    _sized(s_tok, torch.float32, M, "s_tok")
    return int(M), int(K)


def _out(y: torch.Tensor | None, M: int, N: int, like: torch.Tensor) -> torch.Tensor:
    if y is None:
        return torch.empty((M, N), dtype=torch.float16, device=like.device)
    return _sized(y, torch.float16, M * N, "y")


def _ws(workspace: torch.Tensor | None) -> tuple[int | None, int]:
    if workspace is None:
        return None, 0
    _sized(workspace, torch.uint8, workspace.numel(), "workspace")
    return workspace.data_ptr(), workspace.numel()


def _factors(v: torch.Tensor, K: int, name: str) -> torch.Tensor:
    """A per-column factor vector f32 [K] on the device."""
    return _dev(_sized(v, torch.float32, K, name), torch.float32, name)


def _rows(x: torch.Tensor, q: torch.Tensor | None, s_tok: torch.Tensor | None):
    """Outputs of a row quantizer for x f16 [M,K]: created when absent, measured when given."""
    if x.dim() != 2:
        raise ValueError("x: expected a 2-D tensor [M,K]")
    M, K = x.shape
    _sized(x, torch.float16, M * K, "x")
    if q is not None:
        _sized(q, torch.int8, M * K, "q")
    if s_tok is not None:
        _sized(s_tok, torch.float32, M, "s_tok")
    _together(x, q, s_tok)
    q = torch.empty((M, K), dtype=torch.int8, device=x.device) if q is None else q
    s_tok = torch.empty((M,), dtype=torch.float32, device=x.device) if s_tok is None else s_tok
    return int(M), int(K), q, s_tok


def pq_quantize_act(x: torch.Tensor, q: torch.Tensor | None = None, s_tok: torch.Tensor | None = None):
    """x f16 [M,K] -> (q int8 [M,K], s_tok f32 [M])."""
    M, K, q, s_tok = _rows(x, q, s_tok)
    _check("pq_quantize_act", lib().pq_quantize_act(x.data_ptr(), M, K, q.data_ptr(), s_tok.data_ptr(), _stream()))
    return q, s_tok


def pq_quantize_act_smooth(x: torch.Tensor, s_inv: torch.Tensor, q: torch.Tensor | None = None,
                           s_tok: torch.Tensor | None = None):
    """Quantizes X S^-1 (Eq. 3): x f16 [M,K], s_inv f32 [K] -> (q int8 [M,K], s_tok f32 [M])."""
    M, K, q, s_tok = _rows(x, q, s_tok)
    s_inv = _factors(s_inv, K, "s_inv")
    _check("pq_quantize_act_smooth", lib().pq_quantize_act_smooth(x.data_ptr(), s_inv.data_ptr(), M, K, q.data_ptr(),
                                                                  s_tok.data_ptr(), _stream()))
    return q, s_tok


def pq_quantize_act_static(x: torch.Tensor, scale: torch.Tensor, q: torch.Tensor | None = None,
                           s_tok: torch.Tensor | None = None):
    """INT8 codes against one calibrated scale: x f16 [M,K], scale f32 device tensor with one element
    -> (q int8 [M,K], s_tok f32 [M] filled with the scale)."""
    M, K, q, s_tok = _rows(x, q, s_tok)
    scale = _sized(scale, torch.float32, 1, "scale")
    _together(x, scale)
    _check("pq_quantize_act_static", lib().pq_quantize_act_static(x.data_ptr(), scale.data_ptr(), M, K, q.data_ptr(),
                                                                  s_tok.data_ptr(), _stream()))
    return q, s_tok


def pq_quantize_act_static_channel(x: torch.Tensor, inv_s: torch.Tensor, q: torch.Tensor | None = None,
                                   s_tok: torch.Tensor | None = None):
    """INT8 codes against one calibrated scale per feature channel: x f16 [M,K], inv_s f32 [K] (reciprocal
    scales) -> (q int8 [M,K], s_tok f32 [M] = 1; fold the channel scales into the weights)."""
    M, K, q, s_tok = _rows(x, q, s_tok)
    inv_s = _factors(inv_s, K, "inv_s")
    _together(x, inv_s)
    _check("pq_quantize_act_static_channel", lib().pq_quantize_act_static_channel(x.data_ptr(), inv_s.data_ptr(), M, K,
                                                                                  q.data_ptr(), s_tok.data_ptr(), _stream()))
    return q, s_tok


def pq_swiglu_quantize(gate: torch.Tensor, up: torch.Tensor, q: torch.Tensor | None = None,
                       s_tok: torch.Tensor | None = None):
    """The MLP's gated activation fused with the down projection's quantizer: gate, up f16 [M,I] ->
    (q int8 [M,I], s_tok f32 [M]) of h = silu(gate) * up."""
    M, I, q, s_tok = _rows(gate, q, s_tok)
    _sized(up, torch.float16, M * I, "up")
    _together(gate, up)
    _check("pq_swiglu_quantize", lib().pq_swiglu_quantize(gate.data_ptr(), up.data_ptr(), M, I, q.data_ptr(),
                                                          s_tok.data_ptr(), _stream()))
    return q, s_tok


def pq_hadamard_block(K: int) -> int:
    """Order of the Hadamard blocks the Eq. 4 calls use for rows of length K (host-only query)."""
    return int(lib().pq_hadamard_block(int(K)))


def pq_quantize_act_hadamard(x: torch.Tensor, q: torch.Tensor | None = None, s_tok: torch.Tensor | None = None):
    """Quantizes X H (Eq. 4): x f16 [M,K] -> (q int8 [M,K], s_tok f32 [M])."""
    M, K, q, s_tok = _rows(x, q, s_tok)
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


def pq_smooth_scales(x_absmax: torch.Tensor, w_absmax: torch.Tensor, alpha_quarters: int = 2):
    """Eq. 3: (s, s_inv) f32 [K] from the column maxima of X and of W, alpha = alpha_quarters / 4 (default 1/2)."""
    xa = _dev(x_absmax, torch.float32, "x_absmax")
    wa = _factors(w_absmax, xa.shape[0], "w_absmax")
    s, s_inv = torch.empty_like(xa), torch.empty_like(xa)
    _check("pq_smooth_scales_alpha", lib().pq_smooth_scales_alpha(xa.data_ptr(), wa.data_ptr(), xa.shape[0],
                                                                  int(alpha_quarters), s.data_ptr(), s_inv.data_ptr(),
                                                                  _stream()))
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
    wq = _dev(_sized(wq, torch.uint8, N * K, "wq"), torch.uint8, "wq")
    codes = torch.empty((N, K), dtype=torch.int8, device=wq.device)
    _check("pq_unpack_w8", lib().pq_unpack_w8(wq.data_ptr(), N, K, codes.data_ptr(), _stream()))
    return codes


def pq_unpack_w4(wp: torch.Tensor, N: int, K: int) -> torch.Tensor:
    wp = _dev(_sized(wp, torch.uint8, N * K // 2, "wp"), torch.uint8, "wp")
    codes = torch.empty((N, K), dtype=torch.int8, device=wp.device)
    _check("pq_unpack_w4", lib().pq_unpack_w4(wp.data_ptr(), N, K, codes.data_ptr(), _stream()))
    return codes


def pq_plan_w8a8(M: int, N: int, K: int, sms: int = 148, scratch_bytes: int = 0) -> tuple[int, int]:
    """(tile width, number of K parts) the W8A8 GEMM would choose; host-only, needs no GPU."""
    bn, sp = _i32(0), _i32(0)
    _check("pq_plan_w8a8", lib().pq_plan_w8a8(M, N, K, sms, scratch_bytes, ctypes.byref(bn), ctypes.byref(sp)))
    return int(bn.value), int(sp.value)


def pq_workspace_bytes(M: int, Ns, K: int, sms: int = 148) -> int:
    """Bytes of workspace with which pq_gemm_w8a8 (Ns = one width) or pq_gemm_w8a8_group (Ns = the members'
    widths) at these M and K runs the schedule it would pick with unlimited room; 0 if that schedule does not
    split K.  Host-only, needs no GPU."""
    Ns = [int(Ns)] if isinstance(Ns, int) else [int(n) for n in Ns]
    arr = (_i64 * max(len(Ns), 1))(*Ns)
    return int(lib().pq_workspace_bytes(int(M), arr, len(Ns), int(K), int(sms)))


def pq_workspace_init(workspace: torch.Tensor) -> torch.Tensor:
    """Prepares a caller-owned workspace (uint8 CUDA tensor, 256-byte aligned, >= 64 KiB) for the W8A8 calls
    on the current stream: zeroes its arrival counters.  Returns the tensor."""
    workspace = _dev(workspace, torch.uint8, "workspace")
    with torch.cuda.device(workspace.device):
        _check("pq_workspace_init", lib().pq_workspace_init(workspace.data_ptr(), workspace.numel(), _stream()))
    return workspace


def pq_set_wait_limit(polls: int) -> None:
    """Poll bound of the waits inside kernels launched from now on (0 = the default).  Test hook."""
    _check("pq_set_wait_limit", lib().pq_set_wait_limit(int(polls)))


def pq_gemm_w8a8(q, s_tok, wq, s_ch, N: int, y: torch.Tensor | None = None,
                 workspace: torch.Tensor | None = None) -> torch.Tensor:
    """q int8 [M,K], s_tok f32 [M], wq/s_ch from pq_pack_w8 -> y f16 [M,N].  workspace: optional prepared
    scratch of this call (pq_workspace_bytes / pq_workspace_init); without it K is never split."""
    M, K = _tokens(q, s_tok)
    _sized(wq, torch.uint8, N * K, "wq"), _sized(s_ch, torch.float32, N, "s_ch")
    ws, ws_bytes = _ws(workspace)
    if y is not None:
        _sized(y, torch.float16, M * N, "y")
    _together(q, s_tok, wq, s_ch, y, workspace)
    y = _out(y, M, N, q)
    _check("pq_gemm_w8a8", lib().pq_gemm_w8a8(q.data_ptr(), s_tok.data_ptr(), wq.data_ptr(), s_ch.data_ptr(),
                                              M, N, K, y.data_ptr(), ws, ws_bytes, _stream()))
    return y


def _group_arrays(q, s_tok, members, ys, w_dtype, w_numel, s_dtype, s_numel, M, workspace=None):
    n = len(members)
    if not 1 <= n <= MAX_GROUP:
        raise ValueError(f"a group holds 1..{MAX_GROUP} members")
    if ys is None:
        ys = [None] * n
    if len(ys) != n:
        raise ValueError("one output per member")
    for i, ((w, sc, N), y) in enumerate(zip(members, ys)):
        N = int(N)
        _sized(w, w_dtype, w_numel(N), f"members[{i}] weights")
        _sized(sc, s_dtype, s_numel(N), f"members[{i}] scales")
        if y is not None:
            _sized(y, torch.float16, M * N, f"ys[{i}]")
    _together(q, s_tok, workspace, *[m[0] for m in members], *[m[1] for m in members], *ys)
    outs = [_out(y, M, int(m[2]), q) for m, y in zip(members, ys)]
    w_arr = (_vp * n)(*[m[0].data_ptr() for m in members])
    s_arr = (_vp * n)(*[m[1].data_ptr() for m in members])
    n_arr = (_i64 * n)(*[int(m[2]) for m in members])
    y_arr = (_vp * n)(*[y.data_ptr() for y in outs])
    return n, w_arr, s_arr, n_arr, y_arr, outs


def pq_gemm_w8a8_group(q, s_tok, members, ys=None, workspace: torch.Tensor | None = None) -> list[torch.Tensor]:
    """Several W8A8 linears over the same quantized tokens as one call (one kernel launch).  members: sequence of (wq, s_ch, N) from pq_pack_w8; ys: optional outputs f16 [M,N_g]; workspace: as for pq_gemm_w8a8.
    Returns the outputs; each equals pq_gemm_w8a8(q, s_tok, wq, s_ch, N) bit for bit."""
    M, K = _tokens(q, s_tok)
    ws, ws_bytes = _ws(workspace)
    n, wq_arr, sc_arr, n_arr, y_arr, outs = _group_arrays(q, s_tok, members, ys, torch.uint8, lambda N: N * K,
                                                          torch.float32, lambda N: N, M, workspace)
    _check("pq_gemm_w8a8_group", lib().pq_gemm_w8a8_group(q.data_ptr(), s_tok.data_ptr(), n, wq_arr, sc_arr, n_arr,
                                                          y_arr, M, K, ws, ws_bytes, _stream()))
    return outs


def pq_gemm_w4a8_group(q, s_tok, members, ys=None, group: int = GROUP) -> list[torch.Tensor]:
    """Several W4A8 linears over the same quantized tokens as one call (one kernel launch).  members: sequence of (wp, s_grp, N) from pq_pack_w4; ys: optional outputs f16 [M,N_g].
    Each output equals pq_gemm_w4a8(q, s_tok, wp, s_grp, N) bit for bit."""
    M, K = _tokens(q, s_tok)
    n, wp_arr, sg_arr, n_arr, y_arr, outs = _group_arrays(q, s_tok, members, ys, torch.uint8, lambda N: N * K // 2,
                                                          torch.float16, lambda N: (K // max(group, 1)) * N, M)
    _check("pq_gemm_w4a8_group", lib().pq_gemm_w4a8_group(q.data_ptr(), s_tok.data_ptr(), n, wp_arr, sg_arr, group,
                                                          n_arr, y_arr, M, K, _stream()))
    return outs


def pq_gemm_w8a8_noalloc(q, s_tok, wq, s_ch, N: int, y: torch.Tensor) -> torch.Tensor:
    """Same product as pq_gemm_w8a8, for callers that may not allocate: the output tensor is
    required (this wrapper creates none) and the library's built-in scratch array is used instead of
    a workspace.  Raises PQError with status 7 when M > 128 and the padded output exceeds 2 Mi
    elements.  Calls on one device must not overlap on the GPU."""
    M, K = _tokens(q, s_tok)
    _sized(wq, torch.uint8, N * K, "wq"), _sized(s_ch, torch.float32, N, "s_ch")
    if y is None:
        raise ValueError("y: required (this entry point creates no tensor)")
    _sized(y, torch.float16, M * N, "y")
    _together(q, s_tok, wq, s_ch, y)
    _check("pq_gemm_w8a8_noalloc", lib().pq_gemm_w8a8_noalloc(q.data_ptr(), s_tok.data_ptr(), wq.data_ptr(),
                                                              s_ch.data_ptr(), M, N, K, y.data_ptr(), _stream()))
    return y


def pq_gemm_w4a8(q, s_tok, wp, s_grp, N: int, group: int = GROUP, y: torch.Tensor | None = None) -> torch.Tensor:
    """q int8 [M,K], s_tok f32 [M], wp/s_grp from pq_pack_w4 -> y f16 [M,N]."""
    M, K = _tokens(q, s_tok)
    _sized(wp, torch.uint8, N * K // 2, "wp"), _sized(s_grp, torch.float16, (K // max(group, 1)) * N, "s_grp")
    if y is not None:
        _sized(y, torch.float16, M * N, "y")
    _together(q, s_tok, wp, s_grp, y)
    y = _out(y, M, N, q)
    _check("pq_gemm_w4a8", lib().pq_gemm_w4a8(q.data_ptr(), s_tok.data_ptr(), wp.data_ptr(), s_grp.data_ptr(),
                                              group, M, N, K, y.data_ptr(), _stream()))
    return y


def _linear_args(x, y, q_tmp, s_tok_tmp, N):
    if x.dim() != 2:
        raise ValueError("x: expected a 2-D tensor [M,K]")
    M, K = x.shape
    _sized(x, torch.float16, M * K, "x")
    if q_tmp is None:
        q_tmp = torch.empty((M, K), dtype=torch.int8, device=x.device)
    if s_tok_tmp is None:
        s_tok_tmp = torch.empty((M,), dtype=torch.float32, device=x.device)
    _sized(q_tmp, torch.int8, M * K, "q_tmp"), _sized(s_tok_tmp, torch.float32, M, "s_tok_tmp")
    if y is not None:
        _sized(y, torch.float16, M * N, "y")
    return M, K, _out(y, M, N, x), q_tmp, s_tok_tmp


def pq_linear_w8a8(x, wq, s_ch, N: int, y: torch.Tensor | None = None, q_tmp: torch.Tensor | None = None,
                   s_tok_tmp: torch.Tensor | None = None, workspace: torch.Tensor | None = None) -> torch.Tensor:
    """x f16 [M,K] -> y f16 [M,N]: pq_quantize_act + pq_gemm_w8a8 in one call (one launch for one to four tokens
    where the row kernel serves).  q_tmp / s_tok_tmp: the caller's buffers for codes and scales (allocated here
    when not given)."""
    M, K, y, q_tmp, s_tok_tmp = _linear_args(x, y, q_tmp, s_tok_tmp, N)
    _sized(wq, torch.uint8, N * K, "wq"), _sized(s_ch, torch.float32, N, "s_ch")
    ws, ws_bytes = _ws(workspace)
    _together(x, wq, s_ch, y, q_tmp, s_tok_tmp, workspace)
    _check("pq_linear_w8a8", lib().pq_linear_w8a8(x.data_ptr(), wq.data_ptr(), s_ch.data_ptr(), M, N, K, y.data_ptr(),
                                                  q_tmp.data_ptr(), s_tok_tmp.data_ptr(), ws, ws_bytes, _stream()))
    return y


def pq_linear_w4a8(x, wp, s_grp, N: int, group: int = GROUP, y: torch.Tensor | None = None,
                   q_tmp: torch.Tensor | None = None, s_tok_tmp: torch.Tensor | None = None) -> torch.Tensor:
    """x f16 [M,K] -> y f16 [M,N]: pq_quantize_act + pq_gemm_w4a8 in one call (see pq_linear_w8a8)."""
    M, K, y, q_tmp, s_tok_tmp = _linear_args(x, y, q_tmp, s_tok_tmp, N)
    _sized(wp, torch.uint8, N * K // 2, "wp"), _sized(s_grp, torch.float16, (K // max(group, 1)) * N, "s_grp")
    _together(x, wp, s_grp, y, q_tmp, s_tok_tmp)
    _check("pq_linear_w4a8", lib().pq_linear_w4a8(x.data_ptr(), wp.data_ptr(), s_grp.data_ptr(), group, M, N, K,
                                                  y.data_ptr(), q_tmp.data_ptr(), s_tok_tmp.data_ptr(), _stream()))
    return y


def pq_acc_w8a8(q, wq, N: int) -> torch.Tensor:
    """Exact INT32 accumulators [M,N] of the W8A8 product."""
    if q.dim() != 2:
        raise ValueError("q: expected a 2-D tensor [M,K]")
    M, K = q.shape
    _sized(q, torch.int8, M * K, "q"), _sized(wq, torch.uint8, N * K, "wq")
    _together(q, wq)
    acc = torch.empty((M, N), dtype=torch.int32, device=q.device)
    _check("pq_acc_w8a8", lib().pq_acc_w8a8(q.data_ptr(), wq.data_ptr(), M, N, K, acc.data_ptr(), _stream()))
    return acc


def pq_acc_w4a8(q, wp, N: int, group: int = GROUP) -> torch.Tensor:
    """Exact INT32 per-group accumulators [K/group, M, N] of the W4A8 product."""
    if q.dim() != 2:
        raise ValueError("q: expected a 2-D tensor [M,K]")
    M, K = q.shape
    _sized(q, torch.int8, M * K, "q"), _sized(wp, torch.uint8, N * K // 2, "wp")
    _together(q, wp)
    acc = torch.empty((K // group, M, N), dtype=torch.int32, device=q.device)
    _check("pq_acc_w4a8", lib().pq_acc_w4a8(q.data_ptr(), wp.data_ptr(), group, M, N, K, acc.data_ptr(), _stream()))
    return acc


def pq_device_status() -> int:
    """Synchronizes; returns and clears the device status word (0 = ok, 6 = a bounded wait expired)."""
    v = ctypes.c_int(0)
    _check("pq_device_status", lib().pq_device_status(ctypes.byref(v)))
    return int(v.value)
