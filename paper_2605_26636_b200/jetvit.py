"""ctypes binding of libjetvit.so: same names as the C ABI, argument marshalling
only.  Tensors are CUDA ``torch`` tensors (device memory and streams come from
PyTorch); every step of every mixer runs in the library's CUDA kernels.  There
is no CPU path: if the library is missing or a call fails, an exception is raised.
"""
from __future__ import annotations

import ctypes
import os
from typing import Optional, Sequence

import torch

JV_OK, JV_ERR_INVALID_ARG, JV_ERR_UNSUPPORTED, JV_ERR_WORKSPACE, JV_ERR_CUDA, JV_ERR_TIMEOUT = range(6)
JV_F32, JV_BF16 = 0, 1

_HERE = os.path.dirname(os.path.abspath(__file__))
# JETVIT_LIB selects another build of the same library (e.g. one compiled with other tuning macros)
LIB_PATH = os.environ.get("JETVIT_LIB") or os.path.join(_HERE, "libjetvit.so")


class JvShape(ctypes.Structure):
    _fields_ = [("B", ctypes.c_int32), ("H", ctypes.c_int32), ("Hg", ctypes.c_int32),
                ("Wg", ctypes.c_int32), ("D", ctypes.c_int32), ("dtype", ctypes.c_int32), ("P", ctypes.c_int32),
                ("in_layout", ctypes.c_int32), ("in_tok_stride", ctypes.c_int64)]


class JvDwc(ctypes.Structure):
    _fields_ = [("k", ctypes.c_int32), ("R", ctypes.c_int32), ("W1", ctypes.c_void_p),
                ("b1", ctypes.c_void_p), ("W2", ctypes.c_void_p), ("b2", ctypes.c_void_p),
                ("token_wise", ctypes.c_int32)]


class JetVitError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        super().__init__(f"{where}: {status_string(status)} (jv_status {status})")


_lib = None


def lib() -> ctypes.CDLL:
    """Loads libjetvit.so (built in-tree by ``paper_2605_26636_b200.build``)."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise ImportError(f"{LIB_PATH} is missing: run `python -m paper_2605_26636_b200.build` "
                              "(there is no fallback path)")
        L = ctypes.CDLL(LIB_PATH)
        vp, sz, i32, f32 = ctypes.c_void_p, ctypes.c_size_t, ctypes.c_int32, ctypes.c_float
        shp, dwc = ctypes.POINTER(JvShape), ctypes.POINTER(JvDwc)
        L.jv_workspace_bytes.argtypes = [ctypes.c_char, shp, dwc]
        L.jv_workspace_bytes.restype = sz
        L.jv_linear_attn.argtypes = [vp, vp, vp, vp, shp, f32, dwc, vp, sz, vp]
        L.jv_linear_attn_focused.argtypes = [vp, vp, vp, vp, shp, f32, f32, dwc, vp, sz, vp]
        L.jv_linear_attn_focused.restype = ctypes.c_int
        L.jv_linear_attn_static.argtypes = [vp, vp, vp, vp, shp, f32, dwc, vp]
        L.jv_linear_attn_static.restype = ctypes.c_int
        L.jv_window_attn.argtypes = [vp, vp, vp, vp, shp, i32, i32, f32, vp, sz, vp]
        L.jv_full_attn.argtypes = [vp, vp, vp, vp, shp, f32, vp, sz, vp]
        L.jv_hybrid_mixers.argtypes = [i32, ctypes.c_char_p, ctypes.POINTER(vp), ctypes.POINTER(vp),
                                       ctypes.POINTER(vp), ctypes.POINTER(vp), shp, i32, i32, f32, f32,
                                       ctypes.POINTER(dwc), vp, sz, vp]
        L.jv_device_status.argtypes = [vp]
        L.jv_selftest_wait_timeout.argtypes = [ctypes.c_uint32, vp, vp]
        L.jv_selftest_wait_timeout.restype = ctypes.c_int
        L.jv_qkv_proj.argtypes = [vp, vp, vp, vp, vp, vp, shp, vp]
        L.jv_out_proj.argtypes = [vp, vp, vp, vp, shp, vp]
        for f in (L.jv_linear_attn, L.jv_window_attn, L.jv_full_attn, L.jv_hybrid_mixers, L.jv_device_status,
                  L.jv_qkv_proj, L.jv_out_proj):
            f.restype = ctypes.c_int
        L.jv_set_force_generic.argtypes = [i32]
        L.jv_set_force_generic.restype = i32
        L.jv_launch_count.restype = ctypes.c_uint64
        L.jv_status_string.argtypes = [ctypes.c_int]
        L.jv_status_string.restype = ctypes.c_char_p
        L.jv_version.restype = ctypes.c_char_p
        _lib = L
    return _lib


def status_string(status: int) -> str:
    return lib().jv_status_string(int(status)).decode()


def version() -> str:
    return lib().jv_version().decode()


def launch_count() -> int:
    return int(lib().jv_launch_count())


def set_force_generic(on: bool) -> bool:
    return bool(lib().jv_set_force_generic(1 if on else 0))


def _dtype_code(t: torch.Tensor) -> int:
    if t.dtype == torch.float32:
        return JV_F32
    if t.dtype == torch.bfloat16:
        return JV_BF16
    raise TypeError(f"dtype {t.dtype}: the mixers take float32 or bfloat16")


JV_LAYOUT_BHND, JV_LAYOUT_BNHD = 0, 1


def _in_layout(t: torch.Tensor):
    """(jv_layout, token stride) of an input tensor of logical shape [B, H, N, D]: contiguous, or a
    [B, N, H, D] array seen through ``permute(0, 2, 1, 3)`` whose token rows are ``stride(2)`` elements
    apart, e.g. ``qkv[:, :, i].permute(0, 2, 1, 3)`` of a fused [B, N, 3, H, D] activation."""
    if t.is_contiguous():
        return JV_LAYOUT_BHND, 0
    B, H, N, D = t.shape
    sb, sh, sn, sd = t.stride()
    if sd == 1 and sh == D and sn >= H * D and (sb == N * sn or B == 1):
        return JV_LAYOUT_BNHD, sn
    raise ValueError("inputs must be contiguous [B,H,N,D] tensors or permuted views of [B,N,H,D] token rows")


def make_shape(t: torch.Tensor, Hg: int, Wg: int, prefix: int = 0) -> JvShape:
    """Shape of [B, H, prefix + Hg*Wg, D] tensors: ``prefix`` tokens (class / register tokens) in
    front of the grid tokens.  The layout of the inputs is taken from ``t`` (see ``_in_layout``)."""
    B, H, N, D = t.shape
    if prefix < 0 or N != prefix + Hg * Wg:
        raise ValueError(f"N = {N} is not prefix + Hg*Wg = {prefix} + {Hg}*{Wg}")
    layout, tok_stride = _in_layout(t)
    return JvShape(B, H, Hg, Wg, D, _dtype_code(t), prefix, layout, tok_stride)


def _check_tensors(*ts: torch.Tensor):
    """q, k, v[, o]: one shape, dtype and device; q, k, v in one layout; o (a fourth tensor) contiguous."""
    ref = ts[0]
    for i, t in enumerate(ts):
        if not t.is_cuda:
            raise ValueError("tensors must live on a CUDA device (there is no CPU path)")
        if t.shape != ref.shape or t.dtype != ref.dtype or t.device != ref.device:
            raise ValueError("q, k, v, o must be [B,H,N,D] tensors of one shape, dtype and device")
        if i < 3 and _in_layout(t) != _in_layout(ref):
            raise ValueError("q, k and v must share one layout (all contiguous, or all views with the same token stride)")
        if i >= 3 and not t.is_contiguous():
            raise ValueError("o must be a contiguous [B,H,N,D] tensor")


def _empty_out(q: torch.Tensor) -> torch.Tensor:
    return torch.empty(q.shape, dtype=q.dtype, device=q.device)


def make_dwc(d: Optional[dict], device) -> Optional[JvDwc]:
    """dict(k, R, W1, b1, W2, b2) of fp32 CUDA tensors -> jv_dwc.  The dict must stay
    alive until the call has been enqueued."""
    if d is None:
        return None
    static = int(d["R"]) == 0          # static kernels in b2: no generator weights
    for key in (("b2",) if static else ("W1", "W2")):
        t = d.get(key)
        if t is None or not (t.is_cuda and t.dtype == torch.float32 and t.is_contiguous()):
            raise ValueError(f"dwc[{key!r}] must be a contiguous fp32 CUDA tensor")
    ptr = lambda t: None if t is None else t.data_ptr()
    return JvDwc(int(d["k"]), int(d["R"]), ptr(d.get("W1")), ptr(d.get("b1")), ptr(d.get("W2")), ptr(d.get("b2")),
                 int(d.get("token_wise", 0)))


def _stream(stream) -> int:
    s = torch.cuda.current_stream() if stream is None else stream
    return s.cuda_stream


def workspace_bytes(mixer: str, shape: JvShape, dwc: Optional[JvDwc] = None) -> int:
    return int(lib().jv_workspace_bytes(mixer.encode()[:1], ctypes.byref(shape),
                                        ctypes.byref(dwc) if dwc is not None else None))


def alloc_workspace(mixer: str, shape: JvShape, dwc: Optional[JvDwc], device) -> Optional[torch.Tensor]:
    n = workspace_bytes(mixer, shape, dwc)
    return torch.empty(max(n, 256), dtype=torch.uint8, device=device) if n else None


def _ws_args(ws: Optional[torch.Tensor]):
    return (None, 0) if ws is None else (ws.data_ptr(), ws.numel() * ws.element_size())


def _raise(status: int, where: str):
    if status != JV_OK:
        raise JetVitError(status, where)


def linear_attn(q, k, v, Hg: int, Wg: int, eps: float = 1e-6, dwc: Optional[dict] = None, out=None,
                ws: Optional[torch.Tensor] = None, stream=None, prefix: int = 0) -> torch.Tensor:
    """jv_linear_attn.  Allocates ``out`` / ``ws`` with torch when not given."""
    out = _empty_out(q) if out is None else out
    _check_tensors(q, k, v, out)
    shape = make_shape(q, Hg, Wg, prefix)
    d = make_dwc(dwc, q.device)
    with torch.cuda.device(q.device):
        if ws is None:
            ws = alloc_workspace("L", shape, d, q.device)
            if ws is not None and stream is not None:
                ws.record_stream(stream)      # freed by torch on the current stream, used on `stream`
        wp, wn = _ws_args(ws)
        st = lib().jv_linear_attn(q.data_ptr(), k.data_ptr(), v.data_ptr(), out.data_ptr(), ctypes.byref(shape),
                                  float(eps), ctypes.byref(d) if d is not None else None, wp, wn, _stream(stream))
    _raise(st, "jv_linear_attn")
    return out


def linear_attn_focused(q, k, v, Hg: int, Wg: int, focus_p: float, eps: float = 1e-6, dwc: Optional[dict] = None,
                        out=None, ws: Optional[torch.Tensor] = None, stream=None, prefix: int = 0) -> torch.Tensor:
    """jv_linear_attn_focused: the linear block with the focused feature map of Eq. 3 (power focus_p)."""
    out = _empty_out(q) if out is None else out
    _check_tensors(q, k, v, out)
    shape = make_shape(q, Hg, Wg, prefix)
    d = make_dwc(dwc, q.device)
    with torch.cuda.device(q.device):
        if ws is None:
            ws = alloc_workspace("f", shape, d, q.device)
            if ws is not None and stream is not None:
                ws.record_stream(stream)
        wp, wn = _ws_args(ws)
        st = lib().jv_linear_attn_focused(q.data_ptr(), k.data_ptr(), v.data_ptr(), out.data_ptr(), ctypes.byref(shape),
                                          float(eps), float(focus_p), ctypes.byref(d) if d is not None else None, wp, wn,
                                          _stream(stream))
    _raise(st, "jv_linear_attn_focused")
    return out


STATIC_SCRATCH_BYTES = 16 << 20


def linear_attn_static(q, k, v, Hg: int, Wg: int, eps: float = 1e-6, dwc: Optional[dict] = None, *, out,
                       stream=None, prefix: int = 0) -> torch.Tensor:
    """jv_linear_attn_static: the linear block with the library's built-in scratch, for
    callers that must not allocate.  This wrapper allocates nothing either: ``out`` is
    required.  Problems needing more than STATIC_SCRATCH_BYTES raise JV_ERR_WORKSPACE;
    calls that can overlap on the GPU must be ordered by the caller (they share the scratch)."""
    _check_tensors(q, k, v, out)
    shape = make_shape(q, Hg, Wg, prefix)
    d = make_dwc(dwc, q.device)
    with torch.cuda.device(q.device):
        st = lib().jv_linear_attn_static(q.data_ptr(), k.data_ptr(), v.data_ptr(), out.data_ptr(),
                                         ctypes.byref(shape), float(eps),
                                         ctypes.byref(d) if d is not None else None, _stream(stream))
    _raise(st, "jv_linear_attn_static")
    return out


def window_attn(q, k, v, Hg: int, Wg: int, win_h: int, win_w: int, scale: float = 0.0, out=None,
                stream=None, prefix: int = 0) -> torch.Tensor:
    """jv_window_attn (scale <= 0: 1/sqrt(D))."""
    out = _empty_out(q) if out is None else out
    _check_tensors(q, k, v, out)
    shape = make_shape(q, Hg, Wg, prefix)
    with torch.cuda.device(q.device):
        st = lib().jv_window_attn(q.data_ptr(), k.data_ptr(), v.data_ptr(), out.data_ptr(), ctypes.byref(shape),
                                  int(win_h), int(win_w), float(scale), None, 0, _stream(stream))
    _raise(st, "jv_window_attn")
    return out


def full_attn(q, k, v, Hg: Optional[int] = None, Wg: Optional[int] = None, scale: float = 0.0, out=None,
              stream=None) -> torch.Tensor:
    """jv_full_attn (scale <= 0: 1/sqrt(D)).  The grid split of N is irrelevant to F."""
    out = _empty_out(q) if out is None else out
    _check_tensors(q, k, v, out)
    if Hg is None or Wg is None:
        Hg, Wg = 1, q.shape[2]
    shape = make_shape(q, Hg, Wg)
    with torch.cuda.device(q.device):
        st = lib().jv_full_attn(q.data_ptr(), k.data_ptr(), v.data_ptr(), out.data_ptr(), ctypes.byref(shape),
                                float(scale), None, 0, _stream(stream))
    _raise(st, "jv_full_attn")
    return out


def hybrid_mixers(schedule: str, q: Sequence[torch.Tensor], k, v, Hg: int, Wg: int, win_h: int, win_w: int,
                  scale: float = 0.0, eps: float = 1e-6, dwc: Optional[Sequence[Optional[dict]]] = None,
                  out: Optional[Sequence[torch.Tensor]] = None, ws: Optional[torch.Tensor] = None, stream=None,
                  prefix: int = 0):
    """jv_hybrid_mixers: one mixer per layer, schedule[l] in 'L', 'W', 'F'."""
    n = len(schedule)
    if not (len(q) == len(k) == len(v) == n):
        raise ValueError("need one q, k, v per schedule entry")
    out = [_empty_out(t) for t in q] if out is None else list(out)
    for l in range(n):
        _check_tensors(q[l], k[l], v[l], out[l])
        if q[l].shape != q[0].shape or q[l].dtype != q[0].dtype or _in_layout(q[l]) != _in_layout(q[0]):
            raise ValueError("all layers share one shape, dtype and input layout")
    shape = make_shape(q[0], Hg, Wg, prefix)
    arr = lambda ts: (ctypes.c_void_p * n)(*[t.data_ptr() for t in ts])
    dstructs = [make_dwc(d, q[0].device) for d in dwc] if dwc is not None else None
    dptr = None
    if dstructs is not None:
        dptr = (ctypes.POINTER(JvDwc) * n)(*[ctypes.pointer(d) if d is not None else ctypes.POINTER(JvDwc)()
                                             for d in dstructs])
    with torch.cuda.device(q[0].device):
        if ws is None:
            need = 0
            for l, m in enumerate(schedule):
                if m == "L":
                    need = max(need, workspace_bytes("L", shape, dstructs[l] if dstructs else None))
            ws = torch.empty(max(need, 256), dtype=torch.uint8, device=q[0].device) if need else None
            if ws is not None and stream is not None:
                ws.record_stream(stream)      # freed by torch on the current stream, used on `stream`
        wp, wn = _ws_args(ws)
        st = lib().jv_hybrid_mixers(n, schedule.encode(), arr(q), arr(k), arr(v), arr(out), ctypes.byref(shape),
                                    int(win_h), int(win_w), float(scale), float(eps), dptr, wp, wn, _stream(stream))
    _raise(st, "jv_hybrid_mixers")
    return out


def _check_proj(x, w, bias, H: int, rows: int):
    C = 64 * H
    for t in (x, w):
        if not (t.is_cuda and t.dtype == torch.bfloat16 and t.is_contiguous()):
            raise ValueError("projection operands must be contiguous bf16 CUDA tensors")
    if tuple(w.shape) != (rows, C):
        raise ValueError(f"w must be [{rows}, {C}]")
    if bias is not None and not (bias.is_cuda and bias.dtype == torch.float32 and bias.is_contiguous()
                                 and tuple(bias.shape) == (rows,)):
        raise ValueError(f"bias must be a contiguous fp32 CUDA tensor of [{rows}]")


def qkv_proj(x, w, bias, H: int, Hg: int, Wg: int, out=None, stream=None, prefix: int = 0):
    """jv_qkv_proj: x [B, N, C] bf16, w [3C, C] bf16, bias fp32 [3C] or None -> (q, k, v), each
    [B, H, N, 64] in the mixers' layout.  ``out`` is an optional (q, k, v) triple to write into."""
    B, N, C = x.shape
    if C != 64 * H or N != prefix + Hg * Wg:
        raise ValueError("x must be [B, prefix + Hg*Wg, 64*H]")
    _check_proj(x, w, bias, H, 3 * C)
    q, k, v = out if out is not None else (torch.empty((B, H, N, 64), dtype=x.dtype, device=x.device) for _ in range(3))
    _check_tensors(q, k, v)
    if tuple(q.shape) != (B, H, N, 64) or q.dtype != x.dtype:
        raise ValueError("q, k, v must be [B, H, N, 64] bf16")
    shape = JvShape(B, H, Hg, Wg, 64, JV_BF16, prefix)
    with torch.cuda.device(x.device):
        st = lib().jv_qkv_proj(x.data_ptr(), w.data_ptr(), None if bias is None else bias.data_ptr(), q.data_ptr(),
                               k.data_ptr(), v.data_ptr(), ctypes.byref(shape), _stream(stream))
    _raise(st, "jv_qkv_proj")
    return q, k, v


def out_proj(o, w, bias, Hg: int, Wg: int, out=None, stream=None, prefix: int = 0) -> torch.Tensor:
    """jv_out_proj: o [B, H, N, 64] bf16 (a mixer's output), w [C, C] bf16, bias fp32 [C] or None
    -> y [B, N, C]."""
    B, H, N, D = o.shape
    if D != 64 or N != prefix + Hg * Wg:
        raise ValueError("o must be [B, H, prefix + Hg*Wg, 64]")
    C = 64 * H
    _check_proj(o, w, bias, H, C)
    y = torch.empty((B, N, C), dtype=o.dtype, device=o.device) if out is None else out
    if not (y.is_cuda and y.is_contiguous() and tuple(y.shape) == (B, N, C) and y.dtype == o.dtype):
        raise ValueError("y must be a contiguous [B, N, C] bf16 CUDA tensor")
    shape = JvShape(B, H, Hg, Wg, 64, JV_BF16, prefix)
    with torch.cuda.device(o.device):
        st = lib().jv_out_proj(o.data_ptr(), w.data_ptr(), None if bias is None else bias.data_ptr(), y.data_ptr(),
                               ctypes.byref(shape), _stream(stream))
    _raise(st, "jv_out_proj")
    return y


def selftest_wait_timeout(limit_us: int, gave_up: Optional[torch.Tensor] = None, stream=None) -> None:
    """jv_selftest_wait_timeout: enqueues a kernel whose bounded wait runs out after ``limit_us``
    microseconds and sets the sticky status word.  ``gave_up``: optional int32 CUDA tensor (1 element)."""
    st = lib().jv_selftest_wait_timeout(int(limit_us), None if gave_up is None else gave_up.data_ptr(),
                                        _stream(stream))
    _raise(st, "jv_selftest_wait_timeout")


def device_status(stream=None) -> int:
    """jv_device_status: synchronises the stream and returns the sticky status."""
    return int(lib().jv_device_status(_stream(stream)))
