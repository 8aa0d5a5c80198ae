"""ctypes front end of the float64 CPU oracle (``jv_oracle.c``).

TEST INFRASTRUCTURE ONLY: imported by the tests, by the smoke check and by the
CPU-baseline / reference legs of the benchmark.  Nothing here touches the CUDA
library, and the CUDA binding never imports this module.

Every function takes array-likes, converts them exactly to float64 and returns
a float64 ``numpy`` array.  Shapes follow the mixers' ``[B, H, N, D]`` layout.
"""
from __future__ import annotations

import ctypes
import os
import subprocess

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "jv_oracle.c")
_SO = os.path.join(_HERE, "libjv_oracle.so")
_lib = None

_c_dp = ctypes.POINTER(ctypes.c_double)
_i64 = ctypes.c_int64


def build(force: bool = False) -> str:
    """Compile ``jv_oracle.c`` with gcc (no fast-math: fp64 in source order)."""
    if force or not os.path.exists(_SO) or os.path.getmtime(_SO) < os.path.getmtime(_SRC):
        tmp = _SO + f".tmp{os.getpid()}"
        subprocess.check_call(
            ["gcc", "-O2", "-fopenmp", "-shared", "-fPIC", "-o", tmp, _SRC, "-lm"])
        os.replace(tmp, _SO)
    return _SO


def _load():
    global _lib
    if _lib is None:
        lib = ctypes.CDLL(build())
        lib.jvo_num_threads.restype = ctypes.c_int
        lib.jvo_full_attn.argtypes = [_c_dp] * 4 + [_i64] * 4 + [ctypes.c_double]
        lib.jvo_window_attn.argtypes = [_c_dp] * 4 + [_i64] * 6 + [ctypes.c_double]
        lib.jvo_dwc_generate.argtypes = [_c_dp] * 2 + [_i64] * 6 + [_c_dp] * 4
        lib.jvo_linear_attn.argtypes = ([_c_dp] * 4 + [_i64] * 5 + [ctypes.c_double]
                                        + [_i64] * 2 + [_c_dp] * 4)
        lib.jvo_window_attn_prefix.argtypes = [_c_dp] * 4 + [_i64] * 7 + [ctypes.c_double]
        lib.jvo_dwc_generate_prefix.argtypes = [_c_dp] * 2 + [_i64] * 7 + [_c_dp] * 4
        lib.jvo_linear_attn_prefix.argtypes = ([_c_dp] * 4 + [_i64] * 6 + [ctypes.c_double]
                                               + [_i64] * 2 + [_c_dp] * 4)
        lib.jvo_linear_attn_tokenwise.argtypes = lib.jvo_linear_attn_prefix.argtypes
        lib.jvo_linear_attn_tokenwise.restype = None
        lib.jvo_focus_map.argtypes = [_c_dp] * 2 + [_i64] * 2 + [ctypes.c_double]
        lib.jvo_focus_map.restype = None
        for f in (lib.jvo_full_attn, lib.jvo_window_attn, lib.jvo_dwc_generate,
                  lib.jvo_linear_attn, lib.jvo_window_attn_prefix, lib.jvo_dwc_generate_prefix,
                  lib.jvo_linear_attn_prefix):
            f.restype = None
        _lib = lib
    return _lib


def num_threads() -> int:
    """Threads the oracle's OpenMP loops use on this host."""
    return int(_load().jvo_num_threads())


def _f64(a) -> np.ndarray:
    if hasattr(a, "detach"):  # torch tensor (bf16 has no numpy dtype: widen first)
        a = a.detach().cpu().double().numpy()
    return np.ascontiguousarray(a, dtype=np.float64)


def _p(a):
    return None if a is None else a.ctypes.data_as(_c_dp)


def full_attn(q, k, v, scale=None) -> np.ndarray:
    """Eq. 1.  q: [B,H,Nq,D]; k, v: [B,H,Nk,D] -> [B,H,Nq,D]."""
    q, k, v = _f64(q), _f64(k), _f64(v)
    B, H, Nq, D = q.shape
    Nk = k.shape[2]
    assert k.shape == (B, H, Nk, D) and v.shape == (B, H, Nk, D)
    if scale is None or scale <= 0:
        scale = 1.0 / np.sqrt(D)
    o = np.empty_like(q)
    _load().jvo_full_attn(_p(q), _p(k), _p(v), _p(o), B * H, Nq, Nk, D, float(scale))
    return o


def window_attn(q, k, v, Hg, Wg, win_h, win_w, scale=None, prefix=0, _force_prefix_code=False) -> np.ndarray:
    """Sec. 3.2.2 window attention.  q, k, v: [B,H,prefix + Hg*Wg,D]; ``prefix`` tokens in
    front of the grid tokens attend, and are attended by, everything (see jv_oracle.c)."""
    q, k, v = _f64(q), _f64(k), _f64(v)
    B, H, N, D = q.shape
    assert N == prefix + Hg * Wg and k.shape == q.shape and v.shape == q.shape
    if scale is None or scale <= 0:
        scale = 1.0 / np.sqrt(D)
    o = np.empty_like(q)
    if prefix == 0 and not _force_prefix_code:
        _load().jvo_window_attn(_p(q), _p(k), _p(v), _p(o), B * H, Hg, Wg, D,
                                win_h, win_w, float(scale))
    else:
        _load().jvo_window_attn_prefix(_p(q), _p(k), _p(v), _p(o), B * H, prefix, Hg, Wg, D,
                                       win_h, win_w, float(scale))
    return o


def dwc_generate(v, dwc, prefix=0, _force_prefix_code=False) -> np.ndarray:
    """Dynamic depth-wise kernels [B, C, k, k] from V [B,H,prefix + N,D] (Sec. 3.2.1); the
    pooling runs over the N grid tokens only."""
    v = _f64(v)
    B, H, N, D = v.shape
    N -= prefix
    kk, R = int(dwc["k"]), int(dwc["R"])
    W1, W2 = _f64(dwc["W1"]), _f64(dwc["W2"])
    b1 = None if dwc.get("b1") is None else _f64(dwc["b1"])
    b2 = None if dwc.get("b2") is None else _f64(dwc["b2"])
    C = H * D
    assert W1.shape == (R, C) and W2.shape == (C * kk * kk, R)
    w = np.empty((B, C, kk, kk), dtype=np.float64)
    if prefix == 0 and not _force_prefix_code:
        _load().jvo_dwc_generate(_p(v), _p(w), B, H, N, D, kk, R, _p(W1), _p(b1), _p(W2), _p(b2))
    else:
        _load().jvo_dwc_generate_prefix(_p(v), _p(w), B, H, prefix, N, D, kk, R, _p(W1), _p(b1), _p(W2), _p(b2))
    return w


def linear_attn(q, k, v, Hg, Wg, eps=1e-6, dwc=None, prefix=0, _force_prefix_code=False) -> np.ndarray:
    """JetViT linear-attention block (Eqs. 2, 4).  ``dwc``: None or a dict with
    keys k, R, W1 [R,C], b1 [R] or None, W2 [C*k*k,R], b2 [C*k*k] or None.
    q, k, v: [B,H,prefix + Hg*Wg,D]; prefix tokens take part in the attention, not in the
    convolution or its pooling (see jv_oracle.c)."""
    q, k, v = _f64(q), _f64(k), _f64(v)
    B, H, N, D = q.shape
    assert N == prefix + Hg * Wg and k.shape == q.shape and v.shape == q.shape
    o = np.empty_like(q)
    old = prefix == 0 and not _force_prefix_code

    def call(kk, R, W1, b1, W2, b2):
        if old:
            _load().jvo_linear_attn(_p(q), _p(k), _p(v), _p(o), B, H, Hg, Wg, D, float(eps),
                                    kk, R, _p(W1), _p(b1), _p(W2), _p(b2))
        else:
            _load().jvo_linear_attn_prefix(_p(q), _p(k), _p(v), _p(o), B, H, prefix, Hg, Wg, D, float(eps),
                                           kk, R, _p(W1), _p(b1), _p(W2), _p(b2))

    if dwc is None:
        call(0, 0, None, None, None, None)
        return o
    if dwc.get("token_wise"):     # one set of kernels per token (Table 1 "+ Token-wise Dynamic DWC")
        kk, R = int(dwc["k"]), int(dwc["R"])
        W1, W2 = _f64(dwc["W1"]), _f64(dwc["W2"])
        b1 = None if dwc.get("b1") is None else _f64(dwc["b1"])
        b2 = None if dwc.get("b2") is None else _f64(dwc["b2"])
        assert R > 0 and W1.shape == (R, H * D) and W2.shape == (H * D * kk * kk, R)
        _load().jvo_linear_attn_tokenwise(_p(q), _p(k), _p(v), _p(o), B, H, prefix, Hg, Wg, D, float(eps),
                                          kk, R, _p(W1), _p(b1), _p(W2), _p(b2))
        return o
    kk, R = int(dwc["k"]), int(dwc["R"])
    C = H * D
    b1 = None if dwc.get("b1") is None else _f64(dwc["b1"])
    b2 = None if dwc.get("b2") is None else _f64(dwc["b2"])
    if R == 0:      # static depth-wise convolution (Table 1 "DWC"): the kernels are b2, no generator
        assert b2 is not None and b2.size == C * kk * kk
        W1 = W2 = None
    else:
        W1, W2 = _f64(dwc["W1"]), _f64(dwc["W2"])
        assert W1.shape == (R, C) and W2.shape == (C * kk * kk, R)
    assert kk % 2 == 1
    call(kk, R, W1, b1, W2, b2)
    return o


def focus_map(x, p) -> np.ndarray:
    """Focused feature map of Eq. 3 over the last axis: (||r|| / ||r^p||) r^p with r = ReLU(x)."""
    x = _f64(x)
    out = np.empty_like(x)
    _load().jvo_focus_map(_p(x), _p(out), x.size // x.shape[-1], x.shape[-1], float(p))
    return out


def linear_attn_focused(q, k, v, Hg, Wg, focus_p, eps=1e-6, dwc=None, prefix=0) -> np.ndarray:
    """The linear-attention block with the focused feature map in place of ReLU (Table 1,
    "+ DWC on V + Focusing Factor"): Eq. 2 with phi = phi_p of Eq. 3, the row normalisation and
    Eq. 4's convolution as in linear_attn.  phi_p is non-negative, so the block equals the ReLU
    block applied to phi_p(Q), phi_p(K): that is how it is evaluated."""
    return linear_attn(focus_map(q, focus_p), focus_map(k, focus_p), v, Hg, Wg, eps=eps, dwc=dwc, prefix=prefix)


def hybrid_mixers(schedule, q, k, v, Hg, Wg, win_h, win_w, scale=None, eps=1e-6, dwc=None, prefix=0):
    """Per-layer L/W/F schedule over a stack of independent layers.
    q, k, v: sequences of [B,H,prefix + N,D] arrays, one per layer; dwc: None or a
    per-layer sequence whose entries may be None."""
    out = []
    for l, m in enumerate(schedule):
        if m == "L":
            out.append(linear_attn(q[l], k[l], v[l], Hg, Wg, eps,
                                   None if dwc is None else dwc[l], prefix=prefix))
        elif m == "W":
            out.append(window_attn(q[l], k[l], v[l], Hg, Wg, win_h, win_w, scale, prefix=prefix))
        elif m == "F":
            out.append(full_attn(q[l], k[l], v[l], scale))
        else:
            raise ValueError(f"schedule[{l}] = {m!r}: expected one of L, W, F")
    return out


def qkv_proj(x, w, bias, H):
    """The block's input projection W_Q | W_K | W_V (Sec. 3.2.4: inherited linear layers),
    written out as the definition: x [B, N, C], w [3C, C] (row = output feature
    which*C + h*D + e), bias [3C] or None -> q, k, v, each [B, H, N, D] with D = C / H:
    q[b, h, n, e] = sum_c x[b, n, c] w[h*D + e, c] + bias[h*D + e], and k, v from the
    next two row blocks of w."""
    x, w = _f64(x), _f64(w)
    B, N, C = x.shape
    assert C % H == 0 and w.shape == (3 * C, C)
    D = C // H
    y = x @ w.T                                    # [B, N, 3C]
    if bias is not None:
        y = y + _f64(bias).reshape(1, 1, 3 * C)
    out = []
    for which in range(3):
        t = np.empty((B, H, N, D), dtype=np.float64)
        for h in range(H):
            t[:, h] = y[:, :, which * C + h * D: which * C + (h + 1) * D]
        out.append(t)
    return tuple(out)


def out_proj(o, w, bias):
    """The block's output projection W_O (Sec. 3.2.4): o [B, H, N, D], w [C, C] with C = H*D
    (column = input feature h*D + e), bias [C] or None -> y [B, N, C]:
    y[b, n, f] = sum_{h, e} o[b, h, n, e] w[f, h*D + e] + bias[f]."""
    o, w = _f64(o), _f64(w)
    B, H, N, D = o.shape
    C = H * D
    assert w.shape == (C, C)
    y = np.zeros((B, N, C), dtype=np.float64)
    for h in range(H):
        y += o[:, h] @ w[:, h * D:(h + 1) * D].T
    if bias is not None:
        y = y + _f64(bias).reshape(1, 1, C)
    return y
