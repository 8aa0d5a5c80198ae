"""Host-side checks of the C ABI that need no GPU: the library loads, exports every
symbol the header declares, rejects bad arguments before any launch, and fails
loudly (never falls back to a CPU path) when no usable device is present."""
import ctypes
import os
import re

import pytest
import torch

from paper_2605_26636_b200 import build as jv_build
from paper_2605_26636_b200 import jetvit as jv

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def L():
    jv_build.build()
    return jv.lib()


def test_library_exports_every_declared_symbol(L):
    header = open(os.path.join(ROOT, "include", "jetvit.h")).read()
    header = re.sub(r"/\*.*?\*/", "", header, flags=re.S)
    names = set(re.findall(r"\b(jv_[a-z_]+)\s*\(", header))
    assert {"jv_linear_attn", "jv_window_attn", "jv_full_attn", "jv_hybrid_mixers", "jv_workspace_bytes",
            "jv_device_status"} <= names
    for n in sorted(names):
        assert hasattr(L, n), f"libjetvit.so does not export {n}"


def test_version_and_status_strings(L):
    assert "sm_100a" in jv.version()
    assert jv.status_string(jv.JV_OK) == "ok"
    for s in range(1, 6):
        assert jv.status_string(s) not in ("ok", "unknown status")
    assert jv.status_string(99) == "unknown status"


def test_workspace_bytes_host_logic(L):
    shp = jv.JvShape(8, 16, 64, 64, 64, jv.JV_BF16)
    assert jv.workspace_bytes("W", shp) == 0 and jv.workspace_bytes("F", shp) == 0
    nl = jv.workspace_bytes("L", shp)
    assert nl > 128 * 65 * 65 * 4            # at least one fp32 state per (batch, head)
    assert jv.workspace_bytes("S", shp) == nl
    d = jv.JvDwc(3, 128, 1, None, 1, None)    # pointers only need to be non-null here
    assert jv.workspace_bytes("L", shp, d) >= nl + 8 * 1024 * 9 * 4
    assert jv.workspace_bytes("L", jv.JvShape(0, 16, 64, 64, 64, jv.JV_BF16)) == 0
    assert jv.workspace_bytes("X", shp) == 0


# fake device addresses, spaced further apart than any tensor of the shapes used here
FQ, FK, FV, FO, FWS = 1 << 20, 2 << 20, 3 << 20, 4 << 20, 5 << 20


def _call_linear(L, shp, q=FQ, k=FK, v=FV, o=FO, eps=1e-6, dwc=None, ws=FWS, ws_bytes=1 << 40):
    return L.jv_linear_attn(q, k, v, o, ctypes.byref(shp), eps, dwc, ws, ws_bytes, None)


def test_argument_errors_are_found_before_any_launch(L):
    """Fake (never dereferenced) device addresses: every call must return an
    argument error, which it can only do if validation precedes the launch."""
    shp = jv.JvShape(1, 2, 8, 8, 64, jv.JV_F32)
    assert _call_linear(L, shp, q=None) == jv.JV_ERR_INVALID_ARG
    assert _call_linear(L, shp, q=FQ + 4) == jv.JV_ERR_INVALID_ARG         # misaligned
    assert _call_linear(L, shp, o=FQ) == jv.JV_ERR_INVALID_ARG             # o aliases q
    nbytes = 1 * 2 * 8 * 8 * 64 * 4
    assert _call_linear(L, shp, o=FV + nbytes - 16) == jv.JV_ERR_INVALID_ARG   # o overlaps the tail of v
    assert _call_linear(L, shp, o=FK - nbytes + 16) == jv.JV_ERR_INVALID_ARG   # the tail of o overlaps k
    if not torch.cuda.is_available():   # o right behind v, sharing no byte, passes validation
        assert _call_linear(L, shp, o=FV + nbytes) in (jv.JV_ERR_CUDA, jv.JV_ERR_UNSUPPORTED)
    assert _call_linear(L, shp, eps=-1.0) == jv.JV_ERR_INVALID_ARG
    assert _call_linear(L, shp, ws=None) == jv.JV_ERR_WORKSPACE
    assert _call_linear(L, shp, ws=FWS + 4) == jv.JV_ERR_WORKSPACE            # misaligned workspace
    assert _call_linear(L, shp, ws_bytes=16) == jv.JV_ERR_WORKSPACE
    bad = jv.JvDwc(4, 8, 1, None, 1, None)
    assert _call_linear(L, shp, dwc=ctypes.byref(bad)) == jv.JV_ERR_INVALID_ARG
    static_ok = jv.JvDwc(3, 0, None, None, None, 6 << 20)          # R = 0: static kernels in b2
    static_bad = jv.JvDwc(3, 0, None, None, None, None)
    assert _call_linear(L, shp, dwc=ctypes.byref(static_bad)) == jv.JV_ERR_INVALID_ARG
    if not torch.cuda.is_available():   # with fake addresses a call that passes validation may only run where nothing can launch
        assert _call_linear(L, shp, dwc=ctypes.byref(static_ok)) in (jv.JV_ERR_CUDA, jv.JV_ERR_UNSUPPORTED)
    assert _call_linear(L, jv.JvShape(1, 2, 8, 8, 64, 7)) == jv.JV_ERR_INVALID_ARG
    assert _call_linear(L, jv.JvShape(1, 2, 8, 8, 0, jv.JV_F32)) == jv.JV_ERR_INVALID_ARG
    assert _call_linear(L, jv.JvShape(1, 2, 8, 8, 512, jv.JV_F32)) == jv.JV_ERR_UNSUPPORTED
    assert _call_linear(L, jv.JvShape(1, 2, 8, 8, 30, jv.JV_BF16)) == jv.JV_ERR_UNSUPPORTED
    # input layout: unknown code, token rows that would overlap, a stride that breaks 16-byte alignment,
    # a stride without the layout that uses it; and an output inside the span of a strided input
    assert _call_linear(L, jv.JvShape(1, 2, 8, 8, 64, jv.JV_BF16, 0, 2, 0)) == jv.JV_ERR_INVALID_ARG
    assert _call_linear(L, jv.JvShape(1, 2, 8, 8, 64, jv.JV_BF16, 0, jv.JV_LAYOUT_BNHD, 64)) == jv.JV_ERR_INVALID_ARG
    assert _call_linear(L, jv.JvShape(1, 2, 8, 8, 64, jv.JV_BF16, 0, jv.JV_LAYOUT_BNHD, 3 * 128 + 4)) == jv.JV_ERR_INVALID_ARG
    assert _call_linear(L, jv.JvShape(1, 2, 8, 8, 64, jv.JV_BF16, 0, jv.JV_LAYOUT_BHND, 384)) == jv.JV_ERR_INVALID_ARG
    fused = jv.JvShape(1, 2, 8, 8, 64, jv.JV_BF16, 0, jv.JV_LAYOUT_BNHD, 384)
    span = (63 * 384 + 128) * 2                   # bytes from the first to one past the last element of a slice
    assert _call_linear(L, fused, o=FQ + span - 16) == jv.JV_ERR_INVALID_ARG
    if not torch.cuda.is_available():
        assert _call_linear(L, fused, o=FQ + span) in (jv.JV_ERR_CUDA, jv.JV_ERR_UNSUPPORTED)
    assert L.jv_window_attn(FQ, FK, FV, FO, ctypes.byref(shp), 0, 4, 0.0, None, 0, None) == jv.JV_ERR_INVALID_ARG
    assert L.jv_full_attn(FQ, FK, FV, None, ctypes.byref(shp), 0.0, None, 0, None) == jv.JV_ERR_INVALID_ARG
    assert L.jv_full_attn(FQ, FK, FV, FO, None, 0.0, None, 0, None) == jv.JV_ERR_INVALID_ARG


def test_hybrid_schedule_is_validated_before_any_launch(L):
    shp = jv.JvShape(1, 2, 8, 8, 64, jv.JV_F32)
    n = 3
    arr = lambda base: (ctypes.c_void_p * n)(*[base + (64 << 10) * i for i in range(n)])
    q, k, v, o = arr(1 << 20), arr(2 << 20), arr(3 << 20), arr(4 << 20)
    call = lambda sched, nl=n, ws=8 << 20, wsb=1 << 40: L.jv_hybrid_mixers(
        nl, sched, q, k, v, o, ctypes.byref(shp), 4, 4, 0.0, 1e-6, None, ws, wsb, None)
    assert call(b"LWX") == jv.JV_ERR_INVALID_ARG
    assert call(b"LW") == jv.JV_ERR_INVALID_ARG          # shorter than n_layers
    assert call(b"lwf") == jv.JV_ERR_INVALID_ARG
    assert call(b"LWF", nl=0) == jv.JV_ERR_INVALID_ARG
    assert call(b"LWF", ws=None) == jv.JV_ERR_WORKSPACE  # an L layer needs scratch


@pytest.mark.skipif(torch.cuda.is_available(), reason="checks the no-device behaviour")
def test_no_device_means_an_error_not_a_fallback(L):
    shp = jv.JvShape(1, 2, 8, 8, 64, jv.JV_F32)
    assert _call_linear(L, shp) in (jv.JV_ERR_CUDA, jv.JV_ERR_UNSUPPORTED)
    assert L.jv_full_attn(FQ, FK, FV, FO, ctypes.byref(shp), 0.0, None, 0, None) in (
        jv.JV_ERR_CUDA, jv.JV_ERR_UNSUPPORTED)
    with pytest.raises(ValueError):
        t = torch.zeros(1, 2, 64, 64)
        jv.full_attn(t, t, t)                # CPU tensors are refused by the binding


def test_force_generic_switch_roundtrip(L):
    prev = jv.set_force_generic(True)
    assert jv.set_force_generic(prev) is True
    assert jv.launch_count() >= 0
