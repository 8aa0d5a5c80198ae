"""jv_linear_attn_static -- the linear-attention block for callers that cannot allocate
device memory (a server whose pool owns the GPU, a loop that must avoid cudaMalloc's
device-wide synchronisation, a stream-only plug-in hook).  It uses a scratch array built
into the library instead of a caller buffer, so this test checks it against the ordinary
entry point jv_linear_attn: same inputs, the same kernels, so the outputs must be equal bit
for bit (which is well inside the bf16 / fp32 parity tolerance; one case is also compared
with the float64 oracle), on two calls in a row (the second call meets the scratch as the
first one left it).
Collected last on purpose, so that a run stopping at the first failure has already run
every other test.  It passes on its own in a fresh process as well as after the others.
"""
import ctypes

import pytest
import torch

from paper_2605_26636_b200 import inputs
from tests._util import TOL, dwc_to_device, rel_err

DEV = "cuda:0"


@pytest.fixture(scope="module")
def jv():
    from paper_2605_26636_b200 import jetvit
    jetvit.lib()
    return jetvit


def _max_rel(a, b):
    a, b = a.double(), b.double()
    return float((a - b).abs().max() / b.pow(2).mean().sqrt())


@pytest.mark.gpu
@pytest.mark.parametrize("dtype", ["bf16", "f32"])
def test_static_scratch_matches_regular_entry_point_twice(jv, oracle, dtype):
    B, H, Hg, Wg, D = 2, 4, 48, 40, 64
    dh = inputs.dwc_weights(H * D, 32, 3, 123)
    d = dwc_to_device(dh, DEV)
    for call, use_dwc in enumerate([True, False]):          # two calls in a row, different work
        qh, kh, vh = inputs.custom_qkv(B, H, Hg * Wg, D, dtype, seed=70 + call)
        q, k, v = (t.to(DEV) for t in (qh, kh, vh))
        dwc = d if use_dwc else None
        ref = jv.linear_attn(q, k, v, Hg, Wg, dwc=dwc)
        out = torch.full_like(q, float("nan"))
        jv.linear_attn_static(q, k, v, Hg, Wg, dwc=dwc, out=out)
        torch.cuda.synchronize()
        assert torch.isfinite(out).all()
        assert _max_rel(out, ref) <= TOL[dtype], (call, dtype)
        assert torch.equal(out, ref), (call, dtype)          # same kernels, other scratch: the same bits
        assert rel_err(out, oracle.linear_attn(qh, kh, vh, Hg, Wg, dwc=dh if use_dwc else None)) <= TOL[dtype]
    assert jv.device_status() == jv.JV_OK


@pytest.mark.gpu
def test_static_scratch_full_size_dinov3_shape_repeated(jv):
    """The DINOv3-L shape (B=8, H=16, 64x64) needs about 6 MB of scratch: inside the limit."""
    w = inputs.WORKLOADS["dinov3_l"]
    q, k, v = (t.to(DEV) for t in inputs.qkv(w))
    ref = jv.linear_attn(q, k, v, w.Hg, w.Wg)
    out = torch.empty_like(q)
    for _ in range(2):
        out.fill_(float("nan"))
        jv.linear_attn_static(q, k, v, w.Hg, w.Wg, out=out)
        torch.cuda.synchronize()
        assert _max_rel(out, ref) <= TOL["bf16"]
        assert torch.equal(out, ref)


def test_static_scratch_rejects_oversized_problems_on_the_host(jv):
    """Needs no GPU: the size check comes before any CUDA call."""
    big = jv.JvShape(32, 16, 128, 128, 64, jv.JV_BF16)
    assert jv.workspace_bytes("L", big) > jv.STATIC_SCRATCH_BYTES
    st = jv.lib().jv_linear_attn_static(256, 512, 768, 1024, ctypes.byref(big), 1e-6, None, None)
    assert st == jv.JV_ERR_WORKSPACE
    assert jv.lib().jv_linear_attn_static(256, 512, 768, 1024, None, 1e-6, None, None) == jv.JV_ERR_INVALID_ARG
