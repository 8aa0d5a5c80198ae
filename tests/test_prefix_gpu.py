"""Prefix tokens (class / register tokens) beside the grid: every mixer, the schedule driver and the
projections with P tokens in front of the Hg x Wg grid tokens, CUDA kernels against the float64 CPU
oracle on the same seeded inputs, on both kernel paths (tensor-core and shape-generic).  The rule:
prefix tokens are global in F and in the linear attention proper, attend and are attended by every
window in W, and stay outside the depth-wise convolution and its pooling."""
import numpy as np
import pytest
import torch

from paper_2605_26636_b200 import inputs
from tests._util import TOL, dwc_to_device, guarded_empty, rel_err, sample_heads

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


@pytest.fixture(scope="module")
def jv():
    from paper_2605_26636_b200 import jetvit
    jetvit.lib()
    yield jetvit
    assert jetvit.device_status() == jetvit.JV_OK


@pytest.fixture(params=[False, True], ids=["fast", "generic"])
def both_paths(request, jv):
    prev = jv.set_force_generic(request.param)
    yield request.param
    jv.set_force_generic(prev)


def _dev(ts):
    return tuple(t.to(DEV) for t in ts)


CASES = [  # B, H, P, Hg, Wg, win
    (1, 2, 1, 64, 64, 16),
    (1, 2, 5, 64, 64, 16),
    (1, 2, 1, 73, 73, 16),
    (1, 2, 5, 73, 73, 16),
    (2, 3, 5, 17, 33, 16),
    (1, 1, 40, 24, 40, 8),       # more prefix tokens than a 32-key group
    (2, 2, 3, 7, 5, 4),
]


@pytest.mark.parametrize("dtype", ["bf16", "f32"])
@pytest.mark.parametrize("case", CASES, ids=lambda c: "x".join(map(str, c)))
def test_mixers_with_prefix_tokens(jv, oracle, both_paths, case, dtype):
    B, H, P, Hg, Wg, win = case
    if dtype == "f32" and Hg * Wg > 2000:
        pytest.skip("the fp32 kernels are the generic ones either way; the small grids cover them")
    q, k, v = inputs.custom_qkv(B, H, P + Hg * Wg, 64, dtype, seed=1000 * P + Hg + Wg)
    dq, dk, dv = _dev((q, k, v))
    d = inputs.dwc_weights(H * 64, 16, 3, 77 + P)
    dd = dwc_to_device(d, DEV)
    tol = TOL[dtype]
    checks = [
        ("L", lambda o: jv.linear_attn(dq, dk, dv, Hg, Wg, out=o, prefix=P),
         lambda: oracle.linear_attn(q, k, v, Hg, Wg, prefix=P)),
        ("L+dwc", lambda o: jv.linear_attn(dq, dk, dv, Hg, Wg, dwc=dd, out=o, prefix=P),
         lambda: oracle.linear_attn(q, k, v, Hg, Wg, dwc=d, prefix=P)),
        ("W", lambda o: jv.window_attn(dq, dk, dv, Hg, Wg, win, win, out=o, prefix=P),
         lambda: oracle.window_attn(q, k, v, Hg, Wg, win, win, prefix=P)),
        ("F", lambda o: jv.hybrid_mixers("F", [dq], [dk], [dv], Hg, Wg, win, win, out=[o], prefix=P),
         lambda: oracle.full_attn(q, k, v)),
    ]
    for name, run, ref in checks:
        out, check = guarded_empty(q.shape, dq.dtype, DEV)
        out.fill_(float("nan"))
        run(out)
        check()
        assert rel_err(out, ref()) <= tol, (name, case, dtype)


def test_linear_with_5x5_kernels_and_prefix_tokens(jv, oracle, both_paths):
    B, H, P, Hg, Wg = 1, 2, 5, 21, 18
    q, k, v = inputs.custom_qkv(B, H, P + Hg * Wg, 64, "bf16", seed=555)
    d = inputs.dwc_weights(H * 64, 16, 5, 556)
    out = jv.linear_attn(*_dev((q, k, v)), Hg, Wg, dwc=dwc_to_device(d, DEV), prefix=P)
    assert rel_err(out, oracle.linear_attn(q, k, v, Hg, Wg, dwc=d, prefix=P)) <= TOL["bf16"]
    kern = inputs.normal((H * 64 * 9,), 557) * 0.2                      # static 3 x 3 kernels
    out = jv.linear_attn(*_dev((q, k, v)), Hg, Wg, dwc={"k": 3, "R": 0, "b2": kern.to(DEV)}, prefix=P)
    assert rel_err(out, oracle.linear_attn(q, k, v, Hg, Wg, dwc={"k": 3, "R": 0, "b2": kern}, prefix=P)) <= TOL["bf16"]


def test_schedule_driver_with_prefix_tokens(jv, oracle, both_paths):
    B, H, P, Hg, Wg = 1, 2, 5, 32, 32
    sched = "LWFL"
    host = [inputs.custom_qkv(B, H, P + Hg * Wg, 64, "bf16", seed=600 + l) for l in range(4)]
    dws = [inputs.dwc_weights(H * 64, 16, 3, 5), None, None, None]
    dq, dk, dv = ([t[i].to(DEV) for t in host] for i in range(3))
    outs = jv.hybrid_mixers(sched, dq, dk, dv, Hg, Wg, 16, 16, prefix=P,
                            dwc=[None if d is None else dwc_to_device(d, DEV) for d in dws])
    refs = oracle.hybrid_mixers(sched, [t[0] for t in host], [t[1] for t in host], [t[2] for t in host],
                                Hg, Wg, 16, 16, dwc=dws, prefix=P)
    for l in range(4):
        assert rel_err(outs[l], refs[l]) <= TOL["bf16"], l


def test_prefix_full_size_dinov3_shape(jv, oracle):
    """The DINOv3-L shape with its five prefix tokens (class token + four registers): B=8, H=16,
    5 + 64 x 64 tokens; sampled (batch, head) pairs against the oracle."""
    w = inputs.WORKLOADS["dinov3_l"]
    P = 5
    q, k, v = inputs.custom_qkv(w.B, w.H, P + w.N, w.D, "bf16", seed=4101)
    dq, dk, dv = _dev((q, k, v))
    C = w.H * w.D
    d = inputs.dwc_weights(C, C // 8, 3, 4102)
    ol = jv.linear_attn(dq, dk, dv, w.Hg, w.Wg, dwc=dwc_to_device(d, DEV), prefix=P).cpu()
    ow = jv.window_attn(dq, dk, dv, w.Hg, w.Wg, 16, 16, prefix=P).cpu()
    torch.cuda.synchronize()
    ref_l = oracle.linear_attn(q[:2], k[:2], v[:2], w.Hg, w.Wg, dwc=d, prefix=P)     # whole samples (the generator pools per sample)
    assert rel_err(ol[:2], ref_l) <= TOL["bf16"]
    for b, h in sample_heads(w.B, w.H, 8, 41):
        sl = (slice(b, b + 1), slice(h, h + 1))
        assert rel_err(ow[sl], oracle.window_attn(q[sl], k[sl], v[sl], w.Hg, w.Wg, 16, 16, prefix=P)) <= TOL["bf16"], (b, h)


def test_projections_with_prefix_tokens(jv, oracle):
    B, H, P, Hg, Wg = 2, 4, 5, 12, 20
    C, N = 64 * H, P + Hg * Wg
    x = inputs.normal((B, N, C), 701, "bf16")
    w, b = inputs.proj_weights(3 * C, C, 702)
    wo, bo = inputs.proj_weights(C, C, 703)
    q, k, v = jv.qkv_proj(x.to(DEV), w.to(DEV), b.to(DEV), H, Hg, Wg, prefix=P)
    rq, rk, rv = oracle.qkv_proj(x, w, b, H)
    for got, want in ((q, rq), (k, rk), (v, rv)):
        assert rel_err(got, want) <= TOL["bf16"]
    y = jv.out_proj(q, wo.to(DEV), bo.to(DEV), Hg, Wg, prefix=P)
    assert rel_err(y, oracle.out_proj(q.cpu(), wo, bo)) <= TOL["bf16"]
