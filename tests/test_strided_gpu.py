"""Inputs in the layout a model's QKV projection leaves them in: q, k, v as slices of a fused
[B, N, 3, H, D] activation (token stride 3*H*D) or as [B, N, H, D] arrays (token stride H*D), passed
as permuted views of logical shape [B, H, N, D].  The mixers read them through tensor maps with the
caller's strides; the output stays [B, H, N, D] contiguous.  Each case is compared with the float64
CPU oracle on the same values and, bit for bit, with the same call on contiguous copies (the
arithmetic is the same, only the addresses differ)."""
import pytest
import torch

from paper_2605_26636_b200 import inputs
from tests._util import TOL, dwc_to_device, guarded_empty, rel_err

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


@pytest.fixture(scope="module")
def jv():
    from paper_2605_26636_b200 import jetvit
    jetvit.lib()
    yield jetvit
    assert jetvit.device_status() == jetvit.JV_OK


def fused_views(q, k, v):
    """[B, H, N, D] CPU tensors -> views of one fused [B, N, 3, H, D] device activation."""
    qkv = torch.stack([t.permute(0, 2, 1, 3) for t in (q, k, v)], dim=2).contiguous().to(DEV)   # [B, N, 3, H, D]
    views = tuple(qkv[:, :, i].permute(0, 2, 1, 3) for i in range(3))
    assert not views[0].is_contiguous() and views[0].stride(2) == 3 * q.shape[1] * q.shape[3]
    return qkv, views


def bnhd_views(q, k, v):
    """[B, H, N, D] CPU tensors -> views of three separate [B, N, H, D] device arrays."""
    keep = [t.permute(0, 2, 1, 3).contiguous().to(DEV) for t in (q, k, v)]
    return keep, tuple(t.permute(0, 2, 1, 3) for t in keep)


CASES = [  # B, H, Hg, Wg, win_h, win_w
    (2, 3, 64, 64, 16, 16),      # two-tile windows; N = 4096: the four-tile full-attention kernel
    (1, 2, 73, 73, 16, 16),      # ragged grid: edge windows, clipped tiles
    (2, 2, 24, 40, 8, 16),       # one-tile windows
    (1, 4, 17, 33, 8, 8),        # windows of 64 tokens: the two-tile-per-CTA kernel; short full attention
    (3, 1, 40, 24, 40, 24),      # one window: W is F
]


@pytest.mark.parametrize("maker", [fused_views, bnhd_views], ids=["fused_qkv", "bnhd"])
@pytest.mark.parametrize("case", CASES, ids=lambda c: "x".join(map(str, c)))
def test_mixers_read_strided_inputs(jv, oracle, case, maker):
    B, H, Hg, Wg, wh, ww = case
    q, k, v = inputs.custom_qkv(B, H, Hg * Wg, 64, "bf16", seed=4000 + Hg + 7 * Wg + H)
    keep, (sq, sk, sv) = maker(q, k, v)
    cq, ck, cv = (t.to(DEV) for t in (q, k, v))
    d = inputs.dwc_weights(H * 64, 16, 3, 91)
    dd = dwc_to_device(d, DEV)
    ds = {"k": 3, "R": 0, "b2": dd["b2"]}
    checks = [
        ("L", lambda a, b, c, o: jv.linear_attn(a, b, c, Hg, Wg, out=o), lambda: oracle.linear_attn(q, k, v, Hg, Wg)),
        ("L+dwc", lambda a, b, c, o: jv.linear_attn(a, b, c, Hg, Wg, dwc=dd, out=o),
         lambda: oracle.linear_attn(q, k, v, Hg, Wg, dwc=d)),
        ("L+static", lambda a, b, c, o: jv.linear_attn(a, b, c, Hg, Wg, dwc=ds, out=o), None),
        ("W", lambda a, b, c, o: jv.window_attn(a, b, c, Hg, Wg, wh, ww, out=o),
         lambda: oracle.window_attn(q, k, v, Hg, Wg, wh, ww)),
        ("F", lambda a, b, c, o: jv.full_attn(a, b, c, out=o), lambda: oracle.full_attn(q, k, v)),
    ]
    for name, run, ref in checks:
        out, check = guarded_empty(q.shape, cq.dtype, DEV)
        out.fill_(float("nan"))
        run(sq, sk, sv, out)
        check()
        plain = torch.empty_like(cq)
        run(cq, ck, cv, plain)
        assert torch.equal(out, plain), (name, case)
        if ref is not None:
            assert rel_err(out, ref()) <= TOL["bf16"], (name, case)


def test_schedule_driver_reads_strided_inputs(jv, oracle):
    B, H, Hg, Wg = 1, 2, 32, 48
    layers = [inputs.custom_qkv(B, H, Hg * Wg, 64, "bf16", seed=4100 + l) for l in range(3)]
    keep, views = zip(*[fused_views(*t) for t in layers])
    outs = jv.hybrid_mixers("LWF", [t[0] for t in views], [t[1] for t in views], [t[2] for t in views], Hg, Wg, 16, 16)
    refs = oracle.hybrid_mixers("LWF", [t[0] for t in layers], [t[1] for t in layers], [t[2] for t in layers], Hg, Wg, 16, 16)
    for o, r in zip(outs, refs):
        assert o.is_contiguous()
        assert rel_err(o, r) <= TOL["bf16"]


def test_strided_inputs_outside_the_tensor_core_paths_are_refused(jv):
    B, H, Hg, Wg = 1, 2, 16, 16
    q, k, v = inputs.custom_qkv(B, H, Hg * Wg, 64, "f32", seed=4200)
    _, (sq, sk, sv) = fused_views(q, k, v)
    for call in (lambda: jv.linear_attn(sq, sk, sv, Hg, Wg), lambda: jv.window_attn(sq, sk, sv, Hg, Wg, 8, 8),
                 lambda: jv.full_attn(sq, sk, sv)):
        with pytest.raises(jv.JetVitError) as e:
            call()
        assert e.value.status == jv.JV_ERR_UNSUPPORTED
    q, k, v = inputs.custom_qkv(B, H, 3 + Hg * Wg, 64, "bf16", seed=4201)
    _, (sq, sk, sv) = fused_views(q, k, v)
    dd = dwc_to_device(inputs.dwc_weights(H * 64, 16, 3, 92), DEV)
    d5 = dwc_to_device(inputs.dwc_weights(H * 64, 16, 5, 93), DEV)
    for call in (lambda: jv.linear_attn(sq, sk, sv, Hg, Wg, dwc=dd, prefix=3),          # pooling minus the prefix rows
                 lambda: jv.window_attn(sq, sk, sv, Hg, Wg, 8, 8, prefix=3),          # the prefix queries' kernel
                 lambda: jv.linear_attn_focused(sq, sk, sv, Hg, Wg, 3.0, prefix=3)):
        with pytest.raises(jv.JetVitError) as e:
            call()
        assert e.value.status == jv.JV_ERR_UNSUPPORTED
    q, k, v = inputs.custom_qkv(B, H, Hg * Wg, 64, "bf16", seed=4202)
    _, (sq, sk, sv) = fused_views(q, k, v)
    with pytest.raises(jv.JetVitError) as e:
        jv.linear_attn(sq, sk, sv, Hg, Wg, dwc=d5)                                     # 5 x 5 kernels
    assert e.value.status == jv.JV_ERR_UNSUPPORTED
    # prefix tokens without a convolution are folded into the token axis: served
    q, k, v = inputs.custom_qkv(B, H, 3 + Hg * Wg, 64, "bf16", seed=4203)
    _, (sq, sk, sv) = fused_views(q, k, v)
    out = jv.linear_attn(sq, sk, sv, Hg, Wg, prefix=3)
    assert torch.equal(out, jv.linear_attn(*(t.to(DEV) for t in (q, k, v)), Hg, Wg, prefix=3))


def test_binding_rejects_mixed_layouts(jv):
    q, k, v = inputs.custom_qkv(1, 2, 64, 64, "bf16", seed=4300)
    _, (sq, sk, sv) = fused_views(q, k, v)
    with pytest.raises(ValueError):
        jv.full_attn(sq, k.to(DEV), sv)
    with pytest.raises(ValueError):      # a strided output
        jv.full_attn(sq, sk, sv, out=torch.empty(1, 64, 2, 64, dtype=sq.dtype, device=DEV).permute(0, 2, 1, 3))
