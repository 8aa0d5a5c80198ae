"""The projections either side of a mixer (W_Q | W_K | W_V before it, W_O after it; Sec. 3.2.4:
the linear layers every block inherits).  CPU tests pin the oracle's two functions to things
other than themselves; GPU tests compare jv_qkv_proj / jv_out_proj with the oracle element by
element on the same seeded inputs (bf16 tensors, fp32 accumulation: 2e-2 of the output rms)."""
import ctypes

import numpy as np
import pytest
import torch

from paper_2605_26636_b200 import inputs
from tests._util import TOL, guarded_empty, rel_err


# ------------------------------------------------------------------ oracle pins (CPU)
def _rand(shape, seed):
    return np.random.default_rng(seed).standard_normal(shape)


def test_oracle_qkv_proj_against_scalar_loops(oracle):
    """Brute force on a tiny case: every output element from its own scalar sum, with the
    feature index spelled out (a swapped operand, a wrong row block or a head/feature mix-up
    in the layout mapping fails here)."""
    B, N, H, D = 2, 5, 3, 4
    C = H * D
    x, w, b = _rand((B, N, C), 1), _rand((3 * C, C), 2), _rand((3 * C,), 3)
    q, k, v = oracle.qkv_proj(x, w, b, H)
    for which, t in enumerate((q, k, v)):
        assert t.shape == (B, H, N, D)
        for bi in range(B):
            for h in range(H):
                for n in range(N):
                    for e in range(D):
                        f = which * C + h * D + e
                        ref = sum(x[bi, n, c] * w[f, c] for c in range(C)) + b[f]
                        assert abs(t[bi, h, n, e] - ref) <= 1e-12 * max(1.0, abs(ref))


def test_oracle_out_proj_against_scalar_loops(oracle):
    B, N, H, D = 2, 4, 3, 4
    C = H * D
    o, w, b = _rand((B, H, N, D), 4), _rand((C, C), 5), _rand((C,), 6)
    y = oracle.out_proj(o, w, b)
    assert y.shape == (B, N, C)
    for bi in range(B):
        for n in range(N):
            for f in range(C):
                ref = sum(o[bi, h, n, e] * w[f, h * D + e] for h in range(H) for e in range(D)) + b[f]
                assert abs(y[bi, n, f] - ref) <= 1e-12 * max(1.0, abs(ref))


def test_oracle_identity_weights_are_the_layout_permutation(oracle):
    """With w = [I; 2I; 3I] the projection only moves data: q is x with the head axis pulled out
    (torch's view + permute gives the same thing independently), and out_proj with w = I puts
    it back."""
    B, N, H, D = 2, 6, 4, 8
    C = H * D
    x = _rand((B, N, C), 7)
    w = np.concatenate([np.eye(C), 2 * np.eye(C), 3 * np.eye(C)])
    q, k, v = oracle.qkv_proj(x, w, None, H)
    heads = torch.from_numpy(x).view(B, N, H, D).permute(0, 2, 1, 3).numpy()
    assert np.array_equal(q, heads) and np.array_equal(k, 2 * heads) and np.array_equal(v, 3 * heads)
    assert np.array_equal(oracle.out_proj(q, np.eye(C), None), x)


def test_oracle_projections_are_affine(oracle):
    """Linearity in x and in w, and the bias enters once, un-scaled."""
    B, N, H, D = 1, 3, 2, 4
    C = H * D
    x1, x2, w, b = _rand((B, N, C), 8), _rand((B, N, C), 9), _rand((3 * C, C), 10), _rand((3 * C,), 11)
    a = oracle.qkv_proj(x1, w, None, H)
    c = oracle.qkv_proj(x2, w, None, H)
    s = oracle.qkv_proj(2 * x1 - x2, w, None, H)
    sb = oracle.qkv_proj(2 * x1 - x2, w, b, H)
    for which in range(3):
        assert np.allclose(s[which], 2 * a[which] - c[which], rtol=0, atol=1e-12)
        bias_view = b[which * C:(which + 1) * C].reshape(1, H, 1, D)
        assert np.allclose(sb[which] - s[which], np.broadcast_to(bias_view, s[which].shape), rtol=0, atol=1e-12)
    o = _rand((B, H, N, D), 12)
    wo, bo = _rand((C, C), 13), _rand((C,), 14)
    assert np.allclose(oracle.out_proj(o, wo, bo) - oracle.out_proj(o, wo, None), bo.reshape(1, 1, C), atol=1e-12)
    # composing the two with w_o = I recovers the q row block of the fused product
    q = oracle.qkv_proj(x1, w, b, H)[0]
    assert np.allclose(oracle.out_proj(q, np.eye(C), None), x1 @ w[:C].T + b[:C], atol=1e-12)


# ------------------------------------------------------------------ GPU parity
DEV = "cuda:0"


@pytest.fixture(scope="module")
def jv():
    from paper_2605_26636_b200 import jetvit
    jetvit.lib()
    assert torch.cuda.is_available()
    yield jetvit
    assert jetvit.device_status() == jetvit.JV_OK


# (B, H, Hg, Wg): one tile with a ragged tail; several token tiles per batch element with a tail;
# features that fill 1, 1.5 and 3 tiles of 256; C = 64 (a single K block, feature tile mostly empty)
CASES = [(1, 1, 4, 4), (2, 2, 9, 7), (1, 4, 16, 16), (3, 6, 13, 11), (2, 16, 20, 20), (1, 12, 37, 29)]


@pytest.mark.gpu
@pytest.mark.parametrize("with_bias", [True, False], ids=["bias", "nobias"])
@pytest.mark.parametrize("case", CASES, ids=lambda c: "x".join(map(str, c)))
def test_qkv_and_out_proj_match_the_oracle(jv, oracle, case, with_bias):
    B, H, Hg, Wg = case
    N, C = Hg * Wg, 64 * H
    seed = inputs.SEED_BASE + 50_000 + 97 * B + 13 * H + N
    x = inputs.normal((B, N, C), seed, "bf16")
    w, b = inputs.proj_weights(3 * C, C, seed + 1, with_bias)
    wo, bo = inputs.proj_weights(C, C, seed + 2, with_bias)
    ref = oracle.qkv_proj(x, w, b, H)
    outs, checks = zip(*[guarded_empty((B, H, N, 64), torch.bfloat16, DEV) for _ in range(3)])
    dev = lambda t: None if t is None else t.to(DEV)
    q, k, v = jv.qkv_proj(dev(x), dev(w), dev(b), H, Hg, Wg, out=outs)
    for got, want, chk in zip((q, k, v), ref, checks):
        chk()
        assert rel_err(got, want) <= TOL["bf16"]
    # the output projection reads what the first one wrote (bf16), as it reads a mixer's output
    y_ref = oracle.out_proj(q, wo, bo)
    y, chk = guarded_empty((B, N, C), torch.bfloat16, DEV)
    jv.out_proj(q, dev(wo), dev(bo), Hg, Wg, out=y)
    chk()
    assert rel_err(y, y_ref) <= TOL["bf16"]


@pytest.mark.gpu
def test_projection_mixer_projection_at_full_size(jv, oracle):
    """The DINOv3-L shape (B=8, H=16, 64x64 grid, C=1024) in the launch configuration the
    benchmark times: x -> q, k, v -> linear attention -> y, with sampled outputs checked
    against the oracle (whole token rows of sampled (batch, head) pairs; the chain's mixer
    through its own oracle on the projected tensors)."""
    wl = inputs.WORKLOADS["dinov3_l"]
    B, H, Hg, Wg, N, C = wl.B, wl.H, wl.Hg, wl.Wg, wl.N, wl.H * 64
    x = inputs.normal((B, N, C), inputs.seed_for(wl.cfg, 0, 5), "bf16")
    w, b = inputs.proj_weights(3 * C, C, inputs.seed_for(wl.cfg, 0, 6))
    wo, bo = inputs.proj_weights(C, C, inputs.seed_for(wl.cfg, 0, 7))
    dx, dw, db, dwo, dbo = (t.to(DEV) for t in (x, w, b, wo, bo))
    q, k, v = jv.qkv_proj(dx, dw, db, H, Hg, Wg)
    o = jv.linear_attn(q, k, v, Hg, Wg)
    y = jv.out_proj(o, dwo, dbo, Hg, Wg)
    torch.cuda.synchronize()
    # sampled batch elements: the whole fused product for those, every head and token
    for bi in (0, B - 1):
        ref = oracle.qkv_proj(x[bi:bi + 1], w, b, H)
        for got, want in zip((q, k, v), ref):
            assert rel_err(got[bi:bi + 1], want) <= TOL["bf16"]
        y_ref = oracle.out_proj(o[bi:bi + 1], wo, bo)
        assert rel_err(y[bi:bi + 1], y_ref) <= TOL["bf16"]
    # and the mixer in between on the projected tensors of one batch element
    o_ref = oracle.linear_attn(q[:1], k[:1], v[:1], Hg, Wg)
    assert rel_err(o[:1], o_ref) <= TOL["bf16"]


@pytest.mark.gpu
def test_projection_argument_errors(jv):
    L = jv.lib()
    good = jv.JvShape(1, 2, 4, 4, 64, jv.JV_BF16)
    t = torch.zeros(1 << 19, dtype=torch.bfloat16, device=DEV)
    p = [t.data_ptr() + (128 << 10) * i for i in range(6)]       # further apart than any operand here (w: 96 KB)
    call = lambda shp, ptrs=p, bias=None: L.jv_qkv_proj(ptrs[0], ptrs[1], bias, ptrs[2], ptrs[3], ptrs[4],
                                                       ctypes.byref(shp), None)
    assert call(jv.JvShape(1, 2, 4, 4, 64, jv.JV_F32)) == jv.JV_ERR_UNSUPPORTED
    assert call(jv.JvShape(1, 2, 4, 4, 32, jv.JV_BF16)) == jv.JV_ERR_UNSUPPORTED
    assert call(jv.JvShape(0, 2, 4, 4, 64, jv.JV_BF16)) == jv.JV_ERR_INVALID_ARG
    assert call(good, [p[0], p[1], p[2], p[2], p[4]]) == jv.JV_ERR_INVALID_ARG      # k aliases q
    assert call(good, [p[0], p[1], p[0], p[3], p[4]]) == jv.JV_ERR_INVALID_ARG      # q aliases x
    assert call(good, [p[0], p[1], p[2], p[2] + 4096 - 16, p[4]]) == jv.JV_ERR_INVALID_ARG   # k overlaps the tail of q
    assert call(good, [p[0] + 2, p[1], p[2], p[3], p[4]]) == jv.JV_ERR_INVALID_ARG  # misaligned
    assert call(good, bias=p[5] + 4) == jv.JV_ERR_INVALID_ARG
    assert L.jv_out_proj(p[0], p[1], None, None, ctypes.byref(good), None) == jv.JV_ERR_INVALID_ARG
    assert L.jv_out_proj(p[0], p[1], None, p[0], ctypes.byref(good), None) == jv.JV_ERR_INVALID_ARG
    assert jv.device_status() == jv.JV_OK
