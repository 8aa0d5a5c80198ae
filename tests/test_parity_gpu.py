"""GPU parity: the CUDA mixers (through the C ABI binding) against the float64
CPU oracle on the same seeded inputs.  Bar: max-abs error / rms(oracle) <= 1e-4
for fp32 tensors, <= 2e-2 for bf16 tensors with fp32 accumulation."""
import numpy as np
import pytest
import torch

from paper_2605_26636_b200 import inputs
from tests._util import TOL, dwc_to_device, guarded_empty, rel_err, sample_heads

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def jv():
    from paper_2605_26636_b200 import jetvit
    jetvit.lib()
    assert torch.cuda.is_available()
    yield jetvit
    assert jetvit.device_status() == jetvit.JV_OK


@pytest.fixture(params=[False, True], ids=["fast", "generic"])
def both_paths(request, jv):
    prev = jv.set_force_generic(request.param)
    yield request.param
    jv.set_force_generic(prev)


DEV = "cuda:0"


def _dev(ts):
    return tuple(t.to(DEV) for t in ts)


# ------------------------------------------------------------------ config 1: tiny, fp32
def test_tiny_fp32_all_mixers(jv, oracle, both_paths):
    w = inputs.WORKLOADS["tiny"]
    q, k, v = inputs.qkv(w)
    dq, dk, dv = _dev((q, k, v))
    assert rel_err(jv.linear_attn(dq, dk, dv, w.Hg, w.Wg), oracle.linear_attn(q, k, v, w.Hg, w.Wg)) <= TOL["f32"]
    assert rel_err(jv.window_attn(dq, dk, dv, w.Hg, w.Wg, 8, 8),
                   oracle.window_attn(q, k, v, w.Hg, w.Wg, 8, 8)) <= TOL["f32"]
    assert rel_err(jv.full_attn(dq, dk, dv), oracle.full_attn(q, k, v)) <= TOL["f32"]
    # one window covering the grid is full attention
    assert rel_err(jv.window_attn(dq, dk, dv, w.Hg, w.Wg, 16, 16), oracle.full_attn(q, k, v)) <= TOL["f32"]
    assert rel_err(jv.window_attn(dq, dk, dv, w.Hg, w.Wg, 64, 64), oracle.full_attn(q, k, v)) <= TOL["f32"]


@pytest.mark.parametrize("ksz", [3, 5])
def test_tiny_fp32_linear_with_squeeze_dynamic_dwc(jv, oracle, both_paths, ksz):
    w = inputs.WORKLOADS["tiny"]
    q, k, v = inputs.qkv(w)
    C = w.H * w.D
    d = inputs.dwc_weights(C, C // 8, ksz, inputs.seed_for(w.cfg, 0, 3))
    ref = oracle.linear_attn(q, k, v, w.Hg, w.Wg, dwc=d)
    out = jv.linear_attn(*_dev((q, k, v)), w.Hg, w.Wg, dwc=dwc_to_device(d, DEV))
    assert rel_err(out, ref) <= TOL["f32"]
    # without biases
    d2 = dict(d, b1=None, b2=None)
    ref = oracle.linear_attn(q, k, v, w.Hg, w.Wg, dwc=d2)
    out = jv.linear_attn(*_dev((q, k, v)), w.Hg, w.Wg, dwc=dwc_to_device(d2, DEV))
    assert rel_err(out, ref) <= TOL["f32"]


# ------------------------------------------------------------------ shape sweep with canaries
SWEEP = [  # B, H, Hg, Wg, D, win_h, win_w
    (1, 1, 7, 5, 64, 4, 4),
    (2, 3, 17, 33, 64, 16, 16),
    (1, 2, 73, 73, 64, 16, 16),
    (2, 2, 16, 48, 64, 16, 16),
    (1, 2, 40, 24, 64, 8, 16),
    (1, 2, 9, 9, 32, 3, 5),
    (1, 1, 12, 20, 128, 8, 8),
    (3, 1, 1, 1, 64, 1, 1),
    (1, 2, 33, 16, 64, 16, 16),
]


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
@pytest.mark.parametrize("case", SWEEP, ids=lambda c: "x".join(map(str, c)))
def test_shape_sweep(jv, oracle, both_paths, case, dtype):
    B, H, Hg, Wg, D, wh, ww = case
    q, k, v = inputs.custom_qkv(B, H, Hg * Wg, D, dtype, seed=Hg * 100 + Wg)
    dq, dk, dv = _dev((q, k, v))
    tol = TOL[dtype]
    for name in ("L", "W", "F"):
        out, check = guarded_empty(q.shape, dq.dtype, DEV)
        if name == "L":
            jv.linear_attn(dq, dk, dv, Hg, Wg, out=out)
            ref = oracle.linear_attn(q, k, v, Hg, Wg)
        elif name == "W":
            jv.window_attn(dq, dk, dv, Hg, Wg, wh, ww, out=out)
            ref = oracle.window_attn(q, k, v, Hg, Wg, wh, ww)
        else:
            jv.full_attn(dq, dk, dv, Hg, Wg, out=out)
            ref = oracle.full_attn(q, k, v)
        check()
        assert rel_err(out, ref) <= tol, f"{name} {case} {dtype}"


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
def test_sweep_linear_dwc_ragged(jv, oracle, both_paths, dtype):
    B, H, Hg, Wg, D = 2, 2, 19, 13, 64
    q, k, v = inputs.custom_qkv(B, H, Hg * Wg, D, dtype, seed=5)
    d = inputs.dwc_weights(H * D, 16, 3, 99)
    out, check = guarded_empty(q.shape, _dev((q,))[0].dtype, DEV)
    jv.linear_attn(*_dev((q, k, v)), Hg, Wg, dwc=dwc_to_device(d, DEV), out=out)
    check()
    assert rel_err(out, oracle.linear_attn(q, k, v, Hg, Wg, dwc=d)) <= TOL[dtype]


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
@pytest.mark.parametrize("ksz", [3, 5])
def test_linear_with_static_dwc(jv, oracle, both_paths, dtype, ksz):
    """R = 0: the static depth-wise convolution of Table 1 (kernels passed directly in b2)."""
    B, H, Hg, Wg, D = 2, 2, 21, 18, 64
    q, k, v = inputs.custom_qkv(B, H, Hg * Wg, D, dtype, seed=40 + ksz)
    kern = inputs.normal((H * D * ksz * ksz,), inputs.SEED_BASE + 777 + ksz) * 0.2
    d = {"k": ksz, "R": 0, "b2": kern}
    out, check = guarded_empty(q.shape, _dev((q,))[0].dtype, DEV)
    jv.linear_attn(*_dev((q, k, v)), Hg, Wg, dwc={"k": ksz, "R": 0, "b2": kern.to(DEV)}, out=out)
    check()
    assert rel_err(out, oracle.linear_attn(q, k, v, Hg, Wg, dwc=d)) <= TOL[dtype]


@pytest.mark.parametrize("case", [(2, 4, 48, 40), (1, 2, 16, 16), (1, 16, 24, 24), (4, 8, 32, 32)],
                         ids=lambda c: "x".join(map(str, c)))
def test_linear_dwc_with_poisoned_scratch_and_output(jv, oracle, case):
    """The convolution chain is several kernels that overlap through programmatic launches; a kernel that
    starts before the one it depends on has finished reads whatever the buffers held.  Scratch and output
    start as NaN here and the call is repeated, so an ordering mistake cannot pass on stale data."""
    B, H, Hg, Wg = case
    q, k, v = inputs.custom_qkv(B, H, Hg * Wg, 64, "bf16", seed=60 + B + H)
    d = inputs.dwc_weights(H * 64, 32, 3, 321)
    ref = oracle.linear_attn(q, k, v, Hg, Wg, dwc=d)
    dq, dk, dv = _dev((q, k, v))
    dd = dwc_to_device(d, DEV)
    shape = jv.make_shape(dq, Hg, Wg)
    ws = jv.alloc_workspace("L", shape, jv.make_dwc(dd, DEV), DEV)
    out = torch.empty_like(dq)
    for rep in range(4):
        ws.fill_(0xFF)                       # every fp32 word a NaN
        out.fill_(float("nan"))
        jv.linear_attn(dq, dk, dv, Hg, Wg, dwc=dd, out=out, ws=ws)
        torch.cuda.synchronize()
        assert rel_err(out, ref) <= TOL["bf16"], rep


# ------------------------------------------------------------------ window kernel: every box shape
WBOX = [  # B, H, Hg, Wg, win_h, win_w: windows of one or two 128-token boxes (box = win_w x 128 / win_w rows)
    (2, 2, 48, 80, 16, 16),      # two boxes of 16 x 8, whole windows only
    (1, 3, 41, 70, 16, 16),      # ragged: a bottom row of windows with one box (9 rows), a right column 6 wide
    (1, 2, 37, 50, 8, 16),       # one box per window; bottom windows of 5 rows, right windows 2 wide
    (1, 2, 20, 70, 8, 32),       # two boxes of 32 x 4; bottom windows of one box, right windows 6 wide
    (2, 1, 22, 100, 4, 32),      # one box of 32 x 4; bottom windows of 2 rows
    (1, 2, 70, 20, 32, 8),       # two boxes of 8 x 16; bottom windows of 6 rows (one box), right windows 4 wide
    (1, 1, 50, 12, 16, 8),       # one box of 8 x 16
    (1, 2, 100, 9, 64, 4),       # two boxes of 4 x 32; right windows 1 wide
    (5, 7, 16, 16, 16, 16),      # 35 windows: fewer than one CTA pair per SM, an odd count (a slot without work)
    (1, 2, 40, 9, 16, 16),       # a grid narrower than the window's box
    (2, 1, 5, 70, 8, 16),        # a grid lower than the window's box
]


@pytest.mark.parametrize("case", WBOX, ids=lambda c: "x".join(map(str, c)))
def test_window_kernel_box_shapes(jv, oracle, case):
    """The two-windows-per-CTA kernel over every tile box it accepts, with ragged grids in both directions
    (edge windows with one box instead of two, clipped stores, masked keys); one launch per call."""
    B, H, Hg, Wg, wh, ww = case
    q, k, v = inputs.custom_qkv(B, H, Hg * Wg, 64, "bf16", seed=7000 + Hg + 3 * Wg + wh)
    out, check = guarded_empty(q.shape, torch.bfloat16, DEV)
    out.fill_(float("nan"))
    launches = jv.launch_count()
    jv.window_attn(*_dev((q, k, v)), Hg, Wg, wh, ww, out=out)
    assert jv.launch_count() == launches + 1
    check()
    if B * H > 8:
        out = out.cpu()
        for b, h in sample_heads(B, H, 6, 9):
            sl = (slice(b, b + 1), slice(h, h + 1))
            assert rel_err(out[sl], oracle.window_attn(q[sl], k[sl], v[sl], Hg, Wg, wh, ww)) <= TOL["bf16"], (case, b, h)
    else:
        assert rel_err(out, oracle.window_attn(q, k, v, Hg, Wg, wh, ww)) <= TOL["bf16"], case


# ------------------------------------------------------------------ other model sizes and grids
@pytest.mark.parametrize("case", [(1, 12, 64, 128, 64), (1, 24, 32, 64, 64), (1, 4, 24, 40, 128)],
                         ids=["vitb_64x128", "giant_32x64", "d128_24x40"])
def test_other_model_shapes(jv, oracle, case):
    """Non-square grids (a 1024x2048 image at patch 16 is 64x128 tokens) with 12 and 24 heads on the
    tensor-core kernels, and head_dim 128 (F and W on their own tensor-core kernel, L on the shape-generic
    kernels); sampled (batch, head) pairs."""
    B, H, Hg, Wg, D = case
    q, k, v = inputs.custom_qkv(B, H, Hg * Wg, D, "bf16", seed=H + D)
    dq, dk, dv = _dev((q, k, v))
    d = inputs.dwc_weights(H * D, 32, 3, 11)
    ol = jv.linear_attn(dq, dk, dv, Hg, Wg, dwc=dwc_to_device(d, DEV)).cpu()
    ow = jv.window_attn(dq, dk, dv, Hg, Wg, 16, 16).cpu()
    of = jv.full_attn(dq, dk, dv, Hg, Wg).cpu()
    assert rel_err(ol, oracle.linear_attn(q, k, v, Hg, Wg, dwc=d)) <= TOL["bf16"]
    for b, h in sample_heads(B, H, 3, H):
        sl = (slice(b, b + 1), slice(h, h + 1))
        assert rel_err(ow[sl], oracle.window_attn(q[sl], k[sl], v[sl], Hg, Wg, 16, 16)) <= TOL["bf16"], ("W", b, h)
        assert rel_err(of[sl], oracle.full_attn(q[sl], k[sl], v[sl])) <= TOL["bf16"], ("F", b, h)


@pytest.mark.parametrize("case", [(1, 3, 32, 32), (1, 2, 37, 29), (2, 1, 35, 40), (1, 1, 31, 33)],
                         ids=lambda c: "x".join(map(str, c)))
def test_full_attention_long_sequences(jv, oracle, case):
    """N >= 1024 runs on the kernel with four query tiles per CTA: tile counts of 8, 9, 11 (the last item
    of a head holds one or three tiles) with ragged last key tiles, and 1023 tokens just below the switch."""
    B, H, Hg, Wg = case
    q, k, v = inputs.custom_qkv(B, H, Hg * Wg, 64, "bf16", seed=Hg + Wg)
    out, check = guarded_empty(q.shape, torch.bfloat16, DEV)
    jv.full_attn(*_dev((q, k, v)), Hg, Wg, out=out)
    check()
    assert rel_err(out, oracle.full_attn(q, k, v)) <= TOL["bf16"]


@pytest.mark.parametrize("n_tokens", [512, 2048])
def test_full_attention_with_a_rising_reference(jv, oracle, n_tokens):
    """Scores that grow along the sequence make the running softmax reference move again and again
    (accumulator rescaled many times); a sharp step in the middle makes it jump by far more than 2^8."""
    q, k, v = inputs.custom_qkv(1, 2, n_tokens, 64, "bf16", seed=n_tokens)
    ramp = torch.linspace(0.0, 1.0, n_tokens).view(1, 1, n_tokens, 1)
    u = q[:, :, :1, :].float()                      # keys lean more and more towards the first query
    k2 = (k.float() + 6.0 * ramp * u).to(torch.bfloat16)
    k2[:, :, n_tokens // 2] = (40.0 * u[:, :, 0]).to(torch.bfloat16)
    out = jv.full_attn(*_dev((q, k2, v)))
    assert rel_err(out, oracle.full_attn(q, k2, v)) <= TOL["bf16"]


def test_full_and_linear_take_any_token_count(jv, oracle):
    """F and L (without the convolution) do not look at the grid: a DINOv3 sequence with its five prefix
    tokens (CLS + 4 registers) in front of a 64x64 grid is just 4101 tokens, passed as a 1 x 4101 grid."""
    B, H, n_tok = 1, 3, 5 + 64 * 64
    q, k, v = inputs.custom_qkv(B, H, n_tok, 64, "bf16", seed=4101)
    dq, dk, dv = _dev((q, k, v))
    of = jv.full_attn(dq, dk, dv, 1, n_tok)
    ol = jv.linear_attn(dq, dk, dv, 1, n_tok)
    assert rel_err(ol, oracle.linear_attn(q, k, v, 1, n_tok)) <= TOL["bf16"]
    sl = (slice(0, 1), slice(1, 2))
    assert rel_err(of[sl], oracle.full_attn(q[sl], k[sl], v[sl])) <= TOL["bf16"]


def test_explicit_scale_and_eps(jv, oracle, both_paths):
    q, k, v = inputs.custom_qkv(1, 2, 16 * 16, 64, "bf16", seed=8)
    dq, dk, dv = _dev((q, k, v))
    assert rel_err(jv.full_attn(dq, dk, dv, scale=0.3), oracle.full_attn(q, k, v, scale=0.3)) <= TOL["bf16"]
    assert rel_err(jv.window_attn(dq, dk, dv, 16, 16, 16, 16, scale=0.05),
                   oracle.window_attn(q, k, v, 16, 16, 16, 16, scale=0.05)) <= TOL["bf16"]
    assert rel_err(jv.linear_attn(dq, dk, dv, 16, 16, eps=50.0),
                   oracle.linear_attn(q, k, v, 16, 16, eps=50.0)) <= TOL["bf16"]


def test_degenerate_inputs(jv, oracle, both_paths):
    """All-negative q in L gives exactly 0; large logits do not overflow in F / W."""
    q, k, v = inputs.custom_qkv(1, 2, 16 * 16, 64, "bf16", seed=9)
    qn = -q.abs()
    out = jv.linear_attn(*_dev((qn, k, v)), 16, 16)
    assert float(out.abs().max()) == 0.0
    qb, kb = q * 12, k * 12          # logits of a few hundred: softmax is nearly one-hot
    dq, dk, dv = _dev((qb, kb, v))
    assert rel_err(jv.full_attn(dq, dk, dv), oracle.full_attn(qb, kb, v)) <= TOL["bf16"]
    assert rel_err(jv.window_attn(dq, dk, dv, 16, 16, 16, 16), oracle.window_attn(qb, kb, v, 16, 16, 16, 16)) <= TOL["bf16"]


def test_back_to_back_calls_match_isolated_calls_bit_for_bit(jv):
    """Every kernel is deterministic, so a chain of calls enqueued without any synchronisation (kernels of
    neighbouring calls overlap through programmatic launches and share the workspace) must reproduce, bit
    for bit, what each call gives when it runs alone between two synchronisations."""
    B, H, Hg, Wg = 2, 4, 40, 36
    N, C = Hg * Wg, 64 * H
    q, k, v = _dev(inputs.custom_qkv(B, H, N, 64, "bf16", seed=77))
    d = dwc_to_device(inputs.dwc_weights(C, 32, 3, 5), DEV)
    x = inputs.normal((B, N, C), 991, "bf16").to(DEV)
    w, b = (t.to(DEV) for t in inputs.proj_weights(3 * C, C, 992))
    wo, bo = (t.to(DEV) for t in inputs.proj_weights(C, C, 993))
    shape = jv.make_shape(q, Hg, Wg)
    ws = jv.alloc_workspace("L", shape, jv.make_dwc(d, DEV), DEV)

    def chain(sync):
        outs = []
        def done(t):
            if sync:
                torch.cuda.synchronize()
            outs.append(t)
        q1, k1, v1 = jv.qkv_proj(x, w, b, H, Hg, Wg)
        done(q1)
        o1 = jv.linear_attn(q1, k1, v1, Hg, Wg, dwc=d, ws=ws)
        done(o1)
        o2 = jv.linear_attn(q, k, v, Hg, Wg, ws=ws)              # same workspace, no convolution
        done(o2)
        o3 = jv.window_attn(q1, k1, v1, Hg, Wg, 16, 16)
        done(o3)
        o4 = jv.linear_attn(k, q, v, Hg, Wg, dwc=d, ws=ws)
        done(o4)
        o5 = jv.full_attn(q1, k1, v1)
        done(o5)
        done(jv.out_proj(o4, wo, bo, Hg, Wg))
        torch.cuda.synchronize()
        return outs

    ref = chain(sync=True)
    for rep in range(3):
        ws.fill_(0xFF)
        got = chain(sync=False)
        for i, (a, r) in enumerate(zip(got, ref)):
            assert torch.equal(a, r), (rep, i)


def test_bit_determinism(jv):
    w = inputs.WORKLOADS["dinov3_l"]
    q, k, v = _dev(inputs.custom_qkv(2, 4, 64 * 64, 64, "bf16", seed=3))
    d = dwc_to_device(inputs.dwc_weights(4 * 64, 32, 3, 7), DEV)
    for fn in (lambda: jv.linear_attn(q, k, v, 64, 64, dwc=d), lambda: jv.window_attn(q, k, v, 64, 64, 16, 16),
               lambda: jv.full_attn(q, k, v)):
        a, b = fn(), fn()
        torch.cuda.synchronize()
        assert torch.equal(a, b)


# ------------------------------------------------------------------ configs 2-5 at full size
def test_cfg2_linear_dinov3_full_size(jv, oracle):
    w = inputs.WORKLOADS["dinov3_l"]
    q, k, v = inputs.qkv(w)
    out = jv.linear_attn(*_dev((q, k, v)), w.Hg, w.Wg)
    torch.cuda.synchronize()
    assert rel_err(out, oracle.linear_attn(q, k, v, w.Hg, w.Wg)) <= TOL["bf16"]


def test_cfg2d_linear_with_dwc_full_size(jv, oracle):
    w = inputs.WORKLOADS["dinov3_l"]
    q, k, v = inputs.qkv(w)
    C = w.H * w.D
    d = inputs.dwc_weights(C, C // 8, 3, inputs.seed_for(w.cfg, 0, 3))
    out = jv.linear_attn(*_dev((q, k, v)), w.Hg, w.Wg, dwc=dwc_to_device(d, DEV))
    torch.cuda.synchronize()
    assert rel_err(out, oracle.linear_attn(q, k, v, w.Hg, w.Wg, dwc=d)) <= TOL["bf16"]


def test_cfg3_window_dinov3_full_size_sampled_heads(jv, oracle):
    w = inputs.WORKLOADS["dinov3_w"]
    q, k, v = inputs.qkv(w)
    out = jv.window_attn(*_dev((q, k, v)), w.Hg, w.Wg, 16, 16).cpu()
    for b, h in sample_heads(w.B, w.H, 32, 3):       # a quarter of the 128 (batch, head) pairs
        sl = (slice(b, b + 1), slice(h, h + 1))
        ref = oracle.window_attn(q[sl], k[sl], v[sl], w.Hg, w.Wg, 16, 16)
        assert rel_err(out[sl], ref) <= TOL["bf16"], (b, h)


def _sample_rows(N, n, seed, tail=160):
    rng = np.random.default_rng(seed)
    rows = set(rng.choice(N, size=n, replace=False).tolist())
    rows.update(range(max(0, N - tail), N, 7))      # always cover the ragged last tile
    rows.update((0, N - 1))
    return np.array(sorted(rows))


def test_cfg4_dav2_ragged_full_and_window(jv, oracle):
    w = inputs.WORKLOADS["dav2_l"]
    q, k, v = inputs.qkv(w)
    dq, dk, dv = _dev((q, k, v))
    of = jv.full_attn(dq, dk, dv, w.Hg, w.Wg).cpu()
    ow = jv.window_attn(dq, dk, dv, w.Hg, w.Wg, 16, 16).cpu()
    rows = _sample_rows(w.N, 1024, 4)
    for b, h in sample_heads(w.B, w.H, 8, 4):
        sl = (slice(b, b + 1), slice(h, h + 1))
        ref = oracle.full_attn(q[sl][:, :, rows], k[sl], v[sl])
        assert rel_err(of[sl][:, :, rows], ref) <= TOL["bf16"], ("F", b, h)
        ref = oracle.window_attn(q[sl], k[sl], v[sl], w.Hg, w.Wg, 16, 16)
        assert rel_err(ow[sl], ref) <= TOL["bf16"], ("W", b, h)


def test_cfg5_hybrid_stack_and_all_full(jv, oracle):
    w = inputs.WORKLOADS["hybrid24"]
    sched = inputs.HYBRID_SCHEDULE
    assert len(sched) == w.n_layers and [i for i, c in enumerate(sched) if c == "F"] == [5, 11, 17, 23]
    host = [inputs.qkv(w, layer=l) for l in range(w.n_layers)]
    dq, dk, dv = ([t[i].to(DEV) for t in host] for i in range(3))
    outs = jv.hybrid_mixers(sched, dq, dk, dv, w.Hg, w.Wg, 16, 16)
    torch.cuda.synchronize()
    rows = _sample_rows(w.N, 1024, 5, tail=0)        # F layers: 1024 query rows of each checked head
    for l, m in enumerate(sched):
        q, k, v = host[l]
        o = outs[l].cpu()
        for b, h in sample_heads(w.B, w.H, 2, 50 + l):
            sl = (slice(b, b + 1), slice(h, h + 1))
            if m == "L":
                err = rel_err(o[sl], oracle.linear_attn(q[sl], k[sl], v[sl], w.Hg, w.Wg))
            elif m == "W":
                err = rel_err(o[sl], oracle.window_attn(q[sl], k[sl], v[sl], w.Hg, w.Wg, 16, 16))
            else:
                err = rel_err(o[sl][:, :, rows], oracle.full_attn(q[sl][:, :, rows], k[sl], v[sl]))
            assert err <= TOL["bf16"], (l, m, b, h, err)
    del outs
    # the comparison run: the same stack with every layer F
    outs = jv.hybrid_mixers("F" * w.n_layers, dq, dk, dv, w.Hg, w.Wg, 16, 16)
    torch.cuda.synchronize()
    rows = rows[::3]
    for l in range(0, w.n_layers, 5):
        q, k, v = host[l]
        o = outs[l].cpu()
        b, h = sample_heads(w.B, w.H, 1, 80 + l)[0]
        sl = (slice(b, b + 1), slice(h, h + 1))
        assert rel_err(o[sl][:, :, rows], oracle.full_attn(q[sl][:, :, rows], k[sl], v[sl])) <= TOL["bf16"], l


def test_hybrid_small_with_dwc_layers(jv, oracle, both_paths):
    B, H, Hg, Wg, D = 1, 2, 32, 32, 64
    sched = "LWFL"
    host = [inputs.custom_qkv(B, H, Hg * Wg, D, "bf16", seed=20 + l) for l in range(4)]
    dws = [inputs.dwc_weights(H * D, 16, 3, 5), None, None, None]
    dq, dk, dv = ([t[i].to(DEV) for t in host] for i in range(3))
    outs = jv.hybrid_mixers(sched, dq, dk, dv, Hg, Wg, 16, 16,
                            dwc=[None if d is None else dwc_to_device(d, DEV) for d in dws])
    refs = oracle.hybrid_mixers(sched, [t[0] for t in host], [t[1] for t in host], [t[2] for t in host],
                                Hg, Wg, 16, 16, dwc=dws)
    for l in range(4):
        assert rel_err(outs[l], refs[l]) <= TOL["bf16"], l


def test_runtime_errors_on_device(jv):
    q, k, v = _dev(inputs.custom_qkv(1, 2, 64, 64, "f32", seed=1))
    with pytest.raises(jv.JetVitError) as e:
        jv.linear_attn(q, k, v, 8, 8, ws=torch.empty(256, dtype=torch.uint8, device=DEV))
    assert e.value.status == jv.JV_ERR_WORKSPACE
    with pytest.raises(jv.JetVitError):
        jv.window_attn(q, k, v, 8, 8, 0, 4)
    with pytest.raises(jv.JetVitError):
        jv.full_attn(q, k, v, out=q)
    assert jv.device_status() == jv.JV_OK


# ------------------------------------------------------------------ Table 1 variant: focused feature map (Eq. 3)
@pytest.mark.parametrize("dtype", ["f32", "bf16"])
@pytest.mark.parametrize("p", [2.0, 3.0, 2.5])
def test_linear_with_focused_feature_map(jv, oracle, both_paths, dtype, p):
    B, H, Hg, Wg = 2, 2, 21, 18
    q, k, v = inputs.custom_qkv(B, H, Hg * Wg, 64, dtype, seed=int(10 * p))
    d = inputs.dwc_weights(H * 64, 16, 3, 31)
    dq, dk, dv = _dev((q, k, v))
    out = jv.linear_attn_focused(dq, dk, dv, Hg, Wg, p, dwc=dwc_to_device(d, DEV))
    assert rel_err(out, oracle.linear_attn_focused(q, k, v, Hg, Wg, p, dwc=d)) <= TOL[dtype]
    out = jv.linear_attn_focused(dq, dk, dv, Hg, Wg, p)
    assert rel_err(out, oracle.linear_attn_focused(q, k, v, Hg, Wg, p)) <= TOL[dtype]


def test_focused_feature_map_full_size_and_power_one(jv, oracle):
    w = inputs.WORKLOADS["dinov3_l"]
    q, k, v = inputs.qkv(w)
    dq, dk, dv = _dev((q, k, v))
    out = jv.linear_attn_focused(dq, dk, dv, w.Hg, w.Wg, 3.0).cpu()
    for b, h in sample_heads(w.B, w.H, 6, 33):
        sl = (slice(b, b + 1), slice(h, h + 1))
        assert rel_err(out[sl], oracle.linear_attn_focused(q[sl], k[sl], v[sl], w.Hg, w.Wg, 3.0)) <= TOL["bf16"], (b, h)
    # p = 1 is the ReLU block
    assert torch.equal(jv.linear_attn_focused(dq, dk, dv, w.Hg, w.Wg, 1.0), jv.linear_attn(dq, dk, dv, w.Hg, w.Wg))


# ------------------------------------------------------------------ Table 1 variant: token-wise dynamic convolution
@pytest.mark.parametrize("dtype", ["f32", "bf16"])
@pytest.mark.parametrize("case", [(2, 2, 0, 21, 18, 3, 64), (1, 2, 5, 13, 16, 3, 64), (1, 2, 0, 9, 10, 5, 16), (1, 3, 2, 8, 8, 3, 24)],
                         ids=lambda c: "x".join(map(str, c)))
def test_linear_with_tokenwise_dynamic_dwc(jv, oracle, both_paths, dtype, case):
    """R = 64 with 3 x 3 kernels runs on the tensor-core generator (bf16); the other cases, fp32 and
    the forced-generic runs on the per-token kernels."""
    B, H, P, Hg, Wg, ksz, R = case
    q, k, v = inputs.custom_qkv(B, H, P + Hg * Wg, 64, dtype, seed=300 + Hg + R)
    d = dict(inputs.dwc_weights(H * 64, R, ksz, 301), token_wise=1)
    out, check = guarded_empty(q.shape, _dev((q,))[0].dtype, DEV)
    jv.linear_attn(*_dev((q, k, v)), Hg, Wg, dwc=dwc_to_device(d, DEV), out=out, prefix=P)
    check()
    # This variant stores the attention output, reads it back and stores the sum: two bf16 roundings,
    # sqrt(2) x 2.26e-3 rms from the stores alone, hence its own rms bar (the max-norm bar is the usual one).
    assert rel_err(out, oracle.linear_attn(q, k, v, Hg, Wg, dwc=d, prefix=P), rms_tol=4.5e-3) <= TOL[dtype]


def test_tokenwise_dynamic_dwc_larger_grid_sampled(jv, oracle):
    """64 x 64 grid, 4 heads, R = 128: the GEMM tiles of the generator run over several token and
    feature tiles; whole samples against the oracle (the generator mixes the heads of a sample)."""
    B, H, Hg, Wg, R = 2, 4, 64, 64, 128
    q, k, v = inputs.custom_qkv(B, H, Hg * Wg, 64, "bf16", seed=310)
    d = dict(inputs.dwc_weights(H * 64, R, 3, 311), token_wise=1)
    out = jv.linear_attn(*_dev((q, k, v)), Hg, Wg, dwc=dwc_to_device(d, DEV)).cpu()
    ref = oracle.linear_attn(q[1:], k[1:], v[1:], Hg, Wg, dwc=d)
    assert rel_err(out[1:], ref, rms_tol=4.5e-3) <= TOL["bf16"]
