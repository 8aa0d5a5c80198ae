"""Full attention at head_dim 128 on its tensor-core kernel (two query tiles per CTA, tiles held as two
64-channel halves), against the float64 CPU oracle: one tile, odd and even tile counts with ragged last
tiles, a long sequence, several heads and batch elements, inputs read in place from a fused
[B, N, 3, H, D] activation, prefix tokens (folded into the token axis by F), the schedule driver, and
the same shapes on the shape-generic kernels."""
import pytest
import torch

from paper_2605_26636_b200 import inputs
from tests._util import TOL, guarded_empty, rel_err, sample_heads

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


CASES = [  # B, H, N
    (1, 1, 128),       # one tile, one step pair
    (1, 2, 129),       # two tiles, the second with one token
    (2, 3, 300),       # three tiles: the last item of a head holds one
    (1, 2, 1000),      # eight tiles, ragged
    (1, 1, 2048),      # sixteen whole tiles
]


@pytest.mark.parametrize("case", CASES, ids=lambda c: "x".join(map(str, c)))
def test_full_attention_head_dim_128(jv, oracle, both_paths, case):
    B, H, N = case
    if both_paths and N > 1000:
        pytest.skip("the generic kernel is covered by the shorter cases")
    q, k, v = inputs.custom_qkv(B, H, N, 128, "bf16", seed=12800 + N)
    out, check = guarded_empty(q.shape, torch.bfloat16, DEV)
    out.fill_(float("nan"))
    jv.full_attn(*(t.to(DEV) for t in (q, k, v)), out=out)
    check()
    assert rel_err(out, oracle.full_attn(q, k, v)) <= TOL["bf16"], case


def test_head_dim_128_long_sequence_sampled_heads(jv, oracle):
    B, H, N = 2, 4, 4096 + 77
    q, k, v = inputs.custom_qkv(B, H, N, 128, "bf16", seed=12999)
    launches = jv.launch_count()
    out = jv.full_attn(*(t.to(DEV) for t in (q, k, v))).cpu()
    assert jv.launch_count() == launches + 1
    for b, h in sample_heads(B, H, 3, 5):
        sl = (slice(b, b + 1), slice(h, h + 1))
        assert rel_err(out[sl], oracle.full_attn(q[sl], k[sl], v[sl])) <= TOL["bf16"], (b, h)


def test_head_dim_128_strided_inputs_prefix_and_driver(jv, oracle):
    B, H, Hg, Wg, P = 2, 2, 20, 24, 5
    N = P + Hg * Wg
    q, k, v = inputs.custom_qkv(B, H, N, 128, "bf16", seed=12777)
    qkv = torch.stack([t.permute(0, 2, 1, 3) for t in (q, k, v)], dim=2).contiguous().to(DEV)   # [B, N, 3, H, D]
    sq, sk, sv = (qkv[:, :, i].permute(0, 2, 1, 3) for i in range(3))
    ref = oracle.full_attn(q, k, v)
    strided = jv.full_attn(sq, sk, sv)
    assert rel_err(strided, ref) <= TOL["bf16"]
    plain = jv.full_attn(*(t.to(DEV) for t in (q, k, v)))
    assert torch.equal(strided, plain)
    (drv,) = jv.hybrid_mixers("F", [sq], [sk], [sv], Hg, Wg, 8, 8, prefix=P)
    assert torch.equal(drv, plain)
