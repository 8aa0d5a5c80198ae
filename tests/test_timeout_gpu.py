"""The bounded waits of the tensor-core kernels, driven to their limit without hanging or
faulting anything: jv_selftest_wait_timeout enqueues a one-warp kernel that waits (through the
mixers' own bounded wait, limit 1 ms) on a barrier nothing completes.  Checked: the wait gives
up and the kernel returns; jv_device_status reports JV_ERR_TIMEOUT once and JV_OK afterwards;
tensor-core mixer calls enqueued while the status word is set leave their output untouched
(the behaviour include/jetvit.h documents); the next calls compute correctly."""
import pytest
import torch

from paper_2605_26636_b200 import inputs
from tests._util import TOL, dwc_to_device, rel_err

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


@pytest.fixture(scope="module")
def jv():
    from paper_2605_26636_b200 import jetvit
    jetvit.lib()
    return jetvit


def test_a_wait_that_runs_out_sets_the_status_and_nothing_hangs(jv, oracle):
    Hg, Wg = 40, 32                                   # N = 1280: F runs on the four-tile kernel
    qh, kh, vh = inputs.custom_qkv(1, 2, Hg * Wg, 64, "bf16", seed=31)
    q, k, v = (t.to(DEV) for t in (qh, kh, vh))
    qs, ks, vs = (t[:, :, :512].contiguous() for t in (q, k, v))    # 512 tokens: F on the two-tile kernel
    dh = inputs.dwc_weights(2 * 64, 16, 3, 32)
    d = dwc_to_device(dh, DEV)
    calls = {
        "L": lambda out: jv.linear_attn(q, k, v, Hg, Wg, out=out),
        "L+dwc": lambda out: jv.linear_attn(q, k, v, Hg, Wg, dwc=d, out=out),
        "W": lambda out: jv.window_attn(q, k, v, Hg, Wg, 16, 16, out=out),
        "F": lambda out: jv.full_attn(q, k, v, out=out),
        "F short": lambda out: jv.full_attn(qs, ks, vs, out=out.view(-1)[:qs.numel()].view(qs.shape)),
    }
    assert jv.device_status() == jv.JV_OK
    good = {}
    for name, fn in calls.items():
        good[name] = torch.empty_like(q)
        fn(good[name])
    assert jv.device_status() == jv.JV_OK

    gave_up = torch.zeros(1, dtype=torch.int32, device=DEV)
    t0, t1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    t0.record()
    jv.selftest_wait_timeout(1000, gave_up)           # 1 ms
    t1.record()
    # calls enqueued while the status word is set: their kernels leave at once, o keeps the canary
    outs = {}
    for name, fn in calls.items():
        outs[name] = torch.full_like(q, 1234.5)
        fn(outs[name])
    torch.cuda.synchronize()
    assert int(gave_up.item()) == 1
    assert 0.9 <= t0.elapsed_time(t1) < 200.0         # the wait lasted about its limit, not the 2 s default
    for name, o in outs.items():
        assert bool((o == 1234.5).all()), f"{name}: output written while the status word was set"
    assert jv.device_status() == jv.JV_ERR_TIMEOUT    # reported once ...
    assert jv.device_status() == jv.JV_OK             # ... and cleared
    # the context is intact and the next calls compute what they computed before, and what the oracle says
    for name, fn in calls.items():
        o = torch.full_like(q, 1234.5)
        fn(o)
        torch.cuda.synchronize()
        n = qs.numel() if name == "F short" else q.numel()
        assert torch.equal(o.view(-1)[:n], good[name].view(-1)[:n]), name
    assert rel_err(good["L+dwc"], oracle.linear_attn(qh, kh, vh, Hg, Wg, dwc=dh)) <= TOL["bf16"]
    assert rel_err(good["F"], oracle.full_attn(qh, kh, vh)) <= TOL["bf16"]
    assert jv.device_status() == jv.JV_OK


def test_selftest_rejects_bad_limits(jv):
    with pytest.raises(jv.JetVitError):
        jv.selftest_wait_timeout(0)
    with pytest.raises(jv.JetVitError):
        jv.selftest_wait_timeout(5_000_000)
    assert jv.device_status() == jv.JV_OK
