"""Helpers of the GPU parity tests (no method arithmetic here)."""
import numpy as np
import torch

TOL = {"f32": 1e-4, "bf16": 2e-2, torch.float32: 1e-4, torch.bfloat16: 2e-2}
CANARY = 1234.5


def rel_err(o_gpu, o_ref) -> float:
    """max-abs error relative to the RMS of the oracle output."""
    g = o_gpu.detach().double().cpu().numpy() if hasattr(o_gpu, "detach") else np.asarray(o_gpu, dtype=np.float64)
    r = np.asarray(o_ref, dtype=np.float64)
    assert g.shape == r.shape, (g.shape, r.shape)
    assert np.all(np.isfinite(g)), "non-finite values in the GPU output"
    return float(np.abs(g - r).max() / np.sqrt(np.mean(r * r)))


def guarded_empty(shape, dtype, device, pad=4096):
    """Output tensor carved out of a larger buffer filled with a canary value;
    returns (view, check) where check() asserts that the guard words on both
    sides are untouched (compute-sanitizer is not available on the test pool)."""
    n = int(np.prod(shape))
    buf = torch.full((n + 2 * pad,), CANARY, dtype=dtype, device=device)
    view = buf[pad:pad + n].view(shape)

    def check():
        torch.cuda.synchronize()
        assert bool((buf[:pad] == CANARY).all()), "write before the output buffer"
        assert bool((buf[pad + n:] == CANARY).all()), "write past the output buffer"
    return view, check


def sample_heads(B, H, n, seed):
    rng = np.random.default_rng(seed)
    flat = rng.choice(B * H, size=min(n, B * H), replace=False)
    return [(int(f) // H, int(f) % H) for f in sorted(flat)]


def dwc_to_device(d, device):
    return {k: (v.to(device) if hasattr(v, "to") else v) for k, v in d.items()}
