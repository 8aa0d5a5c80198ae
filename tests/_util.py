"""Helpers of the GPU parity tests (no method arithmetic here)."""
import numpy as np
import torch

TOL = {"f32": 1e-4, "bf16": 2e-2, torch.float32: 1e-4, torch.bfloat16: 2e-2}
CANARY = 1234.5


def rel_err(o_gpu, o_ref, plain: bool = False) -> float:
    """Parity metric: max-abs error relative to the RMS of the oracle output.

    fp32 outputs: exactly that.  bf16 outputs: the kernels compute in fp32 and
    round the result to bf16 (nearest-even) when storing it; that last rounding
    alone moves an element by up to 2^-8 |o_i|, which on peaked softmax rows
    (|o|max / rms reaches 14 in 16x16 windows) exceeds 2e-2 rms even for the exact
    result (tests/test_oracle_pins.py::test_bf16_store_floor shows it on the
    oracle output itself).  So for bf16 outputs the storage rounding 2^-8 |o_i| is
    allowed on top, element by element, and the remainder is held to 2e-2 rms.
    ``plain=True`` returns the metric without that allowance."""
    is_bf16 = hasattr(o_gpu, "dtype") and o_gpu.dtype == torch.bfloat16
    g = o_gpu.detach().double().cpu().numpy() if hasattr(o_gpu, "detach") else np.asarray(o_gpu, dtype=np.float64)
    r = np.asarray(o_ref, dtype=np.float64)
    assert g.shape == r.shape, (g.shape, r.shape)
    assert np.all(np.isfinite(g)), "non-finite values in the GPU output"
    d = np.abs(g - r)
    if is_bf16 and not plain:
        d = np.maximum(d - 2.0 ** -8 * np.maximum(np.abs(r), np.abs(g)), 0.0)
    return float(d.max() / np.sqrt(np.mean(r * r)))


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
