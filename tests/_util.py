"""Helpers of the GPU parity tests (no method arithmetic here)."""
import os

import numpy as np
import torch

TOL = {"f32": 1e-4, "bf16": 2e-2, torch.float32: 1e-4, torch.bfloat16: 2e-2}
CANARY = 1234.5
RMS_TOL_BF16 = 3e-3     # bf16 outputs: rms(error) / rms(oracle), no allowance (see rel_err)


PARITY_LOG = []      # one record per bf16 comparison of this session (written out by conftest.py)


def _bf16_round(r: np.ndarray) -> np.ndarray:
    return torch.from_numpy(np.ascontiguousarray(r)).to(torch.bfloat16).double().numpy()


def rel_err(o_gpu, o_ref, plain: bool = False, rms_tol: float = None) -> float:
    """Parity metric: max-abs error relative to the RMS of the oracle output.

    fp32 outputs: exactly that.  bf16 outputs: the kernels compute in fp32 and
    round the result to bf16 (nearest-even) when storing it; that last rounding
    alone moves an element by up to 2^-8 |o_i|, which on peaked softmax rows
    (|o|max / rms reaches 14 in 16x16 windows) exceeds 2e-2 rms even for the exact
    result (tests/test_oracle_pins.py::test_bf16_store_floor shows it on the
    oracle output itself).  So for bf16 outputs the storage rounding 2^-8 |r_i|
    (r = the oracle value) is allowed on top, element by element, and the remainder
    is held to 2e-2 rms by the caller.  ``plain=True`` returns the metric without
    that allowance.

    Every bf16 comparison is also held to a second bar that involves no allowance, on
    the root-mean-square error instead of the maximum: rms(g - r) <= RMS_TOL_BF16 rms(r).
    Rounding an exact result to bf16 alone gives at most 2^-7 / sqrt(12) = 2.26e-3 there
    (an error uniform over one unit in the last place), so the bar leaves the arithmetic
    about 2e-3 rms(r) of systematic error before it trips.  The plain maximum metric, the
    one with the allowance, the rms figure and the plain metric of the oracle output
    itself rounded to bf16 all go into PARITY_LOG."""
    is_bf16 = hasattr(o_gpu, "dtype") and o_gpu.dtype == torch.bfloat16
    g = o_gpu.detach().double().cpu().numpy() if hasattr(o_gpu, "detach") else np.asarray(o_gpu, dtype=np.float64)
    r = np.asarray(o_ref, dtype=np.float64)
    assert g.shape == r.shape, (g.shape, r.shape)
    assert np.all(np.isfinite(g)), "non-finite values in the GPU output"
    d = np.abs(g - r)
    rms = np.sqrt(np.mean(r * r))
    e_plain = float(d.max() / rms)
    if not is_bf16 or plain:
        return e_plain
    e_adj = float(np.maximum(d - 2.0 ** -8 * np.abs(r), 0.0).max() / rms)
    floor = float(np.abs(_bf16_round(r) - r).max() / rms)
    e_rms = float(np.sqrt(np.mean(d * d)) / rms)
    PARITY_LOG.append({"test": os.environ.get("PYTEST_CURRENT_TEST", "").split(" ")[0], "shape": list(r.shape),
                       "plain": e_plain, "adjusted": e_adj, "floor": floor, "rms": e_rms})
    rms_tol = RMS_TOL_BF16 if rms_tol is None else rms_tol    # (a path that stores its output twice passes its own bar)
    assert e_rms <= rms_tol, f"rms error {e_rms:.3e} rms(oracle) > {rms_tol}"
    return e_adj


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
