"""Error metrics used by the parity tests (the tolerances are stated where they are used).

fp32 I/O:  max_i |x_i - r_i| / max(|r_i|, 0.1 * rms(r))  with rms taken per (b,h) slice.
           Outputs are sums with cancellation, so a purely relative error needs a floor;
           a tenth of the slice's rms keeps the gate strict enough to reject TF32-rounded
           operands (about 1e-2 under this metric) while plain fp32 FMA sits near 1e-5.
bf16 I/O:  max_i |x_i - r_i| / max_j |r_j|  per tensor (normalised max error).
"""
import numpy as np


def _np(x):
    if hasattr(x, "detach"):
        x = x.detach().cpu().double().numpy()
    return np.asarray(x, dtype=np.float64)


def rel_err_floor(x, ref):
    x, ref = _np(x), _np(ref)
    red = tuple(range(2, ref.ndim))
    rms = np.sqrt((ref ** 2).mean(axis=red, keepdims=True)) if ref.ndim > 2 else np.sqrt((ref ** 2).mean())
    den = np.maximum(np.abs(ref), 0.1 * rms)
    den = np.where(den == 0.0, 1.0, den)
    return float((np.abs(x - ref) / den).max())


def norm_max_err(x, ref):
    x, ref = _np(x), _np(ref)
    den = np.abs(ref).max()
    return float(np.abs(x - ref).max() / (den if den > 0 else 1.0))
