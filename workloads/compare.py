"""Error metric used when a device result is compared with the oracle (no GNN arithmetic)."""
from __future__ import annotations

import numpy as np


def rel_error(got: np.ndarray, ref: np.ndarray) -> dict:
    """Element (v, f) is compared relative to max(|ref|, rms of ref row v, rms of the whole ref):
    rounding error of an fp32 / bf16 dot product scales with the size of its terms, not with
    the (possibly cancelled or ReLU-zeroed) result, so a pure |ref| denominator is unbounded."""
    got = np.asarray(got, dtype=np.float64)
    ref = np.asarray(ref, dtype=np.float64)
    assert got.shape == ref.shape
    if ref.size == 0:
        return {"max_rel": 0.0, "max_abs": 0.0, "rms": 0.0, "max_rel_plain": 0.0}
    diff = np.abs(got - ref)
    rms = float(np.sqrt(np.mean(ref * ref)))
    row = np.sqrt(np.mean(ref * ref, axis=-1, keepdims=True)) if ref.ndim > 1 else rms
    den = np.maximum(np.maximum(np.abs(ref), row), max(rms, 1e-300))
    big = np.abs(ref) > rms
    return {"max_rel": float((diff / den).max()), "max_abs": float(diff.max()), "rms": rms,
            "max_rel_plain": float((diff[big] / np.abs(ref[big])).max()) if big.any() else 0.0,
            "finite": bool(np.isfinite(got).all())}
