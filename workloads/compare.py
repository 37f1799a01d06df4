"""Error metric used when a device result is compared with the oracle (no GNN arithmetic)."""
from __future__ import annotations

import numpy as np

# Largest relative error allowed: fp32 paths / paths that store bf16.
TOL = {"f32": 1e-4, "bf16": 2e-2}

# An output entry is a sum of terms (self products, neighbour products, bias).  Floating-point evaluation of
# such a sum, in any order, is off by at most c * u * D, where D is the sum of the ABSOLUTE values of the terms
# and u the unit roundoff of the accumulation: the error scales with D, not with a result that cancelled or
# that ReLU zeroed, so |ref| alone cannot be the denominator.  An entry is therefore compared relative to
# max(|ref|, FLOOR * D): plain relative error wherever |ref| >= FLOOR * D, and an absolute bound of
# tol * FLOOR * D on the entries that lost more than that to cancellation.
#   'stored': against the oracle that rounds where the layer contract stores a tensor (the gate).  What is
#             left is accumulation order and width (fp32 or 3xTF32 against fp64) and, on bf16 paths, the rare
#             stored entry that rounds the other way.
#   'exact' : against the fp64-throughout oracle, which charges every storage rounding to the device: an
#             input rounded to bf16 carries a relative error of up to 2^-9 into each of its terms.
FLOOR = {"stored": 2.0 ** -7, "exact": 2.0 ** -4}


def rel_error(got: np.ndarray, ref: np.ndarray, mag: np.ndarray | None = None, floor: float = FLOOR["stored"]) -> dict:
    """max over entries of |got - ref| / max(|ref|, floor * mag), `mag` being the oracle's term magnitudes
    (sum of |terms| of each entry, >= |ref|).  Without `mag` the root mean square of the entry's row and of the
    whole reference stand in for floor * mag (a coarser floor, for callers that have no magnitudes).
    Also returned: max_rel_plain = plain relative error over the entries with |ref| > rms(ref); max_over_mag =
    max |got - ref| / mag; max_abs; rms of the reference; finite."""
    got = np.asarray(got, dtype=np.float64)
    ref = np.asarray(ref, dtype=np.float64)
    assert got.shape == ref.shape
    if ref.size == 0:
        return {"max_rel": 0.0, "max_abs": 0.0, "rms": 0.0, "max_rel_plain": 0.0, "max_over_mag": 0.0, "finite": True}
    diff = np.abs(got - ref)
    rms = float(np.sqrt(np.mean(ref * ref)))
    out = {}
    if mag is None:
        row = np.sqrt(np.mean(ref * ref, axis=-1, keepdims=True)) if ref.ndim > 1 else rms
        den = np.maximum(np.maximum(np.abs(ref), row), max(rms, 1e-300))
        out["max_over_mag"] = None
    else:
        mag = np.asarray(mag, dtype=np.float64)
        assert mag.shape == ref.shape
        den = np.maximum(np.maximum(np.abs(ref), floor * mag), 1e-300)
        out["max_over_mag"] = float((diff / np.maximum(mag, 1e-300)).max())
    big = np.abs(ref) > rms
    out.update(max_rel=float((diff / den).max()), max_abs=float(diff.max()), rms=rms,
               max_rel_plain=float((diff[big] / np.abs(ref[big])).max()) if big.any() else 0.0,
               finite=bool(np.isfinite(got).all()))
    return out
