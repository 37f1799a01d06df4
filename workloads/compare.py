"""Error metric used when a device result is compared with the oracle (no GNN arithmetic)."""
from __future__ import annotations

import numpy as np

# Largest relative error allowed: fp32 paths / paths that store bf16.
TOL = {"f32": 1e-4, "bf16": 2e-2}

# An output entry is a sum of terms (self products, neighbour products, bias).  Floating-point evaluation of
# such a sum, in any order, is off by at most c * u * D, where D is the sum of the ABSOLUTE values of the terms
# and u the unit roundoff of whatever rounds them: the error scales with D, not with a result that cancelled or
# that ReLU zeroed, so |ref| alone cannot be the denominator.  An entry is therefore compared relative to
# max(|ref|, floor * D): plain relative error wherever |ref| >= floor * D, and an absolute bound of
# tol * floor * D on the entries that lost more than that to cancellation.  The floors, as multiples of the unit
# roundoff they allow on such an entry (u32 = 2^-24 for fp32 arithmetic, u16 = 2^-9 for a tensor stored in bf16):
#   'stored': against the oracle that rounds where the layer contract stores a tensor (the gate).
#             f32 : 2^-7 -> 1e-4 * 2^-7 D = 13 u32 D: accumulation order and width (fp32, or 3xTF32, against fp64)
#                   over a few hundred to a few thousand terms.
#             bf16: 2^-3 -> 2e-2 * 2^-3 D = 1.3 u16 D.  The device and the oracle round the same tensors, but
#                   about one stored entry in a thousand lands on the other side of a rounding boundary (their
#                   accumulations differ in the last fp32 bits), and such a one-ulp difference of a layer's
#                   aggregate or output is an input error of the next product.  Measured on the five workloads:
#                   2e-4 D after one layer, 4e-4 to 9e-4 D after two or three; on sum aggregates over hubs of
#                   hundreds of weighted edges (large rows, large ulps) up to 1.4e-3 D after two layers.
#   'exact' : against the fp64-throughout oracle, which charges EVERY storage rounding to the device: each stored
#             tensor on the way (layer input, aggregate, transformed rows, layer output) adds up to u16 to each of
#             its terms.  bf16: 2^-2 -> 2.6 u16 D (measured up to 0.8 u16 D per layer); f32: 2^-4 -> 105 u32 D.
# The figures above hold for one or two layers.  Every further layer passes its stored input through one more product
# whose terms are about ten times its result (the cancellation inside a dot product), so a difference of one ulp in a
# stored entry weighs more on the next layer's small entries than that layer's own rounding: end to end over L layers
# the floor is multiplied by max(1, L - 1) (floor_for); a layer on its own, fed the device's own input, is held to
# the unscaled floor (the per-layer checks of the tests).
FLOOR = {"stored": {"f32": 2.0 ** -7, "bf16": 2.0 ** -3}, "exact": {"f32": 2.0 ** -4, "bf16": 2.0 ** -2}}


def floor_for(mode: str, dtype: str, n_layers: int = 1) -> float:
    return min(1.0, FLOOR[mode][dtype] * max(1, n_layers - 1))


def rel_error(got: np.ndarray, ref: np.ndarray, mag: np.ndarray | None = None, floor: float = 2.0 ** -7) -> dict:
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
