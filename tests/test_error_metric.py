"""The error metric of the parity gate and the term magnitudes it rests on (CPU only).

layer_magnitude is pinned against what it is by definition: a bound of |output| for every layer kind, equal to
the output itself when no term can cancel (non-negative inputs and parameters), and unchanged by the sign of
any input.  The metric is pinned by planting mistakes in the ORACLE's result (never in the CUDA path): a
dropped term, a transposed weight block and a wrong sign must all fail the fp32 gate, while rounding noise of
the size the arithmetic produces must pass."""
from types import SimpleNamespace as NS

import numpy as np
import pytest

from oracle import oracle as O
from workloads import compare


def layer(op, act, fi, fo, rng, heads=1, edge_dim=0, nonneg=False, weights=False):
    k = fi + edge_dim if op in ("gat", "dense", "gcn") else 2 * fi + edge_dim
    W = rng.uniform(-1, 1, (k, fo))
    b = rng.uniform(-0.5, 0.5, fo)
    a_s = rng.uniform(-1, 1, (heads, fo // heads))
    a_d = rng.uniform(-1, 1, (heads, fo // heads))
    if nonneg:
        W, b = np.abs(W), np.abs(b)
    return NS(op=op, act=act, in_dim=fi, out_dim=fo, W=W, bias=b, heads=heads, att_src=a_s, att_dst=a_d, leaky_slope=0.2,
              use_edge_weights=weights, allow_reorder=True, edge_dim=edge_dim)


def graph(rng, n, max_deg):
    deg = rng.integers(0, max_deg + 1, size=n)
    ip = np.zeros(n + 1, np.int64)
    np.cumsum(deg, out=ip[1:])
    ix = rng.integers(0, n, size=int(ip[-1])).astype(np.int32)
    return ip, ix


OPS = ["sum", "mean", "max", "min", "gcn", "dense", "gat"]


@pytest.mark.parametrize("op", OPS)
@pytest.mark.parametrize("act", ["none", "relu", "elu"])
def test_magnitude_bounds_the_output(op, act):
    rng = np.random.default_rng(hash((op, act)) % 1000)
    ip, ix = graph(rng, 60, 9)
    w = rng.uniform(-1, 1, ix.size)
    H = rng.standard_normal((60, 8))
    lay = layer(op, act, 8, 8, rng, heads=2 if op == "gat" else 1, weights=op != "gat" and op != "dense")
    out = O.layer_forward(ip, ix, w, H, lay)
    D = O.layer_magnitude(ip, ix, w, H, lay)
    assert D.shape == out.shape and (D >= 0).all()
    assert (np.abs(out) <= D * (1 + 1e-12) + 1e-300).all()


@pytest.mark.parametrize("op", OPS)
def test_magnitude_equals_the_output_when_nothing_cancels(op):
    rng = np.random.default_rng(7)
    ip, ix = graph(rng, 50, 7)
    w = rng.uniform(0, 1, ix.size)
    H = np.abs(rng.standard_normal((50, 8)))
    lay = layer(op, "none", 8, 4, rng, heads=2 if op == "gat" else 1, nonneg=True, weights=op not in ("gat", "dense"))
    if op == "min":   # the bound of a min is the largest |term|, which is what max pooling returns on these inputs
        lay_max = NS(**{**lay.__dict__, "op": "max"})
        ref = O.layer_forward(ip, ix, w, H, lay_max)
    else:
        ref = O.layer_forward(ip, ix, w, H, lay)
    assert np.allclose(O.layer_magnitude(ip, ix, w, H, lay), ref, rtol=1e-13, atol=0)


@pytest.mark.parametrize("op", ["sum", "mean", "max", "gcn", "dense"])
def test_magnitude_ignores_signs(op):
    rng = np.random.default_rng(11)
    ip, ix = graph(rng, 40, 6)
    w = rng.uniform(-1, 1, ix.size)
    H = rng.standard_normal((40, 8))
    lay = layer(op, "relu", 8, 4, rng, weights=op != "dense")
    D = O.layer_magnitude(ip, ix, w, H, lay)
    flipped = NS(**{**lay.__dict__, "W": -lay.W, "bias": -lay.bias})
    assert np.array_equal(D, O.layer_magnitude(ip, ix, -w, -H, flipped))


def test_magnitude_with_edge_features_and_rows_subset():
    rng = np.random.default_rng(13)
    ip, ix = graph(rng, 40, 6)
    H = rng.standard_normal((40, 8))
    ef = rng.standard_normal((ix.size, 4))
    lay = layer("sum", "none", 8, 4, rng, edge_dim=4)
    D = O.layer_magnitude(ip, ix, None, H, lay, edge_feat=ef)
    out = O.layer_forward(ip, ix, None, H, lay, edge_feat=ef)
    assert (np.abs(out) <= D * (1 + 1e-12)).all()
    rows = np.array([3, 17, 39])
    assert np.allclose(O.layer_magnitude(ip, ix, None, H, lay, rows=rows, edge_feat=ef), D[rows], rtol=1e-13)
    glay = layer("gat", "none", 8, 8, rng, heads=2)
    Dg = O.layer_magnitude(ip, ix, None, H, glay)
    assert np.allclose(O.layer_magnitude(ip, ix, None, H, glay, rows=rows), Dg[rows], rtol=1e-13)


def test_infer_returns_the_magnitudes_of_every_layer_and_infer_at_agrees():
    rng = np.random.default_rng(17)
    ip, ix = graph(rng, 50, 6)
    X = rng.standard_normal((50, 8))
    layers = [layer("mean", "relu", 8, 8, rng), layer("sum", "none", 8, 4, rng)]
    outs, mags = O.infer(ip, ix, None, X, layers, magnitudes=True)
    assert np.array_equal(mags[0], O.layer_magnitude(ip, ix, None, X, layers[0]))
    assert np.array_equal(mags[1], O.layer_magnitude(ip, ix, None, outs[0], layers[1]))
    t = np.array([5, 0, 44])
    o_at, m_at = O.infer_at(ip, ix, None, X, layers, t, magnitudes=True)
    assert np.allclose(o_at, outs[1][t], rtol=1e-13) and np.allclose(m_at, mags[1][t], rtol=1e-13)


# ----------------------------------------------------------------------------- the metric itself

def sage_case(seed=3, n=400, fi=64, fo=32):
    rng = np.random.default_rng(seed)
    ip, ix = graph(rng, n, 20)
    X = rng.standard_normal((n, fi))
    lay = layer("sum", "relu", fi, fo, rng)
    lay.W *= np.sqrt(6.0 / (2 * fi + fo))
    return ip, ix, X, lay


def test_rounding_noise_passes_and_planted_mistakes_fail_the_fp32_gate():
    ip, ix, X, lay = sage_case()
    ref = O.layer_forward(ip, ix, None, X, lay)
    D = O.layer_magnitude(ip, ix, None, X, lay)
    tol, floor = compare.TOL["f32"], compare.FLOOR["stored"]["f32"]
    # an fp32 evaluation of the same layer: every product and sum rounded to fp32
    A = O.aggregate(ip, ix, None, X, "sum").astype(np.float32)
    pre = (X.astype(np.float32) @ lay.W[:64].astype(np.float32) + A @ lay.W[64:].astype(np.float32) + lay.bias.astype(np.float32))
    got = np.maximum(pre, 0).astype(np.float64)
    err = compare.rel_error(got, ref, D, floor)
    assert err["max_rel"] <= tol and err["max_rel_plain"] <= tol and err["max_over_mag"] < 1e-6
    # planted in the oracle's result: one neighbour term of one column dropped, self / neighbour blocks swapped,
    # the sign of the bias flipped
    Wd = lay.W.copy(); Wd[64 + 5, :] = 0.0
    Ws = np.concatenate([lay.W[64:], lay.W[:64]])
    for bad in (NS(**{**lay.__dict__, "W": Wd}), NS(**{**lay.__dict__, "W": Ws}), NS(**{**lay.__dict__, "bias": -lay.bias})):
        wrong = O.layer_forward(ip, ix, None, X, bad)
        e = compare.rel_error(wrong, ref, D, floor)
        assert e["max_rel"] > 100 * tol, e
        # the bf16 gate (its own floor and tolerance) sees them too
        assert compare.rel_error(wrong, ref, D, compare.FLOOR["stored"]["bf16"])["max_rel"] > compare.TOL["bf16"], e


def test_entries_that_cancelled_are_held_to_the_floor_not_to_their_own_size():
    ref = np.array([[1.0, 1e-9, -2.0, 0.0]])
    mag = np.array([[4.0, 4.0, 4.0, 4.0]])
    got = ref + np.array([[0.0, 1e-7, 0.0, 1e-7]])
    e = compare.rel_error(got, ref, mag, 2.0 ** -7)
    assert e["max_rel"] == pytest.approx(1e-7 / (4.0 / 128), rel=1e-12)
    # an error of that size on an entry that did not cancel is a plain relative error
    e2 = compare.rel_error(ref + np.array([[0, 0, 2e-3, 0]]), ref, mag, 2.0 ** -7)
    assert e2["max_rel"] == pytest.approx(1e-3, rel=1e-9) and e2["max_rel_plain"] == pytest.approx(1e-3, rel=1e-9)
    # the floor is a fraction of the magnitudes: a lower floor is a stricter gate
    assert compare.rel_error(got, ref, mag, 2.0 ** -10)["max_rel"] > e["max_rel"]


def test_bf16_storage_rounding_stays_inside_the_bf16_gate_against_the_exact_oracle():
    """Inputs, aggregate and output rounded to bf16 (what a bf16 path stores), everything else exact: against the
    fp64-throughout oracle that is inside 2e-2 with the 'exact' floor."""
    ip, ix, X, lay = sage_case(seed=5, n=600, fi=128, fo=64)
    Xb = O.round_bf16(X)
    lay.W = O.round_bf16(lay.W)
    ref = O.layer_forward(ip, ix, None, Xb, lay)
    D = O.layer_magnitude(ip, ix, None, Xb, lay)
    got = O.layer_forward(ip, ix, None, Xb, lay, storage="bf16")
    e = compare.rel_error(got, ref, D, compare.FLOOR["exact"]["bf16"])
    assert e["max_rel"] <= compare.TOL["bf16"], e
