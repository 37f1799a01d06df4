"""The seeded input generators: determinism, exact sizes, structure."""
import numpy as np

from workloads import graphs, make, rng as wrng


def test_tiny_is_deterministic_and_exact():
    a, b = make("tiny"), make("tiny")
    assert a.n == 10_000 and a.e == 100_000 and a.indptr[-1] == a.e
    for k in ("indptr", "indices", "x"):
        assert np.array_equal(getattr(a, k), getattr(b, k))
    assert np.array_equal(a.layers[0].W, b.layers[0].W)
    deg = np.diff(a.indptr)
    assert deg.min() >= 0 and deg.max() <= 2000 and deg.max() > a.threshold
    assert a.indices.min() >= 0 and a.indices.max() < a.n and a.indices.dtype == np.int32
    # sources ascending inside each segment
    d = np.diff(a.indices.astype(np.int64))
    starts = a.indptr[1:-1][np.diff(a.indptr)[1:] > 0]
    mask = np.ones(a.e - 1, bool)
    mask[starts[(starts > 0) & (starts < a.e)] - 1] = False
    assert np.all(d[mask] >= 0)
    assert [(l.in_dim, l.out_dim, l.op, l.act) for l in a.layers] == [(64, 64, "mean", "relu"), (64, 16, "mean", "none")]
    lim = np.sqrt(6.0 / (128 + 64))
    assert np.abs(a.layers[0].W).max() <= lim and np.abs(a.layers[0].W).max() > 0.9 * lim


def test_power_law_tail_and_mean():
    deg = graphs.power_law_degrees(wrng.stream(1), 200_000, 4_000_000, 2.1, 20_000)
    assert deg.sum() == 4_000_000 and deg.max() <= 20_000
    # heavy tail: a few vertices hold a large share of the edges; the median is far below the mean
    assert np.median(deg) < 8 and np.sort(deg)[-2000:].sum() > 0.3 * deg.sum()


def test_scaled_configs_have_the_right_models():
    m = make("medium", 0.005)
    assert m.dtype == "f32" and m.edge_weights is not None and m.threshold == 1024
    assert m.x.shape == (m.n, 128) and m.layers[0].use_edge_weights and m.layers[1].out_dim == 64
    g = make("gat", 0.002)
    assert g.dtype == "bf16" and g.x.dtype == np.uint16 and g.layers[0].heads == 4 and g.layers[0].act == "elu"
    assert g.layers[0].att_src.shape == (4, 32) and g.threshold == 4096
    # bf16 parameters are exactly representable
    W = g.layers[0].W
    assert np.array_equal(wrng.bf16_bits_to_f32(wrng.f32_to_bf16_bits(W)), W)
    x = make("extreme", 0.001)
    deg = np.diff(x.indptr)
    assert (deg == 1000).sum() >= 4 and x.e == 200_000 and len(x.layers) == 3 and x.layers[0].op == "max"


def test_bf16_helpers_round_to_nearest_even():
    f = np.array([1.0, 1.00390625, 1.01171875, -2.5, 0.0], np.float32)   # 1+2^-8 (tie->1), 1+3*2^-8 (tie->1+2^-6)
    back = wrng.bf16_bits_to_f32(wrng.f32_to_bf16_bits(f))
    assert back.tolist() == [1.0, 1.0, 1.015625, -2.5, 0.0]
