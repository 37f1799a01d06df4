"""Parity of the CUDA layer pass with the CPU oracle, element by element, through the C ABI."""
import numpy as np
import pytest
import torch

from gpu_util import (TOL, assert_close, check_against_oracle, check_each_layer, make_gat_layer, make_plain_layer, make_sage_layer, run_device, run_oracle,
                      small_workload, to_numpy)
from paper_2307_00228_b200 import binding as B
from paper_2307_00228_b200 import host
from workloads import compare

pytestmark = pytest.mark.gpu

HUBS = (257, 300, 1000, 2500, 33, 32, 9, 8, 1)


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
@pytest.mark.parametrize("op", ["sum", "mean", "max", "min"])
@pytest.mark.parametrize("weights", [False, True])
@pytest.mark.parametrize("threshold", [0, 64, 1000])
def test_sage_layer_parity(dtype, op, weights, threshold):
    # 1500 vertices: several 128-row GEMM tiles and a ragged tail; every degree bucket is populated
    fi, fo = 64, 32
    for reorder in ([False, True] if op in ("sum", "mean") else [False]):
        layer = make_sage_layer(1, op, "relu", fi, fo, dtype, weights=weights, allow_reorder=reorder)
        w = small_workload(2, 1500, 40, dtype, [layer], hubs=HUBS, weights=weights, threshold=threshold)
        got, d = run_device(w)
        if threshold:
            assert d.n_split_owners > 0
        check_against_oracle(w, got, label=(dtype, op, weights, threshold, reorder))


@pytest.mark.parametrize("dtype,dims", [("f32", (4, 4)), ("f32", (8, 16)), ("f32", (16, 8)), ("f32", (32, 64)), ("f32", (128, 128)),
                                        ("f32", (128, 64)), ("bf16", (8, 8)), ("bf16", (16, 64)), ("bf16", (64, 128)),
                                        ("bf16", (128, 64)), ("bf16", (256, 32))])
def test_every_supported_row_width(dtype, dims):
    fi, fo = dims
    for op in ("mean", "max", "min"):
        layer = make_sage_layer(3, op, "none", fi, fo, dtype)
        w = small_workload(4, 700, 20, dtype, [layer], hubs=(400, 90), threshold=128)
        got, _ = run_device(w)
        check_against_oracle(w, got, label=(dtype, dims, op))


@pytest.mark.parametrize("dtype,dims", [("f32", (100, 48)), ("f32", (12, 20)), ("f32", (256, 64)), ("f32", (192, 192)),
                                        ("f32", (52, 100)), ("bf16", (768, 64)), ("bf16", (40, 24)), ("bf16", (200, 96)),
                                        ("bf16", (104, 128))])
def test_rows_of_any_multiple_of_16_bytes(dtype, dims):
    """Widths the kernels do not take directly (the paper's datasets have 50-, 100- and 768-entry features) are
    gathered in column chunks; a K that is not a whole number of GEMM k-blocks is padded with zeros."""
    fi, fo = dims
    for op, weights in (("sum", True), ("mean", False), ("max", False)):
        layer = make_sage_layer(3, op, "relu", fi, fo, dtype, weights=weights)
        w = small_workload(4, 700, 20, dtype, [layer], hubs=(400, 90), weights=weights, threshold=128)
        got, d = run_device(w)
        assert d.n_split_owners > 0
        check_against_oracle(w, got, label=(dtype, dims, op))
    gcn = make_plain_layer(5, "gcn", "none", fi, fo, dtype, weights=True)
    w = small_workload(6, 500, 15, dtype, [gcn], hubs=(300,), weights=True, threshold=64)
    got, _ = run_device(w)
    check_against_oracle(w, got, label=(dtype, dims, "gcn"))


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
@pytest.mark.parametrize("act", ["none", "relu", "elu"])
def test_gat_layer_parity(dtype, act):
    layer = make_gat_layer(5, act, 64, 4, 32, dtype)
    w = small_workload(6, 1300, 30, dtype, [layer], hubs=HUBS)
    got, _ = run_device(w)
    check_against_oracle(w, got, label=(dtype, act))


@pytest.mark.parametrize("heads,hd", [(1, 8), (2, 16), (8, 8), (1, 128), (4, 32)])
def test_gat_head_shapes(heads, hd):
    layer = make_gat_layer(7, "elu", 32, heads, hd, "bf16")
    w = small_workload(8, 500, 12, "bf16", [layer], hubs=(300, 40))
    got, _ = run_device(w)
    check_against_oracle(w, got, label=(heads, hd))


def test_gat_large_scores_do_not_overflow():
    """Attention logits of +-100 and more: exp() of them overflows fp32, the running maximum keeps the softmax
    finite.  The logits are fp32 by contract, so a softmax weight carries a relative error of about
    |logit| * 2^-23 (1e-5 here): the plain fp32 tolerance still holds."""
    layer = make_gat_layer(9, "none", 16, 2, 8, "f32")
    layer.att_src *= 60.0
    layer.att_dst *= 60.0
    w = small_workload(10, 400, 25, "f32", [layer], hubs=(300,))
    z = w.x_as_f32() @ layer.W
    logits = np.abs(z.reshape(w.n, 2, 8) * layer.att_src[None]).sum(-1)
    assert logits.max() > 100.0, "the case must reach logits whose exp overflows fp32"
    got, _ = run_device(w)
    assert np.isfinite(got).all()
    check_against_oracle(w, got)


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
@pytest.mark.parametrize("threshold", [16, 100, 3000])
def test_gat_on_a_split_graph(dtype, threshold):
    """Online-softmax states merge associatively, so the groups of a split hub are reduced on their
    own and merged in group order; the result is still the plain per-destination softmax."""
    layer = make_gat_layer(9, "elu", 32, 2, 16, dtype)
    w = small_workload(10, 1200, 25, dtype, [layer], hubs=(5000, 2100, 300, 40), threshold=threshold)
    got, d = run_device(w)
    assert d.n_split_owners > 0
    check_against_oracle(w, got, label=(dtype, threshold))
    base, _ = run_device(w, threshold=0)
    assert compare.rel_error(got, base)["max_rel"] <= TOL[dtype]


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
@pytest.mark.parametrize("dims", [(64, 32), (32, 64), (128, 128), (8, 16)])
@pytest.mark.parametrize("act", ["none", "elu"])
def test_dense_layer_parity(dtype, dims, act):
    """No Gather stage (initial transform / prediction part): the graph must not matter."""
    fi, fo = dims
    layer = make_plain_layer(40, "dense", act, fi, fo, dtype)
    w = small_workload(41, 1300, 10, dtype, [layer], hubs=(300,), threshold=64)
    got, _ = run_device(w)
    check_against_oracle(w, got, label=(dtype, dims, act))


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
@pytest.mark.parametrize("weights", [False, True])
@pytest.mark.parametrize("threshold", [0, 64])
def test_gcn_layer_parity(dtype, weights, threshold):
    for fi, fo in ((64, 32), (32, 64), (64, 64)):      # the first shape reorders (transform before aggregate)
        for reorder in (True, False):
            layer = make_plain_layer(42, "gcn", "relu", fi, fo, dtype, weights=weights, allow_reorder=reorder)
            w = small_workload(43, 1500, 30, dtype, [layer], hubs=HUBS, weights=weights, threshold=threshold)
            got, d = run_device(w)
            check_against_oracle(w, got, label=(dtype, weights, threshold, fi, fo, reorder))


def test_embed_gnn_predict_pipeline():
    """Initial transform of raw features, two message-passing layers, prediction head: the k-layer GNN
    from raw vertex states to scores in one it_infer call."""
    for dtype in ("f32", "bf16"):
        layers = [make_plain_layer(44, "dense", "relu", 24 if dtype == "f32" else 40, 64, dtype),
                  make_sage_layer(45, "mean", "relu", 64, 64, dtype),
                  make_plain_layer(46, "gcn", "relu", 64, 32, dtype, weights=True),
                  make_plain_layer(47, "dense", "none", 32, 8, dtype)]
        w = small_workload(48, 2500, 18, dtype, layers, hubs=HUBS, weights=True, threshold=200)
        got, d = run_device(w)
        check_against_oracle(w, got, label=dtype)
        check_each_layer(w, d, label=dtype)


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
def test_multi_layer_infer_matches_layer_by_layer_and_oracle(dtype):
    layers = [make_sage_layer(11, "mean", "relu", 32, 64, dtype), make_sage_layer(12, "sum", "relu", 64, 32, dtype, weights=True),
              make_sage_layer(13, "max", "none", 32, 16, dtype)]
    w = small_workload(14, 2100, 16, dtype, layers, hubs=HUBS, weights=True, threshold=100)
    got, d = run_device(w)
    check_against_oracle(w, got)
    check_each_layer(w, d, label=dtype)
    # exactly the sequence of it_layer_forward calls: bit-identical
    h = d.x
    for lay, src in zip(d.layers, w.layers):
        ws = torch.empty(B.it_workspace_bytes(d.graph, [lay]), dtype=torch.uint8, device="cuda")
        o = torch.empty((w.n, src.out_dim), dtype=d.x.dtype, device="cuda")
        B.it_layer_forward(d.graph, lay, h, o, ws)
        h = o
    torch.cuda.synchronize()
    assert torch.equal(h, d.out)


def test_run_to_run_results_are_bit_identical():
    """The paper's consistency requirement: the same prediction at every run."""
    layers = [make_sage_layer(15, "sum", "relu", 64, 64, "f32", weights=True), make_sage_layer(16, "mean", "none", 64, 16, "f32")]
    w = small_workload(17, 3000, 30, "f32", layers, hubs=HUBS, weights=True, threshold=64)
    d = host.upload(w)
    outs = []
    for _ in range(4):
        d.out.zero_()
        d.workspace.random_(0, 255)          # stale scratch must not matter
        d.infer()
        torch.cuda.synchronize()
        outs.append(d.out.clone())
    assert all(torch.equal(outs[0], o) for o in outs[1:])


def test_split_does_not_change_max_min_and_integer_sums():
    """Partial gather + combine: exact for max and min, and for sums of small integers."""
    lay_max = make_sage_layer(18, "max", "none", 32, 32, "f32")
    lay_min = make_sage_layer(18, "min", "none", 32, 32, "f32")
    lay_sum = make_sage_layer(19, "sum", "none", 32, 32, "f32")
    for lay in (lay_max, lay_min, lay_sum):
        lay.W[:] = 0
        lay.W[32:] = np.eye(32, dtype=np.float32)   # output = the aggregate itself
        lay.bias = None
        w = small_workload(20, 900, 25, "f32", [lay], hubs=(2000, 513))
        w.x = np.round(w.x * 4).astype(np.float32)
        base, _ = run_device(w, threshold=0)
        for T in (1, 7, 64, 512):
            got, _ = run_device(w, threshold=T)
            assert np.array_equal(got, base), (lay.op, T)
        assert np.array_equal(base, run_oracle(w, storage=None)[-1])


def test_int32_and_int64_indptr_agree():
    layer = make_sage_layer(21, "mean", "relu", 64, 64, "bf16")
    w = small_workload(22, 1000, 20, "bf16", [layer], hubs=(600,), threshold=128)
    a, _ = run_device(w, int32_indptr=False)
    b, _ = run_device(w, int32_indptr=True)
    assert np.array_equal(a, b)


def test_degenerate_inputs():
    layer = make_sage_layer(23, "mean", "relu", 16, 16, "f32")
    # no edges at all: output = act(x W_self + b)
    w = small_workload(24, 300, 0, "f32", [layer])
    assert w.e == 0
    got, _ = run_device(w)
    check_against_oracle(w, got)
    # a single vertex with a self-loop and a multi-edge
    w = small_workload(25, 1, 0, "f32", [layer])
    w.indptr = np.array([0, 3], np.int64)
    w.indices = np.zeros(3, np.int32)
    w.e = 3
    got, _ = run_device(w)
    check_against_oracle(w, got)
    # every vertex has exactly one in-edge
    w = small_workload(26, 257, 1, "f32", [layer], p_zero=0.0)
    got, _ = run_device(w)
    check_against_oracle(w, got)


def test_error_statuses():
    layer = make_sage_layer(27, "sum", "relu", 16, 16, "f32", weights=True)
    w = small_workload(28, 100, 5, "f32", [layer], weights=True)
    d = host.upload(w)
    out = torch.empty((w.n, 16), device="cuda")

    def status_of(fn):
        with pytest.raises(B.ItError) as ei:
            fn()
        return ei.value.status_name

    small = torch.empty(256, dtype=torch.uint8, device="cuda")
    assert status_of(lambda: B.it_layer_forward(d.graph, d.layers[0], d.x, out, small)) == "IT_ERR_WORKSPACE"
    assert status_of(lambda: B.it_layer_forward(d.graph, d.layers[0], d.x, d.x, d.workspace)) == "IT_ERR_INVALID_ARG"
    misaligned = d.workspace[1:]
    assert status_of(lambda: B.it_layer_forward(d.graph, d.layers[0], d.x, out, misaligned)) == "IT_ERR_WORKSPACE"
    # matrices that are not 16-byte aligned are refused on the host (the kernels move 16-byte slices)
    flat = torch.empty(w.n * 16 + 4, device="cuda")
    off4 = flat[1:1 + w.n * 16].view(w.n, 16)
    assert off4.data_ptr() % 16 == 4
    assert status_of(lambda: B.it_layer_forward(d.graph, d.layers[0], off4, out, d.workspace)) == "IT_ERR_INVALID_ARG"
    assert status_of(lambda: B.it_layer_forward(d.graph, d.layers[0], d.x, off4, d.workspace)) == "IT_ERR_INVALID_ARG"
    assert status_of(lambda: B.it_layer_forward_static(d.graph, d.layers[0], off4, out)) == "IT_ERR_INVALID_ARG"
    assert status_of(lambda: B.it_infer(d.graph, d.layers, off4, out, d.workspace)) == "IT_ERR_INVALID_ARG"
    assert status_of(lambda: B.it_infer(d.graph, d.layers, d.x, off4, d.workspace)) == "IT_ERR_INVALID_ARG"
    # input or output inside the workspace, or on top of each other
    inside = d.workspace[:w.n * 16 * 4].view(torch.float32).view(w.n, 16)
    assert status_of(lambda: B.it_infer(d.graph, d.layers, inside, out, d.workspace)) == "IT_ERR_INVALID_ARG"
    assert status_of(lambda: B.it_infer(d.graph, d.layers, d.x, inside, d.workspace)) == "IT_ERR_INVALID_ARG"
    assert status_of(lambda: B.it_infer(d.graph, d.layers, d.x, d.x, d.workspace)) == "IT_ERR_INVALID_ARG"
    bad = host.layer_to_device(make_sage_layer(29, "sum", "relu", 6, 16, "f32"), "f32")   # 24-byte rows
    assert status_of(lambda: B.it_workspace_bytes(d.graph, [bad])) == "IT_ERR_INVALID_ARG"
    mism = [d.layers[0], host.layer_to_device(make_sage_layer(30, "sum", "relu", 32, 16, "f32"), "f32")]
    assert status_of(lambda: B.it_workspace_bytes(d.graph, mism)) == "IT_ERR_INVALID_ARG"
    # edge weights requested from a graph that has none
    w2 = small_workload(28, 100, 5, "f32", [layer], weights=False)
    assert status_of(lambda: host.upload(w2)) == "IT_ERR_INVALID_ARG"
    assert torch.ones(4, device="cuda").sum().item() == 4


def test_exact_oracle_bounds_both_storage_types():
    """Against the fp64-throughout oracle (no rounding at storage points, plain order of operations) a two-layer
    pass stays within the tolerance of its storage type, entry by entry."""
    for dtype in ("bf16", "f32"):
        layers = [make_sage_layer(31, "mean", "relu", 64, 64, dtype), make_sage_layer(32, "mean", "none", 64, 32, dtype)]
        w = small_workload(33, 2000, 20, dtype, layers, hubs=(700,), threshold=256)
        got, _ = run_device(w)
        outs, mags = run_oracle(w, storage=None, magnitudes=True)
        err = assert_close(got, outs[-1], mags[-1], dtype, "exact", label=dtype)
        print(dtype, err)


@pytest.mark.parametrize("dtype,fi", [("bf16", 64), ("bf16", 128), ("f32", 32), ("f32", 64)])
@pytest.mark.parametrize("max_deg", [3, 8])
def test_buckets_of_very_short_rows(dtype, fi, max_deg):
    """Rows of 128 and 256 bytes with at most 8 edges: when the bucket's rows hold at most 4 edges on average the
    launch keeps two rows per lane group in flight (max_deg 3), otherwise one (max_deg 8).  Every reduce, with and
    without edge weights, the transform-first epilogue, a hub that is split, and more rows than one sweep of the grid."""
    for op, weights, fo in (("mean", False, fi), ("sum", True, fi), ("max", False, fi), ("min", True, fi),
                            ("mean", False, fi // 2), ("sum", True, fi // 2)):
        layer = make_sage_layer(7, op, "relu", fi, fo, dtype, weights=weights)
        w = small_workload(8, 4000, max_deg, dtype, [layer], hubs=(300,), weights=weights, threshold=128, p_zero=0.1)
        got, d = run_device(w)
        B.it_graph_check(d.graph)
        check_against_oracle(w, got, label=(dtype, fi, max_deg, op, weights, fo))


def test_very_short_rows_beyond_one_sweep_of_the_grid():
    """More rows of at most 3 edges than the resident lane groups of the whole GPU take in one sweep (148 SMs x 3
    CTAs x 32 lane groups), so that every lane group walks several rows and the row records loaded ahead run past
    the end of the bucket."""
    layer = make_sage_layer(9, "mean", "none", 64, 64, "bf16")
    w = small_workload(10, 60_000, 3, "bf16", [layer], p_zero=0.05)
    got, d = run_device(w)
    B.it_graph_check(d.graph)
    check_against_oracle(w, got)
