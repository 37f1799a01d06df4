"""Parity of layers whose messages carry edge features (Eq. (1): e_{v,u}; message [w_e h_u | e_vu]) with the
CPU oracle, through the C ABI: every reduce, both storage types, split and unsplit, every edge-row width,
GCN, multi-layer inference, and the argument checks."""
import numpy as np
import pytest
import torch

from gpu_util import TOL, assert_close, check_against_oracle, make_plain_layer, make_sage_layer, run_device, small_workload, to_numpy
from oracle import oracle as O
from paper_2307_00228_b200 import binding as B
from paper_2307_00228_b200 import host
from workloads import compare, make, with_edge_features
from workloads import rng as wrng

pytestmark = pytest.mark.gpu

HUBS = (257, 300, 1000, 2500, 33, 32, 9, 8, 1)


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
@pytest.mark.parametrize("op", ["sum", "mean", "max", "min"])
@pytest.mark.parametrize("threshold", [0, 64])
def test_sage_layer_with_edge_features(dtype, op, threshold):
    # aggregate row = 64 + 32 entries: a whole number of GEMM k-blocks for fp32, not for bf16 (CUDA-core path)
    layer = make_sage_layer(1, op, "relu", 64, 32, dtype, weights=(op == "sum"), edge_dim=32)
    w = small_workload(2, 1500, 40, dtype, [layer], hubs=HUBS, weights=(op == "sum"), threshold=threshold, edge_dim=32)
    got, d = run_device(w)
    if threshold:
        assert d.n_split_owners > 0
    check_against_oracle(w, got, label=(dtype, op, threshold))


@pytest.mark.parametrize("dtype,fi,de", [("f32", 32, 4), ("f32", 64, 64), ("f32", 128, 128), ("f32", 16, 8),
                                         ("bf16", 64, 8), ("bf16", 64, 64), ("bf16", 128, 128), ("bf16", 32, 256),
                                         ("f32", 100, 12), ("bf16", 72, 40)])
def test_every_edge_row_width(dtype, fi, de):
    for op in ("mean", "max"):
        layer = make_sage_layer(3, op, "none", fi, 32, dtype, edge_dim=de)
        w = small_workload(4, 700, 20, dtype, [layer], hubs=(400, 90), threshold=128, edge_dim=de)
        got, _ = run_device(w)
        check_against_oracle(w, got, label=(dtype, fi, de, op))


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
def test_gcn_layer_with_edge_features(dtype):
    layer = make_plain_layer(5, "gcn", "elu", 64, 32, dtype, weights=True, edge_dim=64)
    w = small_workload(6, 1300, 30, dtype, [layer], hubs=HUBS, weights=True, threshold=100, edge_dim=64)
    got, d = run_device(w)
    assert d.n_split_owners > 0
    check_against_oracle(w, got, label=dtype)


def test_edge_feature_layers_are_not_reordered_and_stack():
    """Two layers, the second shrinking (it would be reordered without edge features); it_infer = layer by layer."""
    layers = [make_sage_layer(7, "sum", "relu", 64, 64, "f32", edge_dim=32),
              make_sage_layer(8, "mean", "none", 64, 16, "f32", edge_dim=32)]
    w = small_workload(9, 1100, 25, "f32", layers, hubs=(900, 200), threshold=256, edge_dim=32)
    got, d = run_device(w)
    check_against_oracle(w, got)
    h = torch.empty((w.n, 64), device="cuda")
    o = torch.empty((w.n, 16), device="cuda")
    B.it_layer_forward(d.graph, d.layers[0], d.x, h, d.workspace)
    B.it_layer_forward(d.graph, d.layers[1], h, o, d.workspace)
    torch.cuda.synchronize()
    assert torch.equal(o, d.out)


def test_medium_shape_with_edge_features_sampled():
    """A quarter of the Medium workload with 32 edge features per message, checked on sampled vertices."""
    w = with_edge_features(make("medium", 0.25), 32)
    d = host.upload(w)
    d.infer()
    B.it_graph_check(d.graph)
    deg = np.diff(w.indptr)
    targets = np.unique(np.concatenate([np.argsort(-deg, kind="stable")[:3],
                                        np.random.default_rng(5).choice(w.n, size=200, replace=False)]))
    ids, cip, cix, cw, ct, cef = O.compact_neighbourhood(w.indptr, w.indices, w.edge_weights, targets, len(w.layers),
                                                         edge_feat=w.edge_feat)
    got = to_numpy(d.out[torch.from_numpy(targets).cuda()])
    for mode, storage in (("stored", w.dtype), ("exact", None)):
        ref, mag = O.infer_at(cip, cix, cw, w.x[ids], w.layers, ct, storage=storage, threshold=w.threshold,
                              follow_reorder=storage is not None, edge_feat=cef, magnitudes=True)
        assert_close(got, ref, mag, w.dtype, mode, n_layers=len(w.layers))
    first = d.out.clone()
    d.infer()
    torch.cuda.synchronize()
    assert torch.equal(first, d.out)


def test_argument_checks():
    layer = make_sage_layer(1, "sum", "none", 16, 16, "f32", edge_dim=8)
    w = small_workload(2, 50, 5, "f32", [layer], edge_dim=8)
    d = host.upload(w)
    o = torch.empty((w.n, 16), device="cuda")
    B.it_graph_set_edge_features(d.graph, None)
    with pytest.raises(B.ItError) as e:
        B.it_layer_forward(d.graph, d.layers[0], d.x, o, d.workspace)
    assert e.value.status_name == "IT_ERR_INVALID_ARG"
    wrong = torch.zeros((w.e, 4), device="cuda")
    B.it_graph_set_edge_features(d.graph, wrong)
    with pytest.raises(B.ItError):
        B.it_layer_forward(d.graph, d.layers[0], d.x, o, d.workspace)
    with pytest.raises(B.ItError):   # a row of 12 bytes
        B.it_graph_set_edge_features(d.graph, torch.zeros((w.e, 3), device="cuda"))
    gat = B.LayerDesc(op="gat", act="none", in_dim=16, out_dim=16, W=torch.zeros((16, 16), device="cuda"), heads=2,
                      att_src=torch.zeros((2, 8), device="cuda"), att_dst=torch.zeros((2, 8), device="cuda"), edge_dim=4)
    # a GAT layer may read the edge features in its logits, but then it needs the attention vector for them
    ws = torch.empty(B.it_workspace_bytes(d.graph, [gat]), dtype=torch.uint8, device="cuda")
    with pytest.raises(B.ItError) as e:
        B.it_layer_forward(d.graph, gat, d.x, o, ws)
    assert e.value.status_name == "IT_ERR_INVALID_ARG"
    dense = B.LayerDesc(op="dense", act="none", in_dim=16, out_dim=16, W=torch.zeros((16, 16), device="cuda"), edge_dim=4)
    with pytest.raises(B.ItError) as e:
        B.it_workspace_bytes(d.graph, [dense])
    assert e.value.status_name == "IT_ERR_UNSUPPORTED"
