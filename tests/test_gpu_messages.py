"""Layers with learned messages (the general apply_edge: m = w_e act_edge([h_u | e_vu] W_edge + b_edge), Eq. (1))
against the CPU oracle, through the C ABI: every reduce and GCN, both storage types, with and without edge
features and edge weights, on split and unsplit graphs, stacked, and the argument checks."""
import numpy as np
import pytest
import torch

from gpu_util import check_against_oracle, make_gat_layer, make_msg_layer, make_sage_layer, run_device, small_workload
from paper_2307_00228_b200 import binding as B
from paper_2307_00228_b200 import host

pytestmark = pytest.mark.gpu

HUBS = (257, 300, 1000, 2500, 33, 32, 9, 8, 1)


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
@pytest.mark.parametrize("op", ["sum", "mean", "max", "min", "gcn"])
@pytest.mark.parametrize("edge_dim", [0, 8])
@pytest.mark.parametrize("threshold", [0, 64])
def test_message_layer_parity(dtype, op, edge_dim, threshold):
    layer = make_msg_layer(1, op, "relu", 32, 32, 64, dtype, act_edge="elu", weights=(op in ("sum", "max")), edge_dim=edge_dim)
    w = small_workload(2, 1500, 30, dtype, [layer], hubs=HUBS, weights=True, threshold=threshold, edge_dim=edge_dim)
    got, d = run_device(w)
    if threshold:
        assert d.n_split_owners > 0
    check_against_oracle(w, got, label=(dtype, op, edge_dim, threshold))


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
@pytest.mark.parametrize("dims", [(16, 8, 16, 24), (64, 16, 128, 32), (24, 40, 48, 16), (128, 32, 64, 128)])
def test_message_shapes(dtype, dims):
    """(in_dim, edge_dim, msg_dim, out_dim): message rows of several widths, K that is not a whole number of k-blocks."""
    fi, de, fm, fo = dims
    layer = make_msg_layer(3, "sum", "none", fi, fm, fo, dtype, act_edge="relu", edge_dim=de)
    w = small_workload(4, 700, 14, dtype, [layer], hubs=(300, 40), threshold=128, edge_dim=de)
    got, _ = run_device(w)
    check_against_oracle(w, got, label=(dtype, dims))


def test_message_layers_stack_with_plain_layers():
    layers = [make_msg_layer(5, "mean", "relu", 32, 64, 32, "f32", act_edge="relu", edge_dim=8),
              make_sage_layer(6, "sum", "relu", 32, 32, "f32", edge_dim=8),
              make_msg_layer(7, "max", "none", 32, 16, 16, "f32", act_edge="elu", edge_dim=8)]
    w = small_workload(8, 900, 10, "f32", layers, hubs=(200,), threshold=64, edge_dim=8)
    got, d = run_device(w)
    check_against_oracle(w, got)
    # it_infer is the sequence of it_layer_forward calls
    h = d.x
    for lay, src in zip(d.layers, w.layers):
        o = torch.empty((w.n, src.out_dim), device="cuda")
        B.it_layer_forward(d.graph, lay, h, o, d.workspace)
        h = o
    torch.cuda.synchronize()
    assert torch.equal(h, d.out)


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
@pytest.mark.parametrize("threshold", [0, 100])
@pytest.mark.parametrize("heads,hd,de", [(2, 16, 8), (4, 32, 16), (1, 8, 8)])
def test_gat_with_edge_features_in_the_logits(dtype, threshold, heads, hd, de):
    """e = LeakyReLU(a_src . z_u + a_dst . z_v + a_edge . e_vu): split and unsplit, all row kernels (hubs up to 2500 edges)."""
    layer = make_gat_layer(21, "elu", 32, heads, hd, dtype, edge_dim=de)
    w = small_workload(22, 1300, 25, dtype, [layer], hubs=HUBS, threshold=threshold, edge_dim=de)
    got, d = run_device(w)
    if threshold:
        assert d.n_split_owners > 0
    check_against_oracle(w, got, label=(dtype, threshold, heads, hd, de))


def test_gat_edge_logits_change_the_result_and_stack():
    layers = [make_gat_layer(23, "elu", 32, 2, 16, "f32", edge_dim=8), make_gat_layer(24, "none", 32, 2, 8, "f32", edge_dim=8)]
    w = small_workload(25, 800, 12, "f32", layers, hubs=(300,), threshold=64, edge_dim=8)
    got, _ = run_device(w)
    check_against_oracle(w, got)
    plain = [make_gat_layer(23, "elu", 32, 2, 16, "f32"), make_gat_layer(24, "none", 32, 2, 8, "f32")]
    for a, b in zip(plain, layers):   # the same parameters without the edge term
        a.W, a.bias, a.att_src, a.att_dst = b.W, b.bias, b.att_src, b.att_dst
    w2 = small_workload(25, 800, 12, "f32", plain, hubs=(300,), threshold=64)
    base, _ = run_device(w2)
    assert np.abs(got - base).max() > 1e-3


def test_message_argument_checks():
    layer = make_msg_layer(9, "sum", "none", 16, 16, 16, "f32", edge_dim=8)
    w = small_workload(10, 100, 5, "f32", [layer], edge_dim=8)
    d = host.upload(w)
    out = torch.empty((w.n, 16), device="cuda")

    def status_of(fn):
        with pytest.raises(B.ItError) as ei:
            fn()
        return ei.value.status_name

    bad = host.layer_to_device(make_msg_layer(11, "sum", "none", 16, 6, 16, "f32", edge_dim=8), "f32")   # 24-byte message rows
    assert status_of(lambda: B.it_workspace_bytes(d.graph, [bad])) == "IT_ERR_INVALID_ARG"
    no_w = host.layer_to_device(layer, "f32")
    no_w.W_edge = None
    assert status_of(lambda: B.it_layer_forward(d.graph, no_w, d.x, out, d.workspace)) == "IT_ERR_INVALID_ARG"
    gat = host.layer_to_device(layer, "f32")
    gat.op = "gat"
    gat.edge_dim = 0
    assert status_of(lambda: B.it_workspace_bytes(d.graph, [gat])) == "IT_ERR_UNSUPPORTED"   # learned messages are not for GAT
    g2 = host.layer_to_device(make_gat_layer(12, "none", 16, 2, 8, "f32", edge_dim=8), "f32")
    g2.att_edge = None
    ws = torch.empty(B.it_workspace_bytes(d.graph, [g2]), dtype=torch.uint8, device="cuda")
    assert status_of(lambda: B.it_layer_forward(d.graph, g2, d.x, out, ws)) == "IT_ERR_INVALID_ARG"
    assert torch.ones(3, device="cuda").sum().item() == 3
