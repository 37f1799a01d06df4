"""The stage calls (it_layer_transform / it_layer_gather / it_layer_update), graph parts and the vertex-partitioned
pass on one GPU: the stages reproduce it_layer_forward bit for bit, and several workers run one after another in
one process (tables concatenated in place of the all-gather, partial results reduced in place of the
reduce-scatter) reproduce the unsharded pass and the oracle."""
import numpy as np
import pytest
import torch

from gpu_util import (TOL, assert_close, check_against_oracle, check_each_layer, make_gat_layer, make_msg_layer, make_plain_layer, make_sage_layer,
                      run_device, run_oracle, small_workload, to_numpy)
from paper_2307_00228_b200 import binding as B
from paper_2307_00228_b200 import host, sharded

pytestmark = pytest.mark.gpu


def layer_cases(dtype):
    return {
        "sage": make_sage_layer(1, "mean", "relu", 32, 32, dtype),
        "sage_reorder": make_sage_layer(2, "sum", "none", 64, 16, dtype, weights=True),
        "max": make_sage_layer(3, "max", "relu", 32, 32, dtype, weights=True),
        "gcn": make_plain_layer(4, "gcn", "relu", 32, 32, dtype, weights=True),
        "gcn_reorder": make_plain_layer(5, "gcn", "none", 64, 32, dtype),
        "gat": make_gat_layer(6, "elu", 32, 2, 16, dtype),
        "dense": make_plain_layer(7, "dense", "relu", 32, 64, dtype),
        "msg": make_msg_layer(8, "sum", "relu", 32, 32, 32, dtype, act_edge="relu", weights=True),
    }


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
@pytest.mark.parametrize("kind", ["sage", "sage_reorder", "max", "gcn", "gcn_reorder", "gat", "dense", "msg"])
def test_stage_calls_reproduce_layer_forward(dtype, kind):
    layer = layer_cases(dtype)[kind]
    w = small_workload(10, 1500, 20, dtype, [layer], hubs=(900, 300, 40), weights=True, threshold=128)
    d = host.upload(w)
    lay = d.layers[0]
    ref = torch.empty((w.n, layer.out_dim), dtype=d.x.dtype, device="cuda")
    B.it_layer_forward(d.graph, lay, d.x, ref, d.workspace)
    sd = B.it_layer_stages(d.graph, lay)
    table, scores = d.x, None
    if not sd["table_is_input"]:
        table = torch.empty((w.n, sd["table_dim"]), dtype=d.x.dtype, device="cuda")
        scores = torch.empty((w.n, sd["score_dim"]), device="cuda") if sd["score_dim"] else None
        B.it_layer_transform(d.graph, lay, d.x, table, scores, d.workspace)
    out = torch.full_like(ref, float("nan"))
    if sd["table_dim"] == 0:
        B.it_layer_update(d.graph, lay, d.x, None, out, d.workspace)
    elif sd["agg_dim"] == 0:
        B.it_layer_gather(d.graph, lay, table, scores, 0, False, out, d.workspace)
    else:
        agg = torch.empty((w.n, sd["agg_dim"]), dtype=d.x.dtype, device="cuda")
        B.it_layer_gather(d.graph, lay, table, scores, 0, False, agg, d.workspace)
        B.it_layer_update(d.graph, lay, d.x, agg, out, d.workspace)
    B.it_graph_check(d.graph)
    assert torch.equal(out, ref)


def emulate(w, world, layout, threshold=None):
    eng = sharded.CudaEngine(threshold=w.threshold if threshold is None else threshold)
    ranges = sharded.vertex_ranges(w.n, world)
    x = host.features_to_device(w.x, w.dtype)
    workers = [sharded.Worker(r, world, w.indptr, w.indices, w.edge_weights, x[v0:v1], w.layers, w.dtype, eng, layout=layout)
               for r, (v0, v1) in enumerate(ranges)]
    out = sharded.run_emulated(workers)
    torch.cuda.synchronize()
    for wk in workers:
        B.it_graph_check(wk.part)
    return out


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
@pytest.mark.parametrize("world", [1, 2, 3])
def test_destination_partition_reproduces_the_unsharded_pass(dtype, world):
    """Every layer kind in one model; a part gathers from the all-gathered table of all workers."""
    L = layer_cases(dtype)
    layers = [L["dense"], make_sage_layer(11, "mean", "relu", 64, 64, dtype), make_sage_layer(12, "sum", "relu", 64, 32, dtype, weights=True),
              L["gat"], L["gcn"], L["max"]]
    w = small_workload(13, 1201, 15, dtype, layers, hubs=(700, 300, 40), weights=True, threshold=64)
    whole, d = run_device(w)
    if world == 1:
        check_each_layer(w, d, label=dtype)
    got = to_numpy(emulate(w, world, "gather"))
    check_against_oracle(w, got, label=(dtype, world), exact=False)
    if world == 1:
        assert np.array_equal(got, whole)
    else:   # a part buckets its own rows, so a sum may be taken in another order: close, not identical
        assert np.allclose(got, whole, rtol=TOL[dtype], atol=TOL[dtype])


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
@pytest.mark.parametrize("op", ["sum", "mean", "max", "min", "gcn"])
def test_source_partition_with_reduced_partial_results(dtype, op):
    """Partial-gather across workers: raw fp32 partial results of every destination, reduced, finished, updated."""
    mk = make_plain_layer if op == "gcn" else make_sage_layer
    layers = [mk(14, op, "relu", 32, 32, dtype, weights=(op != "mean")), mk(15, op, "none", 32, 16, dtype)]
    w = small_workload(16, 1003, 12, dtype, layers, hubs=(800, 200), weights=True, threshold=64)
    got = to_numpy(emulate(w, 3, "partial"))
    for l in w.layers:
        l.allow_reorder = False    # layers that run as a partial-gather keep the plain order
    outs, mags = run_oracle(w, magnitudes=True)
    assert_close(got, outs[-1], mags[-1], dtype, "stored", label=(dtype, op), n_layers=2)
    if op in ("max", "min"):   # exact reduces: the partition cannot change a bit
        whole, _ = run_device(w)
        assert np.array_equal(got, whole)


def test_part_graph_checks():
    layer = make_sage_layer(17, "sum", "relu", 16, 16, "f32")
    w = small_workload(18, 100, 5, "f32", [layer])
    ip, ix, _ = sharded.destination_part(w.indptr, w.indices, None, 20, 60)
    g = B.it_graph_create_part(torch.from_numpy(ip).cuda(), torch.from_numpy(ix).cuda(), 100)
    lay = host.layer_to_device(layer, "f32")
    ws = torch.empty(B.it_workspace_bytes(g, [lay]), dtype=torch.uint8, device="cuda")
    x = torch.zeros((100, 16), device="cuda")
    out = torch.empty((40, 16), device="cuda")

    def status_of(fn):
        with pytest.raises(B.ItError) as ei:
            fn()
        return ei.value.status_name

    # a part is not a whole graph: the one-call forms refuse it
    assert status_of(lambda: B.it_layer_forward(g, lay, x, out, ws)) == "IT_ERR_INVALID_ARG"
    # source ids beyond the table are a bad graph
    assert status_of(lambda: B.it_graph_create_part(torch.from_numpy(ip).cuda(), torch.from_numpy(ix).cuda(), 50)) == "IT_ERR_BAD_GRAPH"
    # raw partial results only from layers that gather their input
    gat = host.layer_to_device(make_gat_layer(19, "none", 16, 2, 8, "f32"), "f32")
    wsg = torch.empty(B.it_workspace_bytes(g, [gat]), dtype=torch.uint8, device="cuda")
    raw = torch.empty((40, 16), device="cuda")
    assert status_of(lambda: B.it_layer_gather(g, gat, x, torch.zeros((100, 4), device="cuda"), 20, True, raw, wsg)) == "IT_ERR_UNSUPPORTED"
    assert status_of(lambda: B.it_layer_gather(g, gat, x, torch.zeros((100, 4), device="cuda"), 90, False, raw, wsg)) == "IT_ERR_INVALID_ARG"
    assert torch.ones(2, device="cuda").sum().item() == 2
