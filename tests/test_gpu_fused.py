"""it_infer where the update of one layer and the transform of the next run as one kernel (bf16 layers whose widths
are multiples of 64, the second one transforming before it aggregates): the intermediate layer output is never
stored, and the result is the one of the layer-by-layer pass bit for bit, and the oracle's within the tolerance."""
import numpy as np
import pytest
import torch

from gpu_util import check_against_oracle, make_plain_layer, make_sage_layer, small_workload, to_numpy
from paper_2307_00228_b200 import binding as B
from paper_2307_00228_b200 import host

pytestmark = pytest.mark.gpu


def layer_by_layer(d, w):
    """The same model as a chain of it_layer_forward calls (every layer output stored)."""
    h = d.x
    for lay, src in zip(d.layers, w.layers):
        o = torch.empty((w.n, src.out_dim), dtype=d.x.dtype, device="cuda")
        B.it_layer_forward(d.graph, lay, h, o, d.workspace)
        h = o
    return h


def models():
    s = make_sage_layer
    p = make_plain_layer
    return {
        # the shape of the largest workload: GraphSAGE-mean 64 -> 128 -> 64
        "sage_64_128_64": [s(1, "mean", "relu", 64, 128, "bf16"), s(2, "mean", "none", 128, 64, "bf16")],
        "sage_sum_128_128_64_weights": [s(3, "sum", "relu", 128, 128, "bf16", weights=True), s(4, "sum", "none", 128, 64, "bf16", weights=True)],
        "sage_elu_64_256_64": [s(5, "mean", "elu", 64, 256, "bf16"), s(6, "mean", "relu", 256, 64, "bf16")],
        "max_then_reorder": [s(7, "max", "relu", 64, 128, "bf16"), s(8, "sum", "none", 128, 64, "bf16")],
        "gcn_then_gcn_reorder": [p(9, "gcn", "relu", 64, 128, "bf16", weights=True), p(10, "gcn", "none", 128, 64, "bf16", weights=True)],
        "dense_then_reorder": [p(11, "dense", "relu", 64, 128, "bf16"), s(12, "mean", "none", 128, 64, "bf16")],
        "edge_features_then_reorder": [s(13, "sum", "relu", 64, 128, "bf16", edge_dim=16), s(14, "mean", "none", 128, 64, "bf16")],
        # two pairs in one model, and a layer in front that belongs to no pair
        "four_layers_two_pairs": [s(15, "mean", "relu", 64, 128, "bf16"), s(16, "mean", "relu", 128, 64, "bf16"),
                                  s(17, "max", "relu", 64, 128, "bf16"), s(18, "sum", "none", 128, 64, "bf16")],
        "three_layers_pair_last": [s(19, "max", "relu", 64, 64, "bf16"), s(20, "mean", "relu", 64, 128, "bf16"), s(21, "mean", "none", 128, 64, "bf16")],
        # shapes the fused kernel does not take run layer by layer inside it_infer
        "not_fused_32_wide": [s(22, "mean", "relu", 64, 64, "bf16"), s(23, "mean", "none", 64, 32, "bf16")],
        "not_fused_96_wide": [s(24, "mean", "relu", 64, 128, "bf16"), s(25, "mean", "none", 128, 96, "bf16")],
    }


@pytest.mark.parametrize("name", list(models()))
@pytest.mark.parametrize("n", [1000, 5003])
def test_infer_with_fused_pairs_equals_layer_by_layer_and_the_oracle(name, n):
    layers = models()[name]
    edge_dim = 16 if "edge_features" in name else 0
    w = small_workload(30, n, 24, "bf16", layers, hubs=(700, 90), weights=True, threshold=128, edge_dim=edge_dim)
    d = host.upload(w)
    d.infer()
    B.it_graph_check(d.graph)
    got = d.out.clone()
    ref = layer_by_layer(d, w)
    B.it_graph_check(d.graph)
    assert torch.equal(got, ref)
    check_against_oracle(w, to_numpy(got), label=name)


def test_fused_pair_is_one_kernel_and_stores_no_intermediate():
    """Instrumentation names the kernels of a pass: the pair runs as gemm2_tc, with no separate gemm_tc launch."""
    w = small_workload(31, 3000, 16, "bf16", models()["sage_64_128_64"])
    d = host.upload(w)
    d.infer()
    B.it_profile_begin()
    d.infer()
    torch.cuda.synchronize()
    names = {s["name"]: s["launches"] for s in B.it_profile_end()}
    assert names.get("gemm2_tc") == 1 and "gemm_tc" not in names


def test_tail_tile_and_single_tile():
    """Fewer rows than one tile, and a last tile of one row."""
    for n in (7, 129):
        w = small_workload(32, n, 5, "bf16", models()["sage_64_128_64"])
        d = host.upload(w)
        d.infer()
        B.it_graph_check(d.graph)
        assert torch.equal(d.out, layer_by_layer(d, w))
        check_against_oracle(w, to_numpy(d.out))


def test_fused_pair_replays_from_a_cuda_graph():
    """it_infer with a fused pair captured in a CUDA graph on a side stream (the library allocates nothing and
    synchronises nothing inside it_infer): the replay writes the same result bit for bit."""
    w = small_workload(33, 3000, 16, "bf16", models()["sage_64_128_64"], hubs=(500,), threshold=128)
    d = host.upload(w)
    d.infer()
    torch.cuda.synchronize()
    eager = d.out.clone()
    side = torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.stream(side):
        d.infer(stream=side)
        side.synchronize()
        with torch.cuda.graph(graph, stream=side):
            d.infer(stream=side)
    torch.cuda.synchronize()
    for _ in range(3):
        d.out.zero_()
        graph.replay()
        torch.cuda.synchronize()
        assert torch.equal(d.out, eager)
    B.it_graph_check(d.graph)
