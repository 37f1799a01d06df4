"""The layer pass with the edge arrays kept in page-locked host memory and streamed through two staging buffers, one
block of destinations at a time, against the same blocks held resident (bit for bit) and against the oracle."""
import numpy as np
import pytest
import torch

from gpu_util import check_against_oracle, make_gat_layer, make_plain_layer, make_sage_layer, small_workload, to_numpy
from paper_2307_00228_b200 import binding as B
from paper_2307_00228_b200 import host, sharded, streamed
from workloads import make

pytestmark = pytest.mark.gpu


def resident_blocks(w, n_blocks):
    eng = sharded.CudaEngine(threshold=w.threshold)
    x = host.features_to_device(w.x, w.dtype)
    ws = [sharded.Worker(b, n_blocks, w.indptr, w.indices, w.edge_weights, x[v0:v1], w.layers, w.dtype, eng)
          for b, (v0, v1) in enumerate(sharded.vertex_ranges(w.n, n_blocks))]
    out = sharded.run_emulated(ws)
    torch.cuda.synchronize()
    return out


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
@pytest.mark.parametrize("block", [97, 400, 5000])
def test_streamed_pass_equals_the_resident_blocks_and_the_oracle(dtype, block):
    layers = [make_sage_layer(1, "mean", "relu", 32, 32, dtype), make_sage_layer(2, "sum", "relu", 32, 16, dtype, weights=True),
              make_gat_layer(3, "elu", 16, 2, 8, dtype), make_plain_layer(4, "gcn", "none", 16, 16, dtype, weights=True)]
    w = small_workload(5, 1301, 14, dtype, layers, hubs=(900, 300, 40), weights=True, threshold=64)
    sp = streamed.StreamedPass(w.indptr, w.indices, w.edge_weights, host.features_to_device(w.x, w.dtype), w.layers, w.dtype,
                               block_vertices=block, threshold=w.threshold)
    first = sp.infer().clone()
    second = sp.infer()          # every block is streamed in again
    torch.cuda.synchronize()
    for wk in sp.workers:
        B.it_graph_check(wk.part)
    assert torch.equal(first, second)
    assert torch.equal(first, resident_blocks(w, sp.n_blocks))
    check_against_oracle(w, to_numpy(first), label=(dtype, block), exact=False)
    if sp.n_blocks > 2:
        assert sp.staging_bytes < sp.edge_bytes and sp.engine.h2d_bytes > 0


def test_streamed_medium_shape():
    """A twentieth of the Medium workload in 16 blocks: the staging buffers hold an eighth of the edge arrays."""
    w = make("medium", 0.05)
    sp = streamed.StreamedPass(w.indptr, w.indices, w.edge_weights, host.features_to_device(w.x, w.dtype), w.layers, w.dtype,
                               block_vertices=-(-w.n // 16), threshold=w.threshold)
    out = sp.infer()
    torch.cuda.synchronize()
    assert sp.staging_bytes * 4 < sp.edge_bytes
    check_against_oracle(w, to_numpy(out), exact=False)
