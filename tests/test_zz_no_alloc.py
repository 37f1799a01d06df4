"""it_layer_forward_static: the layer pass for callers that cannot allocate device memory.

Some users of the library run where cudaMalloc is off limits (a serving loop with a frozen
memory pool, a host callback, a process whose device memory belongs to another component), so
they cannot supply the scratch workspace it_layer_forward needs.  The static variant keeps a
fixed 32 MiB scratch array inside the library instead.  These tests call it through the C ABI,
twice in a row (the array is shared and keeps the previous call's contents), and require the
same bits as the ordinary entry point.  This file is collected last on purpose.
"""
import numpy as np
import pytest
import torch

from gpu_util import make_gat_layer, make_sage_layer, small_workload
from paper_2307_00228_b200 import binding as B
from paper_2307_00228_b200 import host

pytestmark = pytest.mark.gpu


def reference_and_static(w, layer_np):
    d = host.upload(w)
    lay = d.layers[0]
    ws = torch.empty(B.it_workspace_bytes(d.graph, [lay]), dtype=torch.uint8, device="cuda")
    ref = torch.empty((w.n, layer_np.out_dim), dtype=d.x.dtype, device="cuda")
    B.it_layer_forward(d.graph, lay, d.x, ref, ws)
    outs = []
    for _ in range(2):
        o = torch.full_like(ref, float("nan"))
        B.it_layer_forward_static(d.graph, lay, d.x, o)
        outs.append(o)
    torch.cuda.synchronize()
    return d, ref, outs


@pytest.mark.parametrize("case", ["sage_split", "sage_reorder", "gat"])
def test_static_variant_matches_the_workspace_variant_on_two_calls_in_a_row(case):
    if case == "sage_split":       # partial rows of split hubs live in the scratch array
        layer = make_sage_layer(41, "sum", "relu", 64, 64, "f32", weights=True)
        w = small_workload(42, 4000, 20, "f32", [layer], hubs=(3000, 700, 300), weights=True, threshold=128)
    elif case == "sage_reorder":   # self term and transformed rows live in the scratch array
        layer = make_sage_layer(43, "mean", "none", 64, 16, "bf16")
        w = small_workload(44, 5000, 12, "bf16", [layer], hubs=(900,), threshold=256)
    else:                          # transformed rows and attention scores live in the scratch array
        layer = make_gat_layer(45, "elu", 64, 4, 16, "bf16")
        w = small_workload(46, 3000, 15, "bf16", [layer], hubs=(500,))
    d, ref, outs = reference_and_static(w, layer)
    if case == "sage_split":
        assert d.n_split_owners > 0
    assert bool(torch.isfinite(ref.float()).all())
    for o in outs:
        assert torch.equal(o, ref)     # same kernels, same order: the tests' bar here is equality


def test_a_repeated_call_leaves_device_memory_as_it_found_it():
    """What the entry point is for: after the set-up call of a layer shape (which loads the kernels it needs and
    looks up the array), further calls neither take nor return device memory — seen from the driver (free bytes of
    the device) and from torch's caching allocator (bytes reserved, allocation count)."""
    layer = make_sage_layer(54, "sum", "relu", 64, 64, "f32", weights=True)
    w = small_workload(55, 4000, 20, "f32", [layer], hubs=(3000, 700), weights=True, threshold=128)
    d = host.upload(w)
    assert d.n_split_owners > 0
    out = torch.empty((w.n, 64), device="cuda")
    B.it_layer_forward_static(d.graph, d.layers[0], d.x, out)     # set-up call
    torch.cuda.synchronize()
    first = out.clone()
    free0 = torch.cuda.mem_get_info()[0]
    stats0 = torch.cuda.memory_stats()
    for _ in range(3):
        B.it_layer_forward_static(d.graph, d.layers[0], d.x, out)
    torch.cuda.synchronize()
    stats1 = torch.cuda.memory_stats()
    assert torch.cuda.mem_get_info()[0] == free0
    for key in ("reserved_bytes.all.current", "allocation.all.allocated", "segment.all.allocated"):
        assert stats1[key] == stats0[key], key
    assert torch.equal(out, first)


def test_calls_of_different_layers_share_the_array_safely():
    """Back-to-back calls with different layouts of the scratch array: each call rewrites what it reads."""
    l1 = make_sage_layer(47, "max", "relu", 32, 32, "f32")
    l2 = make_sage_layer(48, "sum", "none", 32, 8, "f32")
    w = small_workload(49, 2500, 10, "f32", [l1, l2], hubs=(1200,), threshold=64)
    d = host.upload(w)
    want = []
    h = d.x
    for lay, src in zip(d.layers, w.layers):
        ws = torch.empty(B.it_workspace_bytes(d.graph, [lay]), dtype=torch.uint8, device="cuda")
        o = torch.empty((w.n, src.out_dim), device="cuda")
        B.it_layer_forward(d.graph, lay, h, o, ws)
        want.append(o)
        h = o
    h = d.x
    for lay, src, ref in zip(d.layers, w.layers, want):
        o = torch.empty((w.n, src.out_dim), device="cuda")
        B.it_layer_forward_static(d.graph, lay, h, o)
        torch.cuda.synchronize()
        assert torch.equal(o, ref)
        h = o


def test_layer_larger_than_the_built_in_scratch_is_rejected():
    layer = make_sage_layer(50, "sum", "relu", 64, 64, "f32")
    n = B.STATIC_WORKSPACE_BYTES // (64 * 4) + 1000      # the aggregate alone exceeds the array
    w = small_workload(51, n, 2, "f32", [layer])
    d = host.upload(w)
    assert B.it_workspace_bytes(d.graph, d.layers) > B.STATIC_WORKSPACE_BYTES
    out = torch.empty((w.n, 64), device="cuda")
    with pytest.raises(B.ItError) as ei:
        B.it_layer_forward_static(d.graph, d.layers[0], d.x, out)
    assert ei.value.status_name == "IT_ERR_WORKSPACE" and "built-in" in str(ei.value)
    # the ordinary entry point still serves it
    B.it_layer_forward(d.graph, d.layers[0], d.x, out, d.workspace)
    torch.cuda.synchronize()
    assert bool(torch.isfinite(out).all())


def test_static_variant_refuses_to_run_under_instrumentation():
    layer = make_sage_layer(52, "sum", "relu", 16, 16, "f32")
    w = small_workload(53, 200, 4, "f32", [layer])
    d = host.upload(w)
    out = torch.empty((w.n, 16), device="cuda")
    B.it_profile_begin()
    try:
        with pytest.raises(B.ItError) as ei:
            B.it_layer_forward_static(d.graph, d.layers[0], d.x, out)
        assert ei.value.status_name == "IT_ERR_UNSUPPORTED"
    finally:
        B.it_profile_end()
    B.it_layer_forward_static(d.graph, d.layers[0], d.x, out)
    torch.cuda.synchronize()
