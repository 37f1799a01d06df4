"""Index side on the GPU (validation, hub split, degree buckets): bit-exact against the oracle."""
import numpy as np
import pytest
import torch

from oracle import oracle as O
from paper_2307_00228_b200 import binding as B
from workloads import make

pytestmark = pytest.mark.gpu


def device_split(indptr_np, indices_np, threshold, int32=False):
    ip = torch.from_numpy(indptr_np.astype(np.int32) if int32 else indptr_np).cuda()
    ix = torch.from_numpy(indices_np).cuda()
    g = B.it_graph_create(ip, ix)
    n_rows, n_split = B.it_split_hubs(g, threshold)
    s = B.it_graph_get_split(g)
    return g, n_rows, n_split, {k: (v.cpu().numpy() if torch.is_tensor(v) else v) for k, v in s.items()}


def assert_split_matches_oracle(indptr, indices, T, int32=False):
    g, n_rows, n_split, s = device_split(indptr, indices, T, int32)
    sp, so, op = O.split_hubs(indptr, T)
    assert n_rows == sp.shape[0] - 1 == s["n_rows"]
    assert n_split == int((np.diff(op) > 1).sum())
    assert np.array_equal(s["shadow_indptr"], sp)
    assert np.array_equal(s["shadow_owner"], so)
    assert np.array_equal(s["owner_indptr"], op)
    off, rows = O.buckets(sp, s["bucket_bounds"])
    assert np.array_equal(s["bucket_offsets"], off)
    assert np.array_equal(s["bucket_rows"], rows)
    return s


def random_csr(seed, n, max_deg, hubs=()):
    rng = np.random.default_rng(seed)
    deg = rng.integers(0, max_deg + 1, size=n)
    deg[rng.random(n) < 0.3] = 0
    for i, d in enumerate(hubs):
        deg[(11 * i + 5) % n] = d
    ip = np.zeros(n + 1, np.int64)
    np.cumsum(deg, out=ip[1:])
    return ip, rng.integers(0, max(n, 1), size=int(ip[-1])).astype(np.int32)


@pytest.mark.parametrize("T", [0, 1, 2, 7, 8, 9, 32, 33, 256, 257, 1024, 100000])
@pytest.mark.parametrize("int32", [False, True])
def test_split_and_buckets_bit_exact(T, int32):
    ip, ix = random_csr(T + 1, 5000, 40, hubs=(300, 257, 256, 255, 1025, 2049, 5000, 33, 32, 9, 8))
    s = assert_split_matches_oracle(ip, ix, T, int32)
    assert s["bucket_bounds"] == sorted(set(s["bucket_bounds"]))


def test_split_spans_many_scan_tiles_and_ragged_tail():
    # more vertices than several 2048-wide scan tiles, not a multiple of the tile
    ip, ix = random_csr(3, 2048 * 37 + 517, 6, hubs=(4000, 4097, 9000))
    assert_split_matches_oracle(ip, ix, 64)
    assert_split_matches_oracle(ip, ix, 0)


def test_tiny_config_split():
    w = make("tiny")
    s = assert_split_matches_oracle(w.indptr, w.indices, w.threshold)
    assert s["bucket_bounds"] == [0, 8, 32, 256]


def test_extreme_shape_split():
    w = make("extreme", 0.005)
    assert_split_matches_oracle(w.indptr, w.indices, 64)


def test_degenerate_graphs():
    # no vertices
    g = B.it_graph_create(torch.zeros(1, dtype=torch.int64, device="cuda"), torch.zeros(0, dtype=torch.int32, device="cuda"))
    assert B.it_split_hubs(g, 4) == (0, 0)
    # vertices but no edges
    ip = np.zeros(1001, np.int64)
    assert_split_matches_oracle(ip, np.zeros(0, np.int32), 4)
    # one vertex holding every edge, split into single-edge rows
    ip = np.array([0, 777], np.int64)
    ix = np.zeros(777, np.int32)
    s = assert_split_matches_oracle(ip, ix, 1)
    assert s["n_rows"] == 777


def test_resplit_replaces_the_previous_split():
    ip, ix = random_csr(9, 3000, 50, hubs=(700,))
    g = B.it_graph_create(torch.from_numpy(ip).cuda(), torch.from_numpy(ix).cuda())
    for T in (5, 0, 64, 5):
        n_rows, _ = B.it_split_hubs(g, T)
        sp, so, op = O.split_hubs(ip, T)
        s = B.it_graph_get_split(g)
        assert n_rows == so.shape[0] and np.array_equal(s["shadow_indptr"].cpu().numpy(), sp)


@pytest.mark.parametrize("kind", ["start", "decreasing", "end", "source_high", "source_negative"])
def test_bad_csr_is_rejected_with_a_status(kind):
    ip, ix = random_csr(1, 200, 5)
    ip, ix = ip.copy(), ix.copy()
    if kind == "start":
        ip[0] = 1
    elif kind == "decreasing":
        ip[50], ip[51] = ip[51] + 3, ip[50]
    elif kind == "end":
        ip[-1] += 1
        ix = np.concatenate([ix, [0]]).astype(np.int32)[: ix.shape[0]]
    elif kind == "source_high":
        ix[len(ix) // 2] = 200
    else:
        ix[3] = -1
    with pytest.raises(B.ItError) as ei:
        B.it_graph_create(torch.from_numpy(ip).cuda(), torch.from_numpy(ix).cuda())
    assert ei.value.status_name == "IT_ERR_BAD_GRAPH"
    # the context is still healthy afterwards
    assert torch.ones(4, device="cuda").sum().item() == 4


def test_invalid_arguments():
    ip, ix = random_csr(1, 20, 3)
    with pytest.raises(B.ItError) as ei:
        B.it_graph_create(torch.from_numpy(ip).cuda(), torch.from_numpy(ix).cuda(), n_vertices=-1)
    assert ei.value.status_name == "IT_ERR_INVALID_ARG"
    assert B.lib().it_split_hubs(None, 4, None, None, None) == 1
    assert B.lib().it_graph_destroy(None) == 0


@pytest.mark.parametrize("tdtype", [torch.bfloat16, torch.float32, "fused"])
def test_a_wait_that_runs_out_is_reported_and_the_library_goes_on(tdtype):
    """The tensor-core apply waits on hardware barriers with a poll limit.  With its copy producer switched off
    every wait runs out: the kernel must return by itself, it_graph_check must say IT_ERR_TIMEOUT once, and a
    real layer afterwards must still be right."""
    from gpu_util import check_against_oracle, make_sage_layer, run_device, small_workload
    layer = make_sage_layer(1, "sum", "relu", 64, 64, "bf16")
    w = small_workload(2, 600, 12, "bf16", [layer])
    got, d = run_device(w)
    check_against_oracle(w, got)
    fused = tdtype == "fused"   # the kernel that runs two products back to back
    tdtype = torch.bfloat16 if fused else tdtype
    x = torch.zeros((128, 64), dtype=tdtype, device="cuda")
    o = torch.empty((128, 64), dtype=tdtype, device="cuda")
    ws = torch.empty(1 << 16, dtype=torch.uint8, device="cuda")
    if fused:
        B.it_debug_expire_wait_fused(d.graph, x, o, ws)
    else:
        B.it_debug_expire_wait(d.graph, x, o, ws)
    with pytest.raises(B.ItError) as e:
        B.it_graph_check(d.graph)
    assert e.value.status_name == "IT_ERR_TIMEOUT"
    B.it_graph_check(d.graph)          # reported once
    d.infer()
    B.it_graph_check(d.graph)
    from gpu_util import to_numpy
    check_against_oracle(w, to_numpy(d.out))
