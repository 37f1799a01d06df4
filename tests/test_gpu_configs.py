"""The five workload shapes through it_infer, against the oracle.

Tiny runs at full size with a full-graph oracle.  The others run (a) shrunk, with a full-graph
oracle, and (b) at full size in the launch configuration the benchmark times, checked on sampled
vertices that the oracle evaluates from their L-hop in-neighbourhood.  The 100M-vertex workload at
full size needs ten minutes of host time to generate and check and is left to the benchmark, which
runs the same sampled check on the result it has just timed; here it runs when IT_RUN_LARGE is set.
"""
import os

import numpy as np
import pytest
import torch

from gpu_util import assert_close, check_against_oracle, run_device, to_numpy
from oracle import oracle as O
from paper_2307_00228_b200 import binding as B
from paper_2307_00228_b200 import host
from workloads import compare, make
from workloads import rng as wrng

pytestmark = pytest.mark.gpu


def test_tiny_full_size():
    w = make("tiny")
    got, d = run_device(w)
    assert d.n_split_owners > 0
    check_against_oracle(w, got)   # against the storage-rounding oracle and the fp64-throughout one


@pytest.mark.parametrize("name,scale,int32", [("medium", 0.01, False), ("gat", 0.004, False), ("extreme", 0.005, False),
                                             ("large", 0.0002, True)])
def test_shrunk_configs_full_oracle(name, scale, int32):
    w = make(name, scale)
    if name in ("large", "gat"):
        w.threshold = 16      # the shrunk graph has no vertex above the config's 4096; keep the split in play
    got, d = run_device(w, int32_indptr=int32)
    if w.threshold:
        assert d.n_split_owners > 0, "the shrunk case must still exercise the split"
    check_against_oracle(w, got, label=name)


def sampled_targets(w, n_top, n_random, seed=5):
    deg = np.diff(w.indptr)
    top = np.argsort(-deg, kind="stable")[:n_top]
    rnd = np.random.default_rng(seed).choice(w.n, size=n_random, replace=False)
    return np.unique(np.concatenate([top, rnd]))


def check_sampled(w, d, targets, label):
    got = to_numpy(d.out[torch.from_numpy(targets).cuda()])
    for mode, storage in (("stored", w.dtype), ("exact", None)):
        ref, mag = O.infer_at(w.indptr, w.indices, w.edge_weights, w.x_as_f32(), w.layers, targets, storage=storage,
                              threshold=w.threshold, follow_reorder=storage is not None, magnitudes=True)
        err = assert_close(got, ref, mag, w.dtype, mode, label=label, n_layers=len(w.layers))
        print(f"{label} ({mode}):", err)
    # properties that hold at any size: finite everywhere, and identical on a second run
    assert bool(torch.isfinite(d.out.float()).all())
    first = d.out.clone()
    d.infer()
    torch.cuda.synchronize()
    assert torch.equal(first, d.out)


def test_medium_full_size_sampled():
    """The benchmark's workload and launch configuration (2M vertices, 40M edges, threshold 1024)."""
    w = make("medium")
    d = host.upload(w)
    d.infer()
    torch.cuda.synchronize()
    # hubs are split, their in-neighbourhoods are large: a few hubs + a random sample
    check_sampled(w, d, sampled_targets(w, 4, 300), "medium")


def test_extreme_hub_rows_at_scale():
    """1/10 of the Extreme config keeps 100 hubs of 100k in-edges: ~25 shadow rows per hub at threshold 4096."""
    w = make("extreme", 0.1)
    d = host.upload(w)
    assert d.n_split_owners == 100
    d.infer()
    torch.cuda.synchronize()
    check_sampled(w, d, sampled_targets(w, 3, 200), "extreme")


def check_compact(w, d, targets, label, out=None, layers=None):
    """Sampled vertices of a big workload against the oracle evaluated on their L-hop in-neighbourhood,
    relabelled to a compact graph so that no full-size fp64 array is needed."""
    layers = w.layers if layers is None else layers
    out = d.out if out is None else out
    ids, cip, cix, cw, ct = O.compact_neighbourhood(w.indptr, w.indices, w.edge_weights, targets, len(layers))
    xc = w.x[ids] if w.dtype == "f32" else wrng.bf16_bits_to_f32(w.x[ids])
    got = to_numpy(out[torch.from_numpy(targets).cuda()])
    for mode, storage in (("stored", w.dtype), ("exact", None)):
        ref, mag = O.infer_at(cip, cix, cw, xc, layers, ct, storage=storage, threshold=w.threshold,
                              follow_reorder=storage is not None, magnitudes=True)
        err = assert_close(got, ref, mag, w.dtype, mode, label=label, n_layers=len(layers))
        print(f"{label} full size ({mode}):", err, "rows", d.n_rows, "split owners", d.n_split_owners, "compact vertices", len(ids))
    assert bool(torch.isfinite(out.float().sum()))


def test_gat_full_size_sampled():
    """5M vertices, 100M edges, bf16, two GAT layers of 4 heads, hubs split at 4096 (partial softmax states
    merged): the two largest hubs and a random sample."""
    w = make("gat")
    d = host.upload(w)
    assert d.n_split_owners > 0
    d.infer()
    B.it_graph_check(d.graph)
    check_compact(w, d, sampled_targets(w, 2, 200), "gat")


def test_extreme_full_size_sampled():
    """20M vertices, 200M edges, 100 hubs of 1M in-edges (245 shadow rows each), bf16, three max-pooling layers.
    A hub's 3-hop in-neighbourhood is the whole graph, so the final output is checked on random vertices
    with no hub within two hops, and the hubs themselves on the output of the first layer alone."""
    w = make("extreme")
    d = host.upload(w)
    assert d.n_split_owners == 100
    d.infer()
    B.it_graph_check(d.graph)
    deg = np.diff(w.indptr)
    hubs = np.flatnonzero(deg >= 1_000_000)
    assert hubs.size == 100
    is_hub = np.zeros(w.n, bool)
    is_hub[hubs] = True
    cand = np.random.default_rng(11).choice(w.n, size=600, replace=False)
    keep = []
    for v in cand:
        hop1 = w.indices[w.indptr[v]:w.indptr[v + 1]]
        hop2 = np.concatenate([w.indices[w.indptr[u]:w.indptr[u + 1]] for u in hop1]) if hop1.size else hop1
        if not (is_hub[v] or is_hub[hop1].any() or is_hub[hop2].any()):
            keep.append(v)
    targets = np.unique(np.array(keep[:300], dtype=np.int64))
    assert targets.size >= 100
    check_compact(w, d, targets, "extreme")
    # the hubs after one layer: 245 partial max rows each, combined
    h3 = hubs[:3].astype(np.int64)
    o1 = torch.empty((w.n, w.layers[0].out_dim), dtype=d.x.dtype, device="cuda")
    B.it_layer_forward(d.graph, d.layers[0], d.x, o1, d.workspace)
    B.it_graph_check(d.graph)
    check_compact(w, d, h3, "extreme hubs after layer 1", out=o1, layers=w.layers[:1])


@pytest.mark.skipif(not os.environ.get("IT_RUN_LARGE"), reason="set IT_RUN_LARGE=1: needs ~100 GB of HBM, ~60 GB of host RAM and ~10 minutes")
def test_large_full_size_sampled():
    """100M vertices, 1.5B edges, int32 CSR, bf16: sampled vertices against the oracle evaluated on
    their 2-hop in-neighbourhood (relabelled to a compact graph)."""
    w = make("large")
    d = host.upload(w, int32_indptr=True)
    d.infer()
    B.it_graph_check(d.graph)
    check_compact(w, d, sampled_targets(w, 2, 150), "large")
