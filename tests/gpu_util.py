"""Helpers shared by the GPU parity tests: run a workload through the C ABI and through the
oracle and compare.  The oracle never sees a value produced by the CUDA path."""
from __future__ import annotations

import numpy as np
import torch

from oracle import oracle as O
from paper_2307_00228_b200 import binding as B
from paper_2307_00228_b200 import host
from workloads import Layer, Workload, compare
from workloads import rng as wrng

TOL = compare.TOL   # max relative error: fp32 paths / bf16 apply paths


def to_numpy(t: torch.Tensor) -> np.ndarray:
    return t.float().cpu().numpy().astype(np.float64)


def storage_exact(a: np.ndarray, dtype: str) -> np.ndarray:
    """float32 values that are exactly representable in the storage dtype."""
    a = np.ascontiguousarray(a, dtype=np.float32)
    return wrng.bf16_bits_to_f32(wrng.f32_to_bf16_bits(a)) if dtype == "bf16" else a


def small_workload(seed, n, max_deg, dtype, layers, hubs=(), weights=False, threshold=0, p_zero=0.2, edge_dim=0) -> Workload:
    rng = np.random.default_rng(seed)
    deg = rng.integers(0, max_deg + 1, size=n)
    deg[rng.random(n) < p_zero] = 0
    for i, d in enumerate(hubs):
        deg[(7 * i + 3) % n] = d
    indptr = np.zeros(n + 1, np.int64)
    np.cumsum(deg, out=indptr[1:])
    e = int(indptr[-1])
    indices = rng.integers(0, n, size=e).astype(np.int32)
    w = rng.random(e, dtype=np.float32) if weights else None
    x = rng.standard_normal((n, layers[0].in_dim)).astype(np.float32)
    xs = x if dtype == "f32" else wrng.f32_to_bf16_bits(x)
    ef = None
    if edge_dim:
        ef = rng.standard_normal((e, edge_dim)).astype(np.float32)
        ef = ef if dtype == "f32" else wrng.f32_to_bf16_bits(ef)
    return Workload("small", n, e, indptr, indices, w, dtype, xs, layers, threshold, ef)


def make_sage_layer(seed, op, act, fi, fo, dtype, weights=False, allow_reorder=True, bias=True, edge_dim=0) -> Layer:
    rng = np.random.default_rng(seed)
    lim = np.sqrt(6.0 / (2 * fi + edge_dim + fo))
    return Layer(op=op, act=act, in_dim=fi, out_dim=fo,
                 W=storage_exact(rng.uniform(-lim, lim, (2 * fi + edge_dim, fo)), dtype),
                 bias=rng.uniform(-0.1, 0.1, fo).astype(np.float32) if bias else None,
                 use_edge_weights=weights, allow_reorder=allow_reorder, edge_dim=edge_dim)


def make_plain_layer(seed, op, act, fi, fo, dtype, weights=False, allow_reorder=True, bias=True, edge_dim=0) -> Layer:
    """op = "dense" (no Gather stage) or "gcn" (update on the aggregate alone): W is [fi (+ edge_dim), fo]."""
    rng = np.random.default_rng(seed)
    lim = np.sqrt(6.0 / (fi + edge_dim + fo))
    return Layer(op=op, act=act, in_dim=fi, out_dim=fo,
                 W=storage_exact(rng.uniform(-lim, lim, (fi + edge_dim, fo)), dtype),
                 bias=rng.uniform(-0.1, 0.1, fo).astype(np.float32) if bias else None,
                 use_edge_weights=weights, allow_reorder=allow_reorder, edge_dim=edge_dim)


def make_msg_layer(seed, op, act, fi, fm, fo, dtype, act_edge="relu", weights=False, edge_dim=0, bias=True) -> Layer:
    """A layer with learned messages m = w_e act_edge([h_u | e_vu] W_edge + b_edge) of length fm; op may be "gcn"."""
    rng = np.random.default_rng(seed)
    k = fm if op == "gcn" else fi + fm
    lim, lim_e = np.sqrt(6.0 / (k + fo)), np.sqrt(6.0 / (fi + edge_dim + fm))
    return Layer(op=op, act=act, in_dim=fi, out_dim=fo, W=storage_exact(rng.uniform(-lim, lim, (k, fo)), dtype),
                 bias=rng.uniform(-0.1, 0.1, fo).astype(np.float32) if bias else None, use_edge_weights=weights,
                 edge_dim=edge_dim, msg_dim=fm, W_edge=storage_exact(rng.uniform(-lim_e, lim_e, (fi + edge_dim, fm)), dtype),
                 bias_edge=rng.uniform(-0.1, 0.1, fm).astype(np.float32) if bias else None, act_edge=act_edge)


def make_gat_layer(seed, act, fi, heads, hd, dtype, bias=True, edge_dim=0) -> Layer:
    rng = np.random.default_rng(seed)
    fo = heads * hd
    lim = np.sqrt(6.0 / (fi + fo))
    return Layer(op="gat", act=act, in_dim=fi, out_dim=fo, W=storage_exact(rng.uniform(-lim, lim, (fi, fo)), dtype),
                 bias=rng.uniform(-0.1, 0.1, fo).astype(np.float32) if bias else None, heads=heads,
                 att_src=rng.uniform(-0.4, 0.4, (heads, hd)).astype(np.float32),
                 att_dst=rng.uniform(-0.4, 0.4, (heads, hd)).astype(np.float32), edge_dim=edge_dim,
                 att_edge=rng.uniform(-0.4, 0.4, (heads, edge_dim)).astype(np.float32) if edge_dim else None)


def run_device(w: Workload, int32_indptr=False, threshold=None):
    """it_infer through the C ABI; returns (final output as fp64 numpy, DeviceWorkload)."""
    d = host.upload(w, int32_indptr=int32_indptr, threshold=threshold)
    d.infer()
    B.it_graph_check(d.graph)     # synchronises; raises if a kernel gave up a bounded wait
    return to_numpy(d.out), d


def run_oracle(w: Workload, storage="same", threshold=None, magnitudes=False):
    """Oracle over all layers.  storage='same': round at the storage points like the device
    contract (the gate); storage=None: fp64 throughout, plain order of operations."""
    st = w.dtype if storage == "same" else storage
    thr = w.threshold if threshold is None else threshold
    return O.infer(w.indptr, w.indices, w.edge_weights, w.x_as_f32(), w.layers, storage=st, threshold=thr,
                   follow_reorder=st is not None, edge_feat=w.edge_feat_as_f32(), magnitudes=magnitudes)


def assert_close(got, ref, mag, dtype, mode="stored", tol=None, label="", n_layers=1):
    """The parity gate: every entry within tol of the reference relative to max(|ref|, floor * term magnitude); against
    the storage-rounding oracle, for up to three layers, also the plain relative error of the entries above the
    reference's rms.  (Against the fp64-throughout oracle, and at the end of a deep pipeline, an entry above the rms may
    still be a small remainder of large terms, each carrying the rounding of a stored tensor, so only the floored form is
    a bound there.)"""
    err = compare.rel_error(got, ref, mag, compare.floor_for(mode, dtype, n_layers))
    tol = TOL[dtype] if tol is None else tol
    assert err["finite"], (label, err)
    assert err["max_rel"] <= tol, (label, mode, n_layers, err)
    if mode == "stored" and n_layers <= 3:
        assert err["max_rel_plain"] <= tol, (label, mode, n_layers, err)
    return err


def check_against_oracle(w: Workload, got: np.ndarray, tol=None, label="", exact=True):
    """The result of all layers against the oracle run from the raw inputs."""
    L = len(w.layers)
    outs, mags = run_oracle(w, magnitudes=True)
    err = assert_close(got, outs[-1], mags[-1], w.dtype, "stored", tol, label, n_layers=L)
    if exact:   # and against the fp64-throughout oracle, which charges the storage roundings to the device
        outs_a, mags_a = run_oracle(w, storage=None, magnitudes=True)
        assert_close(got, outs_a[-1], mags_a[-1], w.dtype, "exact", tol, label, n_layers=L)
    return err


def check_each_layer(w: Workload, d, label=""):
    """Every layer on its own: the device runs layer l on ITS OWN output of layer l - 1, and the oracle is given exactly
    those values, so nothing compounds and each layer is held to the single-layer floors."""
    h = d.x
    for l, (lay, src) in enumerate(zip(d.layers, w.layers)):
        o = torch.empty((w.n, src.out_dim), dtype=d.x.dtype, device=d.x.device)
        B.it_layer_forward(d.graph, lay, h, o, d.workspace)
        B.it_graph_check(d.graph)
        H = to_numpy(h)
        for mode, storage in (("stored", w.dtype), ("exact", None)):
            ref = O.layer_forward(w.indptr, w.indices, w.edge_weights, H, src, storage=storage, threshold=w.threshold,
                                  reorder=storage is not None and O.will_reorder(src), edge_feat=w.edge_feat_as_f32())
            mag = O.layer_magnitude(w.indptr, w.indices, w.edge_weights, H, src, edge_feat=w.edge_feat_as_f32())
            assert_close(to_numpy(o), ref, mag, w.dtype, mode, label=(label, "layer", l))
        h = o
    return h
