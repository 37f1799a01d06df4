"""The five seeded synthetic workloads (graph + features + layer parameters).

Each stands in for the paper's Power-Law / MAG240M-class inputs, which are not
distributable with this repository: same kind of structure (power-law in-degree,
hubs), same order of size, seeded and synthetic.  `scale` < 1 shrinks vertices and
edges together (mean degree, degree cap rule and model unchanged) for cases a CPU
check can finish quickly.

This module holds no GNN arithmetic; parameters are only drawn, never applied.
"""
from __future__ import annotations

from dataclasses import dataclass, field

import numpy as np

from . import graphs, rng as wrng


@dataclass
class Layer:
    op: str                  # 'sum' | 'mean' | 'max' | 'gat'
    act: str                 # 'none' | 'relu' | 'elu'
    in_dim: int
    out_dim: int
    W: np.ndarray            # float32; SAGE [2*in, out] (rows 0..in-1 self, in..2in-1 neighbour); GAT [in, out]
    bias: np.ndarray | None  # float32 [out]
    heads: int = 1
    att_src: np.ndarray | None = None   # float32 [heads, out/heads]
    att_dst: np.ndarray | None = None
    leaky_slope: float = 0.2
    att_edge: np.ndarray | None = None  # GAT with edge features: float32 [heads, edge_dim]
    use_edge_weights: bool = False
    allow_reorder: bool = True
    edge_dim: int = 0        # > 0: the message carries the edge's feature vector; W has edge_dim more neighbour rows
    msg_dim: int = 0         # > 0: learned message m = w_e act_edge([h_u | e_vu] W_edge + bias_edge); W is [in + msg_dim, out] (GCN: [msg_dim, out])
    W_edge: np.ndarray | None = None      # float32 [in + edge_dim, msg_dim]
    bias_edge: np.ndarray | None = None   # float32 [msg_dim]
    act_edge: str = "none"


@dataclass
class Workload:
    name: str
    n: int
    e: int
    indptr: np.ndarray        # int64 [n+1]
    indices: np.ndarray       # int32 [e], sources, ascending inside each destination segment
    edge_weights: np.ndarray | None   # float32 [e]
    dtype: str                # 'f32' | 'bf16': storage type of features and layer outputs
    x: np.ndarray             # float32 [n, f] (f32) or uint16 bf16 bit patterns [n, f] (bf16)
    layers: list = field(default_factory=list)
    threshold: int = 0        # shadow-row threshold; <= 0 means no split
    edge_feat: np.ndarray | None = None   # [e, edge_dim], float32 or bf16 bit patterns like x; row j belongs to CSR entry j

    def x_as_f32(self) -> np.ndarray:
        return self.x if self.dtype == "f32" else wrng.bf16_bits_to_f32(self.x)

    def edge_feat_as_f32(self) -> np.ndarray | None:
        if self.edge_feat is None:
            return None
        return self.edge_feat if self.dtype == "f32" else wrng.bf16_bits_to_f32(self.edge_feat)


def _glorot(rng, fan_in: int, fan_out: int, shape) -> np.ndarray:
    lim = np.sqrt(6.0 / (fan_in + fan_out))
    return rng.uniform(-lim, lim, size=shape).astype(np.float32)


def _storage_round(a: np.ndarray, dtype: str) -> np.ndarray:
    """Parameters are stored in the workload's dtype; return their exact float32 values."""
    if dtype == "bf16":
        return wrng.bf16_bits_to_f32(wrng.f32_to_bf16_bits(a))
    return a


def sage_layers(dims, op, acts, dtype, use_edge_weights=False, edge_dim=0) -> list:
    """GraphSAGE layers dims[0]->dims[1]->...; Glorot-uniform over the whole [2*in (+ edge_dim), out]
    matrix; bias ~ U(-0.1, 0.1)."""
    out = []
    for i in range(len(dims) - 1):
        fi, fo = dims[i], dims[i + 1]
        k = 2 * fi + edge_dim
        W = _glorot(wrng.stream(wrng.SEED_WEIGHTS, i), k, fo, (k, fo))
        b = wrng.stream(wrng.SEED_BIAS, i).uniform(-0.1, 0.1, size=fo).astype(np.float32)
        out.append(Layer(op=op, act=acts[i], in_dim=fi, out_dim=fo, W=_storage_round(W, dtype),
                         bias=b, use_edge_weights=use_edge_weights, edge_dim=edge_dim))
    return out


def gat_layers(dims, heads, acts, dtype, slope=0.2) -> list:
    out = []
    for i in range(len(dims) - 1):
        fi, fo = dims[i], dims[i + 1]
        hd = fo // heads
        r = wrng.stream(wrng.SEED_WEIGHTS, i)
        W = _glorot(r, fi, fo, (fi, fo))
        a_s = _glorot(r, hd, 1, (heads, hd))
        a_d = _glorot(r, hd, 1, (heads, hd))
        b = wrng.stream(wrng.SEED_BIAS, i).uniform(-0.1, 0.1, size=fo).astype(np.float32)
        out.append(Layer(op="gat", act=acts[i], in_dim=fi, out_dim=fo, W=_storage_round(W, dtype),
                         bias=b, heads=heads, att_src=a_s, att_dst=a_d, leaky_slope=slope))
    return out


def _features(n, f, dtype):
    r = wrng.stream(wrng.SEED_FEATURES)
    return wrng.normal_f32(r, (n, f)) if dtype == "f32" else wrng.normal_bf16_bits(r, (n, f))


def with_edge_features(w: Workload, edge_dim: int) -> Workload:
    """The same workload with seeded N(0,1) edge features of length edge_dim in every message (GraphSAGE
    workloads only): the layers are redrawn with edge_dim more neighbour rows."""
    if edge_dim <= 0:
        return w
    if any(l.op == "gat" for l in w.layers):
        raise ValueError("edge features are defined for the pooling layers and GCN")
    r = wrng.stream(wrng.SEED_EDGE_FEATURES)
    w.edge_feat = wrng.normal_f32(r, (w.e, edge_dim)) if w.dtype == "f32" else wrng.normal_bf16_bits(r, (w.e, edge_dim))
    dims = [w.layers[0].in_dim] + [l.out_dim for l in w.layers]
    w.layers = sage_layers(dims, w.layers[0].op, [l.act for l in w.layers], w.dtype,
                           use_edge_weights=w.layers[0].use_edge_weights, edge_dim=edge_dim)
    return w


def make(name: str, scale: float = 1.0) -> Workload:
    """Build one of 'tiny', 'medium', 'gat', 'extreme', 'large' (optionally shrunk)."""
    g = wrng.stream(wrng.SEED_GRAPH)
    s = lambda v: max(1, int(round(v * scale)))
    if name == "tiny":
        n, e = s(10_000), s(100_000)
        indptr, indices = graphs.power_law_graph(g, n, e, 2.1, 2_000, source_exponent=2.1)
        return Workload(name, n, e, indptr, indices, None, "f32", _features(n, 64, "f32"),
                        sage_layers([64, 64, 16], "mean", ["relu", "none"], "f32"), 256)
    if name == "medium":
        n, e = s(2_000_000), s(40_000_000)
        indptr, indices = graphs.power_law_graph(g, n, e, 2.1, s(200_000))
        w = wrng.stream(wrng.SEED_EDGE_WEIGHTS).random(e, dtype=np.float32)
        return Workload(name, n, e, indptr, indices, w, "f32", _features(n, 128, "f32"),
                        sage_layers([128, 128, 64], "sum", ["relu", "none"], "f32",
                                    use_edge_weights=True), 1024)
    if name == "gat":
        n, e = s(5_000_000), s(100_000_000)
        indptr, indices = graphs.power_law_graph(g, n, e, 2.0, s(200_000))
        return Workload(name, n, e, indptr, indices, None, "bf16", _features(n, 128, "bf16"),
                        gat_layers([128, 128, 128], 4, ["elu", "none"], "bf16"), 4096)
    if name == "extreme":
        n, e = s(20_000_000), s(200_000_000)
        n_hubs = 100 if scale >= 0.01 else 4
        indptr, indices = graphs.extreme_hubs_graph(g, n, e, n_hubs, s(1_000_000))
        return Workload(name, n, e, indptr, indices, None, "bf16", _features(n, 64, "bf16"),
                        sage_layers([64, 64, 64, 32], "max", ["relu", "relu", "none"], "bf16"), 4096)
    if name == "large":
        n, e = s(100_000_000), s(1_500_000_000)
        indptr, indices = graphs.power_law_graph(g, n, e, 2.1, s(200_000))
        return Workload(name, n, e, indptr, indices, None, "bf16", _features(n, 64, "bf16"),
                        sage_layers([64, 128, 64], "mean", ["relu", "none"], "bf16"), 4096)
    raise ValueError(f"unknown workload {name!r}")
