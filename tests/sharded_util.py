"""A CPU stand-in for the stage calls of the library, built from the oracle's primitives, so that the host-side
logic of the vertex-partitioned layer pass (who owns which rows, what is exchanged, where a worker's rows sit in
an all-gathered table) can run as gloo ranks without a GPU.  Test infrastructure only."""
from types import SimpleNamespace as NS

import numpy as np
import torch

from oracle import oracle as O


class OracleEngine:
    def __init__(self, dtype: str):
        self.dtype = dtype

    # ---- memory
    def feat_dtype(self, dtype):
        return torch.float32 if dtype == "f32" else torch.bfloat16

    def to_device(self, a, dtype=None):
        if a is None:
            return None
        if dtype == "bf16":
            return torch.from_numpy(a.view(np.int16)).view(torch.bfloat16)
        return torch.from_numpy(a)

    def empty(self, rows, cols, dtype):
        return torch.zeros((rows, cols), dtype=dtype)

    def workspace(self, part, layers):
        return {}

    @staticmethod
    def _np(t):
        return None if t is None else t.float().numpy().astype(np.float64)

    def _store(self, out, a, n):
        out[:n] = torch.from_numpy(O.round_to(a, self.dtype).astype(np.float32)).to(out.dtype)

    # ---- graph parts and layers
    def create_part(self, indptr, indices, weights, n_sources):
        assert indices.size == 0 or (indices.min() >= 0 and indices.max() < n_sources)
        return NS(indptr=np.asarray(indptr, np.int64), indices=np.asarray(indices, np.int32), weights=weights,
                  n=indptr.shape[0] - 1, n_sources=n_sources)

    def layer(self, layer_np, dtype):
        return layer_np

    def stages(self, part, layer):
        if layer.op == "gat":
            return dict(table_dim=layer.out_dim, score_dim=2 * layer.heads, table_is_input=False, agg_dim=0)
        if layer.op == "dense":
            return dict(table_dim=0, score_dim=0, table_is_input=True, agg_dim=0)
        if O.will_reorder(layer):
            return dict(table_dim=layer.out_dim, score_dim=0, table_is_input=False, agg_dim=0)
        return dict(table_dim=layer.in_dim, score_dim=0, table_is_input=True, agg_dim=layer.in_dim)

    # ---- the three stages
    def transform(self, part, layer, h_self, table_out, scores_out, ws):
        H = self._np(h_self)[:part.n]
        W, Fi = np.asarray(layer.W, np.float64), layer.in_dim
        if layer.op == "gat":
            z = O.linear(H, W)
            self._store(table_out, z, part.n)
            s = np.concatenate([O.gat_scores(z, layer.att_src, layer.heads), O.gat_scores(z, layer.att_dst, layer.heads)], axis=1)
            scores_out[:part.n] = torch.from_numpy(s.astype(np.float32))
        elif layer.op == "gcn":
            self._store(table_out, O.linear(H, W), part.n)
        else:
            self._store(table_out, O.linear(H, W[Fi:]), part.n)
            S = O.linear(H, W[:Fi]) + (0 if layer.bias is None else np.asarray(layer.bias, np.float64)[None, :])
            ws["S"] = O.round_to(S, self.dtype)

    def gather(self, part, layer, table, scores, first, raw, out, ws):
        T = self._np(table)
        w = part.weights if layer.use_edge_weights else None
        n = part.n
        if layer.op == "gat":
            s = self._np(scores)
            h = layer.heads
            A = O.gat_aggregate(part.indptr, part.indices, T, np.ascontiguousarray(s[:, :h]),
                                np.ascontiguousarray(s[first:first + n, h:]), h, layer.leaky_slope)
            self._store(out, O.bias_act(A, layer.bias, layer.act), n)
            return
        op = "sum" if layer.op == "gcn" else layer.op
        if raw:
            A = O.aggregate(part.indptr, part.indices, w, T, "sum" if op == "mean" else op)
            empty = np.diff(part.indptr) == 0
            if op == "max":
                A[empty] = -np.inf
            if op == "min":
                A[empty] = np.inf
            out[:n] = torch.from_numpy(A.astype(np.float32))
            return
        A = O.aggregate(part.indptr, part.indices, w, T, op)
        if O.will_reorder(layer):
            if layer.op == "gcn":
                self._store(out, O.bias_act(A, layer.bias, layer.act), n)
            else:
                self._store(out, O.bias_act(ws["S"] + A, None, layer.act), n)
            return
        self._store(out, A, n)

    def update(self, part, layer, h_self, agg, h_out, ws):
        H = self._np(h_self)[:part.n]
        W = np.asarray(layer.W, np.float64)
        if layer.op == "dense":
            res = O.bias_act(O.linear(H, W), layer.bias, layer.act)
        elif layer.op == "gcn":
            res = O.bias_act(O.linear(self._np(agg)[:part.n], W), layer.bias, layer.act)
        else:
            res = O.sage_apply(H, self._np(agg)[:part.n], W, layer.bias, layer.act)
        self._store(h_out, res, part.n)

    def finish(self, raw, scale, out):
        r, s = raw.numpy().astype(np.float64), scale.numpy().astype(np.float64)
        a = np.where(s[:, None] == 0, 0.0, r * s[:, None])
        self._store(out, a, a.shape[0])
