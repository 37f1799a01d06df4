"""The layer pass over several workers that each own a range of the vertices.

The paper's only parallelism is this one (Section "InferTurbo on Graph Processing System"): vertices are
partitioned over the workers together with their edges, every worker runs one layer per superstep on its own
vertices, and what the vertices hand to their out-edges is exchanged in between — exactly one exchange per layer.
Two layouts:

  "gather"   destinations are partitioned.  A worker holds the in-edges of its own vertices (source ids global).
             Per layer: transform what the local vertices send (it_layer_transform; nothing for layers that gather
             their input), ALL-GATHER that table so that every worker holds all of its rows in local memory,
             then gather + update locally.  Works for every layer kind.
  "partial"  the partial-gather of Section "Optimization Strategies": SOURCES are partitioned.  A worker holds, for
             EVERY destination, the in-edges whose source it owns, reduces them locally (raw fp32 partial results:
             sum, max or min), the partial results are REDUCE-SCATTERed (sum / max / min) so that each worker
             receives the finished reduce of its own destinations, which it scales (mean), rounds and updates.
             Traffic per vertex depends on the number of workers only, not on its degree.  For pooling / GCN
             layers that gather their input and carry no edge features; other layers of a model use "gather".

This module is host-side orchestration only: which rows go where.  Every step of the layer runs in the library's
kernels (through an `engine`, by default the CUDA binding); the exchange is torch.distributed (NCCL between GPUs),
and every table is landed in the worker's own memory before a kernel reads it.  A worker is written as two
phases per layer, `pre` (before the exchange) and `post` (after it), so that the same code runs one process per
GPU (`run_spmd`) or, for tests on one device, several workers one after another in one process (`run_emulated`).
"""
from __future__ import annotations

from dataclasses import dataclass, replace

import numpy as np
import torch


def vertex_ranges(n: int, world: int) -> list:
    """Equal blocks of ceil(n / world) vertices; the last ones may be short or empty."""
    per = -(-n // world) if n > 0 else 0
    return [(min(n, r * per), min(n, (r + 1) * per)) for r in range(world)]


def rows_per_worker(n: int, world: int) -> int:
    return -(-n // world) if n > 0 else 0


def destination_part(indptr: np.ndarray, indices: np.ndarray, weights, v0: int, v1: int):
    """CSR of the in-edges of destinations [v0, v1): local indptr, the source ids as they are (global), weights."""
    e0, e1 = int(indptr[v0]), int(indptr[v1])
    ip = (indptr[v0:v1 + 1] - indptr[v0]).astype(np.int64)
    return ip, np.ascontiguousarray(indices[e0:e1]), (None if weights is None else np.ascontiguousarray(weights[e0:e1]))


def source_part(indptr: np.ndarray, indices: np.ndarray, weights, u0: int, u1: int, n_rows: int):
    """CSR over ALL destinations (padded to n_rows rows) of the in-edges whose source lies in [u0, u1); source ids
    are made local (minus u0).  The order of the kept edges inside a destination is unchanged."""
    keep = (indices >= u0) & (indices < u1)
    n = indptr.shape[0] - 1
    counts = np.add.reduceat(np.concatenate([keep, [False]]).astype(np.int64), np.minimum(indptr[:-1], keep.size)) if n > 0 else np.zeros(0, np.int64)
    counts = counts * (np.diff(indptr) > 0)
    ip = np.zeros(n_rows + 1, np.int64)
    np.cumsum(counts, out=ip[1:n + 1])
    ip[n + 1:] = ip[n]
    return ip, (indices[keep] - u0).astype(np.int32), (None if weights is None else np.ascontiguousarray(weights[keep]))


def partial_eligible(layer) -> bool:
    """Layers whose Gather stage can run as a partial-gather over source partitions."""
    return layer.op in ("sum", "mean", "max", "min", "gcn") and not getattr(layer, "edge_dim", 0) and not getattr(layer, "msg_dim", 0)


# ----------------------------------------------------------------------------- the default engine: the CUDA library

class CudaEngine:
    """The stage calls of the C ABI on the current CUDA device."""

    def __init__(self, threshold: int = 0, device="cuda"):
        from . import binding as B
        self.B, self.threshold, self.device = B, threshold, device

    def to_device(self, a: np.ndarray, dtype: str | None = None):
        if a is None:
            return None
        if dtype == "bf16":
            return torch.from_numpy(a.view(np.int16)).to(self.device).view(torch.bfloat16)
        return torch.from_numpy(a).to(self.device)

    def create_part(self, indptr, indices, weights, n_sources):
        g = self.B.it_graph_create_part(self.to_device(indptr), self.to_device(indices), n_sources, self.to_device(weights))
        self.B.it_split_hubs(g, self.threshold)
        return g

    def layer(self, layer_np, dtype):
        from . import host
        return host.layer_to_device(layer_np, dtype, self.device)

    def stages(self, part, layer):
        return self.B.it_layer_stages(part, layer)

    def workspace(self, part, layers):
        return torch.empty(max(256, self.B.it_workspace_bytes(part, layers)), dtype=torch.uint8, device=self.device)

    def empty(self, rows, cols, dtype):
        # not cleared: every row that is later read is written first (the padding rows of a block are exchanged but no
        # source id names them)
        return torch.empty((rows, cols), dtype=dtype, device=self.device)

    def transform(self, part, layer, h_self, table_out, scores_out, ws):
        self.B.it_layer_transform(part, layer, h_self, table_out, scores_out, ws)

    def gather(self, part, layer, table, scores, first, raw, out, ws):
        self.B.it_layer_gather(part, layer, table, scores, first, raw, out, ws)

    def update(self, part, layer, h_self, agg, h_out, ws):
        self.B.it_layer_update(part, layer, h_self, agg, h_out, ws)

    def finish(self, raw, scale, out):
        self.B.it_aggregate_finish(raw, scale, out)

    def feat_dtype(self, dtype: str):
        return torch.float32 if dtype == "f32" else torch.bfloat16


# ----------------------------------------------------------------------------- one worker

@dataclass
class Exchange:
    """What a worker hands to the exchange of one layer, and which collective it wants."""
    kind: str                      # "none" | "all_gather" | "reduce_scatter"
    table: torch.Tensor | None = None     # all_gather: [rows_per_worker, table_dim]; reduce_scatter: [world * rows_per_worker, dim] fp32
    scores: torch.Tensor | None = None    # all_gather only: [rows_per_worker, score_dim] fp32
    op: str = "sum"                # reduce_scatter: "sum" | "max" | "min"


class Worker:
    """Rank `rank` of `world`: owns vertices [v0, v1) of an n-vertex graph given as a whole CSR on the host (every
    worker cuts its own part out of it)."""

    def __init__(self, rank: int, world: int, indptr, indices, weights, x_local, layers, dtype: str, engine,
                 layout: str = "gather"):
        assert layout in ("gather", "partial")
        self.rank, self.world, self.engine, self.dtype, self.layout = rank, world, engine, dtype, layout
        n = indptr.shape[0] - 1
        self.n = n
        self.per = rows_per_worker(n, world)
        self.v0, self.v1 = vertex_ranges(n, world)[rank]
        self.n_loc = self.v1 - self.v0
        self.n_table = self.per * world            # rows of an all-gathered table (>= n; the padding is never read)
        ip, ix, w = destination_part(indptr, indices, weights, self.v0, self.v1)
        self.part = engine.create_part(ip, ix, w, self.n_table)
        self.layers_np = list(layers)
        self.partial = [layout == "partial" and partial_eligible(l) for l in layers]
        # a layer that runs as a partial-gather keeps the plain order (its raw aggregate is reduced across workers)
        self.layers = [engine.layer(replace(l, allow_reorder=False) if p else l, dtype) for l, p in zip(layers, self.partial)]
        self.src_part = None
        self.scale = None
        if any(self.partial):
            sp, sx, sw = source_part(indptr, indices, weights, self.v0, self.v1, self.n_table)
            self.src_part = engine.create_part(sp, sx, sw, max(self.per, 1))
            deg = np.diff(indptr)[self.v0:self.v1].astype(np.float32)
            with np.errstate(divide="ignore"):
                inv = np.where(deg > 0, np.float32(1.0) / deg, np.float32(0.0)).astype(np.float32)
            one = (deg > 0).astype(np.float32)
            pad = np.zeros(self.per - self.n_loc, np.float32)
            self.scale = {"mean": engine.to_device(np.concatenate([inv, pad])), "other": engine.to_device(np.concatenate([one, pad]))}
        self.ws = engine.workspace(self.part, self.layers)
        self.ws_src = engine.workspace(self.src_part, [l for l, p in zip(self.layers, self.partial) if p]) if self.src_part is not None else None
        fd = engine.feat_dtype(dtype)
        self.h = engine.empty(self.per, layers[0].in_dim, fd)    # padded to the common block size
        if self.n_loc:
            self.h[:self.n_loc] = x_local
        self.x0 = self.h                                          # the pass can be run again from the same input
        self._stage = None

    def reset(self):
        self.h = self.x0

    # -- before the exchange of layer i
    def pre(self, i: int) -> Exchange:
        e, lay = self.engine, self.layers[i]
        fd = e.feat_dtype(self.dtype)
        if self.partial[i]:
            sd = e.stages(self.src_part, lay)
            raw = e.empty(self.n_table, sd["agg_dim"], torch.float32)
            e.gather(self.src_part, lay, self.h, None, 0, True, raw, self.ws_src)
            op = self.layers_np[i].op
            return Exchange("reduce_scatter", table=raw, op=op if op in ("max", "min") else "sum")
        sd = e.stages(self.part, lay)
        self._stage = sd
        if sd["table_dim"] == 0:
            return Exchange("none")
        if sd["table_is_input"]:
            return Exchange("all_gather", table=self.h)
        table = e.empty(self.per, sd["table_dim"], fd)
        scores = e.empty(self.per, sd["score_dim"], torch.float32) if sd["score_dim"] else None
        if self.n_loc:
            e.transform(self.part, lay, self.h, table, scores, self.ws)
        return Exchange("all_gather", table=table, scores=scores)

    # -- after it: `table` is the all-gathered table [n_table, dim] (scores likewise), or this worker's block of the
    # reduced partial results [per, dim]
    def post(self, i: int, table, scores=None):
        e, lay, src = self.engine, self.layers[i], self.layers_np[i]
        fd = e.feat_dtype(self.dtype)
        h_next = e.empty(self.per, src.out_dim, fd)
        if self.partial[i]:
            agg = e.empty(self.per, table.shape[1], fd)
            e.finish(table, self.scale["mean" if src.op == "mean" else "other"], agg)
            if self.n_loc:
                e.update(self.part, lay, self.h, agg, h_next, self.ws)
        else:
            sd = self._stage
            if self.n_loc:
                if sd["table_dim"] == 0:                 # no Gather stage
                    e.update(self.part, lay, self.h, None, h_next, self.ws)
                elif sd["agg_dim"] == 0:                 # the gather finishes the vertex
                    e.gather(self.part, lay, table, scores, self.v0, False, h_next, self.ws)
                else:
                    agg = e.empty(self.per, sd["agg_dim"], fd)
                    e.gather(self.part, lay, table, scores, self.v0, False, agg, self.ws)
                    e.update(self.part, lay, self.h, agg, h_next, self.ws)
        self.h = h_next

    def result(self):
        return self.h[:self.n_loc]


# ----------------------------------------------------------------------------- drivers

_REDUCE = {"sum": "SUM", "max": "MAX", "min": "MIN"}


def run_spmd(worker: Worker, group=None):
    """One process per worker: the exchanges are torch.distributed collectives (NCCL between GPUs, gloo on CPU)."""
    import torch.distributed as dist
    worker.reset()
    for i in range(len(worker.layers)):
        ex = worker.pre(i)
        if ex.kind == "none":
            worker.post(i, None)
        elif ex.kind == "all_gather":
            full = torch.empty((worker.n_table, ex.table.shape[1]), dtype=ex.table.dtype, device=ex.table.device)
            dist.all_gather_into_tensor(full, ex.table.contiguous(), group=group)
            sfull = None
            if ex.scores is not None:
                sfull = torch.empty((worker.n_table, ex.scores.shape[1]), dtype=torch.float32, device=ex.scores.device)
                dist.all_gather_into_tensor(sfull, ex.scores.contiguous(), group=group)
            worker.post(i, full, sfull)
        else:
            mine = torch.empty((worker.per, ex.table.shape[1]), dtype=torch.float32, device=ex.table.device)
            op = getattr(dist.ReduceOp, _REDUCE[ex.op])
            if dist.get_backend(group) == "gloo":   # gloo has no reduce-scatter: reduce everything, keep the own block
                buf = ex.table.clone()
                dist.all_reduce(buf, op=op, group=group)
                mine.copy_(buf[worker.rank * worker.per:(worker.rank + 1) * worker.per])
            else:
                dist.reduce_scatter_tensor(mine, ex.table.contiguous(), op=op, group=group)
            worker.post(i, mine)
    return worker.result()


def run_emulated(workers: list):
    """All workers in one process, one after another (for tests on a single device): the exchange is a
    concatenation / an elementwise reduce of the workers' tables."""
    n_layers = len(workers[0].layers)
    for w in workers:
        w.reset()
    for i in range(n_layers):
        exs = [w.pre(i) for w in workers]
        kind = exs[0].kind
        assert all(e.kind == kind for e in exs)
        if kind == "none":
            for w in workers:
                w.post(i, None)
        elif kind == "all_gather":
            full = torch.cat([e.table for e in exs], dim=0)
            sfull = torch.cat([e.scores for e in exs], dim=0) if exs[0].scores is not None else None
            for w in workers:
                w.post(i, full, sfull)
        else:
            stack = torch.stack([e.table for e in exs], dim=0)
            red = {"sum": lambda t: t.sum(0), "max": lambda t: t.max(0).values, "min": lambda t: t.min(0).values}[exs[0].op](stack)
            for w in workers:
                w.post(i, red[w.rank * w.per:(w.rank + 1) * w.per].contiguous())
    return torch.cat([w.result() for w in workers], dim=0)
