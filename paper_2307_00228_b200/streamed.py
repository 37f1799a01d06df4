"""The layer pass over a graph whose edge arrays do not stay in device memory.

The paper's MapReduce backend handles inputs that exceed a worker's memory by keeping them in external storage and
loading a part of a partition at a time (Section "InferTurbo on MapReduce").  The analogue on one GPU: the vertex
tables (layer inputs and outputs, one row per vertex) stay in HBM, because the gather reads them at random, while
the edge arrays (source ids and edge weights, 4 + 4 bytes per edge, the bulk of a graph with many edges) stay in
page-locked host memory and are streamed through two staging buffers, one block of destinations at a time: while
the kernels of block k run, the copy of block k + 1 is in flight on a second stream.

A block is a part of the graph in the sense of it_graph_create_part (the in-edges of a range of destinations,
source ids global), so the pass is the vertex-partitioned pass of `sharded.py` with one process playing every
worker in turn, and a Gather stage that first waits for its block's edges.  The derived arrays of a block (its row
split and degree buckets, 28 bytes per vertex) are built once and stay resident.

Host-side orchestration only: every step of a layer runs in the library's kernels.
"""
from __future__ import annotations

import numpy as np
import torch

from . import sharded


class StreamingEngine(sharded.CudaEngine):
    """CudaEngine whose graph parts borrow their edge arrays from two shared staging buffers that are refilled from
    page-locked host memory before the part's Gather stage runs."""

    def __init__(self, max_block_edges: int, has_weights: bool, threshold: int = 0, device="cuda"):
        super().__init__(threshold, device)
        cap = max(1, max_block_edges)
        self.stage_idx = [torch.empty(cap, dtype=torch.int32, device=device) for _ in range(2)]
        self.stage_w = [torch.empty(cap, dtype=torch.float32, device=device) for _ in range(2)] if has_weights else [None, None]
        self.copy_stream = torch.cuda.Stream(device=device)
        self.parts = []                 # creation order = the order in which the blocks are walked
        self.resident = [None, None]    # which part's edges each staging buffer holds
        self.free_event = [None, None]  # recorded on the compute stream after the last kernel that read the buffer
        self.ready_event = [None, None]  # recorded on the copy stream after the buffer was filled
        self.h2d_bytes = 0

    def create_part(self, indptr, indices, weights, n_sources):
        k = len(self.parts)
        slot = k % 2
        host_idx = torch.from_numpy(np.ascontiguousarray(indices)).pin_memory()
        host_w = None if weights is None else torch.from_numpy(np.ascontiguousarray(weights)).pin_memory()
        e = host_idx.numel()
        torch.cuda.current_stream().synchronize()   # set-up: the buffer's previous part has been validated and split
        self.stage_idx[slot][:e].copy_(host_idx)
        if host_w is not None:
            self.stage_w[slot][:e].copy_(host_w)
        g = self.B.it_graph_create_part(self.to_device(indptr), self.stage_idx[slot][:e],
                                        n_sources, None if host_w is None else self.stage_w[slot][:e])
        self.B.it_split_hubs(g, self.threshold)
        g._stream_slot, g._host_idx, g._host_w, g._order = slot, host_idx, host_w, k
        self.parts.append(g)
        self.resident[slot] = k
        return g

    def _fill(self, part):
        """Enqueue the copy of `part`'s edge arrays into its staging buffer on the copy stream, after the kernels
        that still read the buffer's previous contents."""
        slot = part._stream_slot
        if self.resident[slot] == part._order:
            return
        with torch.cuda.stream(self.copy_stream):
            if self.free_event[slot] is not None:
                self.copy_stream.wait_event(self.free_event[slot])
            e = part._host_idx.numel()
            self.stage_idx[slot][:e].copy_(part._host_idx, non_blocking=True)
            self.h2d_bytes += e * 4
            if part._host_w is not None:
                self.stage_w[slot][:e].copy_(part._host_w, non_blocking=True)
                self.h2d_bytes += e * 4
            ev = torch.cuda.Event()
            ev.record(self.copy_stream)
            self.ready_event[slot] = ev
        self.resident[slot] = part._order

    def gather(self, part, layer, table, scores, first, raw, out, ws):
        slot = part._stream_slot
        self._fill(part)
        compute = torch.cuda.current_stream()
        if self.ready_event[slot] is not None:
            compute.wait_event(self.ready_event[slot])
        super().gather(part, layer, table, scores, first, raw, out, ws)
        ev = torch.cuda.Event()
        ev.record(compute)
        self.free_event[slot] = ev
        # the next block's copy overlaps these kernels (its buffer is the other one)
        nxt = self.parts[(part._order + 1) % len(self.parts)]
        if nxt is not part:
            self._fill(nxt)


class StreamedPass:
    """L layers over a graph given as host arrays, `block_vertices` destinations at a time."""

    def __init__(self, indptr: np.ndarray, indices: np.ndarray, weights, x: torch.Tensor, layers, dtype: str,
                 block_vertices: int, threshold: int = 0):
        n = indptr.shape[0] - 1
        self.n_blocks = max(1, -(-n // max(1, block_vertices)))
        ranges = sharded.vertex_ranges(n, self.n_blocks)
        max_edges = max(int(indptr[v1] - indptr[v0]) for v0, v1 in ranges)
        self.engine = StreamingEngine(max_edges, weights is not None, threshold)
        self.workers = [sharded.Worker(b, self.n_blocks, indptr, indices, weights, x[v0:v1], layers, dtype, self.engine, layout="gather")
                        for b, (v0, v1) in enumerate(ranges)]
        self.staging_bytes = 2 * max_edges * (4 + (4 if weights is not None else 0))
        self.edge_bytes = int(indices.size) * (4 + (4 if weights is not None else 0))

    def infer(self) -> torch.Tensor:
        """Runs every layer; returns the output [n, out_dim] (device).  Asynchronous on the current stream."""
        return sharded.run_emulated(self.workers)
