"""The vertex-partitioned layer pass on CPU: world_size-2 (and 3) gloo ranks run the host-side orchestration of
paper_2307_00228_b200/sharded.py with the oracle's primitives standing in for the CUDA stage calls, and the
sharded result must equal the unsharded oracle.  What is under test is the partition and exchange logic: the
ranges, the parts of the CSR, the padding of the all-gathered tables, the offsets of a worker's own rows, the
reduce of partial results."""
import os
import socket
import sys

import numpy as np
import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
sys.path.insert(0, ROOT)
sys.path.insert(0, os.path.join(ROOT, "tests"))

from oracle import oracle as O                                     # noqa: E402
from paper_2307_00228_b200 import sharded                          # noqa: E402
from workloads import Layer, rng as wrng                           # noqa: E402


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def case(seed, n=203, dtype="f32", kind="sage"):
    r = np.random.default_rng(seed)
    deg = r.integers(0, 9, size=n)
    deg[r.random(n) < 0.2] = 0
    deg[5] = 120
    ip = np.zeros(n + 1, np.int64)
    np.cumsum(deg, out=ip[1:])
    ix = r.integers(0, n, size=int(ip[-1])).astype(np.int32)
    w = r.random(ix.size, dtype=np.float32)
    x = r.standard_normal((n, 16)).astype(np.float32)

    def st(a):
        a = np.asarray(a, np.float32)
        return wrng.bf16_bits_to_f32(wrng.f32_to_bf16_bits(a)) if dtype == "bf16" else a
    x = st(x)
    mk = lambda rows, cols: st(r.uniform(-0.4, 0.4, (rows, cols)))
    b = lambda c: r.uniform(-0.1, 0.1, c).astype(np.float32)
    if kind == "sage":      # plain, then transform-first (16 -> 8), then max
        layers = [Layer("sum", "relu", 16, 16, mk(32, 16), b(16), use_edge_weights=True),
                  Layer("mean", "relu", 16, 8, mk(32, 8), b(8)),
                  Layer("max", "none", 8, 8, mk(16, 8), b(8))]
    elif kind == "gat":
        layers = [Layer("gat", "elu", 16, 16, mk(16, 16), b(16), heads=2, att_src=r.uniform(-0.4, 0.4, (2, 8)).astype(np.float32),
                        att_dst=r.uniform(-0.4, 0.4, (2, 8)).astype(np.float32)),
                  Layer("dense", "none", 16, 8, mk(16, 8), b(8))]
    else:                   # gcn, transform-first gcn, min
        layers = [Layer("gcn", "relu", 16, 16, mk(16, 16), b(16), use_edge_weights=True),
                  Layer("gcn", "relu", 16, 8, mk(16, 8), b(8)),
                  Layer("min", "none", 8, 8, mk(16, 8), b(8))]
    return ip, ix, w, x, layers


def _rank_main(rank, world, port, out_dir, seed, dtype, kind, layout):
    from sharded_util import OracleEngine
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    ip, ix, w, x, layers = case(seed, dtype=dtype, kind=kind)
    v0, v1 = sharded.vertex_ranges(ip.shape[0] - 1, world)[rank]
    eng = OracleEngine(dtype)
    xl = torch.from_numpy(x[v0:v1]).to(eng.feat_dtype(dtype))
    worker = sharded.Worker(rank, world, ip, ix, w, xl, layers, dtype, eng, layout=layout)
    res = sharded.run_spmd(worker)
    np.save(os.path.join(out_dir, f"r{rank}.npy"), res.float().numpy())
    dist.barrier()
    dist.destroy_process_group()


@pytest.mark.parametrize("world", [2, 3])
@pytest.mark.parametrize("kind,layout,dtype", [("sage", "gather", "f32"), ("sage", "gather", "bf16"), ("gat", "gather", "f32"),
                                               ("gcn", "gather", "f32"), ("sage", "partial", "f32"), ("gcn", "partial", "bf16")])
def test_sharded_pass_equals_the_unsharded_oracle(tmp_path, world, kind, layout, dtype):
    seed = 7
    mp.spawn(_rank_main, args=(world, _free_port(), str(tmp_path), seed, dtype, kind, layout), nprocs=world, join=True)
    got = np.concatenate([np.load(tmp_path / f"r{r}.npy") for r in range(world)], axis=0).astype(np.float64)
    ip, ix, w, x, layers = case(seed, dtype=dtype, kind=kind)
    if layout == "partial":   # layers that run as a partial-gather keep the plain order
        from dataclasses import replace
        layers = [replace(l, allow_reorder=False) if sharded.partial_eligible(l) else l for l in layers]
    ref = O.infer(ip, ix, w, x, layers, storage=dtype, follow_reorder=True)[-1]
    assert got.shape == ref.shape
    if layout == "gather" and dtype == "f32":
        assert np.array_equal(got, ref)        # the same arithmetic on the same rows: nothing may differ
    else:                                      # partial results pass through fp32; bf16 entries may round the other way
        tol = 1e-5 if dtype == "f32" else 2e-2
        assert np.allclose(got, ref, rtol=tol, atol=tol)


def test_ranges_and_parts_cover_the_graph_exactly_once():
    ip, ix, w, _, _ = case(3)
    n = ip.shape[0] - 1
    for world in (1, 2, 3, 5, 8):
        ranges = sharded.vertex_ranges(n, world)
        per = sharded.rows_per_worker(n, world)
        assert ranges[0][0] == 0 and ranges[-1][1] == n and all(a[1] == b[0] for a, b in zip(ranges, ranges[1:]))
        assert all(v1 - v0 <= per for v0, v1 in ranges)
        # destination parts: concatenated, they are the CSR again
        parts = [sharded.destination_part(ip, ix, w, v0, v1) for v0, v1 in ranges]
        assert np.array_equal(np.concatenate([p[1] for p in parts]), ix)
        assert np.array_equal(np.concatenate([p[2] for p in parts]), w)
        assert np.array_equal(np.concatenate([np.diff(p[0]) for p in parts]), np.diff(ip))
        # source parts: every edge is kept by exactly the worker that owns its source, order inside a destination kept
        sparts = [sharded.source_part(ip, ix, w, u0, u1, per * world) for u0, u1 in ranges]
        assert sum(p[1].size for p in sparts) == ix.size
        deg = sum(np.diff(p[0])[:n] for p in sparts)
        assert np.array_equal(deg, np.diff(ip))
        for (u0, u1), (sp, sx, sw) in zip(ranges, sparts):
            assert sp.shape[0] == per * world + 1 and (sx.size == 0 or (sx.min() >= 0 and sx.max() < u1 - u0))
            v = 5   # the hub
            mine = ix[ip[v]:ip[v + 1]]
            keep = (mine >= u0) & (mine < u1)
            assert np.array_equal(sx[sp[v]:sp[v + 1]], mine[keep] - u0)
            assert np.array_equal(sw[sp[v]:sp[v + 1]], w[ip[v]:ip[v + 1]][keep])
