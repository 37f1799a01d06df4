"""Seeded synthetic graphs in CSR-by-destination form.

The graphs follow the structure of the paper's synthetic Power-Law workload
(Section "Experiment Settings": in-degree and/or out-degree drawn from a power
law, one skewed side at a time for the in-degree experiments).  Output is the
structure only: `indptr` (int64, N+1), `indices` (int32 source ids, E).  Source
ids are ascending inside every destination segment, as in a CSR built from a
sorted edge list.

This module holds no GNN arithmetic.
"""
from __future__ import annotations

import numpy as np


def _pl_pmf(q: float, exponent: float, cap: int) -> np.ndarray:
    k = np.arange(cap + 1, dtype=np.float64)
    p = (k + q) ** (-exponent)
    return p / p.sum()


def shifted_power_law_cdf(mean: float, exponent: float, cap: int) -> np.ndarray:
    """CDF over k = 0..cap of P(k) ~ (k + q)^-exponent, q found by bisection so E[k] = mean."""
    k = np.arange(cap + 1, dtype=np.float64)
    lo, hi = 1e-6, 1e6
    for _ in range(200):
        mid = np.sqrt(lo * hi)
        m = float((_pl_pmf(mid, exponent, cap) * k).sum())
        if m < mean:
            lo = mid
        else:
            hi = mid
    cdf = np.cumsum(_pl_pmf(np.sqrt(lo * hi), exponent, cap))
    cdf[-1] = 1.0
    return cdf


def power_law_degrees(rng: np.random.Generator, n: int, e_total: int, exponent: float,
                      cap: int) -> np.ndarray:
    """n iid degrees from the shifted power law with mean e_total/n, then nudged by +-1 in
    vertex-id order (cyclically) until they sum to e_total exactly."""
    cdf = shifted_power_law_cdf(e_total / n, exponent, cap)
    deg = np.searchsorted(cdf, rng.random(n), side="left").astype(np.int64)
    np.minimum(deg, cap, out=deg)
    diff = int(e_total - deg.sum())
    while diff != 0:
        if diff > 0:
            ok = np.flatnonzero(deg < cap)[:diff]
            deg[ok] += 1
            diff -= ok.size
        else:
            ok = np.flatnonzero(deg > 0)[:-diff]
            deg[ok] -= 1
            diff += ok.size
    return deg


def _sort_within_segments(dst_of_edge: np.ndarray, src: np.ndarray) -> np.ndarray:
    key = (dst_of_edge.astype(np.uint64) << np.uint64(32)) | src.astype(np.uint64)
    key.sort(kind="stable")
    return (key & np.uint64(0xFFFFFFFF)).astype(np.int32)


def csr_from_degrees(rng: np.random.Generator, deg: np.ndarray, n_src: int,
                     source_exponent: float | None = None,
                     chunk_vertices: int = 1 << 22) -> tuple[np.ndarray, np.ndarray]:
    """Attach source ids to a degree sequence.

    source_exponent None: sources uniform over [0, n_src).
    source_exponent g:   source popularity follows a rank power law whose induced
                         out-degree distribution has tail exponent g (rank exponent
                         1/(g-1)), ranks mapped to ids through a seeded permutation.
    """
    n = deg.shape[0]
    indptr = np.zeros(n + 1, dtype=np.int64)
    np.cumsum(deg, out=indptr[1:])
    e = int(indptr[-1])
    indices = np.empty(e, dtype=np.int32)
    if source_exponent is not None:
        alpha = 1.0 / (source_exponent - 1.0)
        pop = (np.arange(n_src, dtype=np.float64) + 1.0) ** (-alpha)
        pop_cdf = np.cumsum(pop / pop.sum())
        pop_cdf[-1] = 1.0
        perm = rng.permutation(n_src).astype(np.int32)
    for v0 in range(0, n, chunk_vertices):
        v1 = min(n, v0 + chunk_vertices)
        e0, e1 = int(indptr[v0]), int(indptr[v1])
        if e1 == e0:
            continue
        if source_exponent is None:
            src = rng.integers(0, n_src, size=e1 - e0, dtype=np.int64)
        else:
            src = perm[np.searchsorted(pop_cdf, rng.random(e1 - e0), side="left")].astype(np.int64)
        dst = np.repeat(np.arange(v0, v1, dtype=np.int64), deg[v0:v1])
        indices[e0:e1] = _sort_within_segments(dst - v0, src)
    return indptr, indices


def power_law_graph(rng: np.random.Generator, n: int, e_total: int, exponent: float, cap: int,
                    source_exponent: float | None = None) -> tuple[np.ndarray, np.ndarray]:
    """Power-law in-degree graph with n vertices and exactly e_total edges."""
    deg = power_law_degrees(rng, n, e_total, exponent, min(cap, e_total))
    return csr_from_degrees(rng, deg, n, source_exponent)


def extreme_hubs_graph(rng: np.random.Generator, n: int, e_total: int, n_hubs: int,
                       hub_degree: int) -> tuple[np.ndarray, np.ndarray]:
    """n_hubs seeded vertices receive exactly hub_degree in-edges each; the remaining
    edges pick uniform destinations among the other vertices.  All sources uniform."""
    hubs = rng.choice(n, size=n_hubs, replace=False)
    is_hub = np.zeros(n, dtype=bool)
    is_hub[hubs] = True
    non_hubs = np.flatnonzero(~is_hub)
    rest = e_total - n_hubs * hub_degree
    assert rest >= 0
    deg = np.zeros(n, dtype=np.int64)
    deg[hubs] = hub_degree
    # uniform destinations among non-hubs == multinomial counts; draw by chunks of picks
    chunk = 1 << 26
    for c0 in range(0, rest, chunk):
        m = min(chunk, rest - c0)
        picks = rng.integers(0, non_hubs.size, size=m, dtype=np.int64)
        deg[non_hubs] += np.bincount(picks, minlength=non_hubs.size)
    return csr_from_degrees(rng, deg, n, None)
