"""Seeded random streams for the synthetic workloads.

Every array a workload needs (graph structure, features, edge weights, layer
weights, biases) is drawn from its own counter-based Philox stream keyed by
(seed, purpose), so one array can be regenerated without touching the others
and the result does not depend on generation order.

This module holds no GNN arithmetic: it only produces inputs.
"""
from __future__ import annotations

import numpy as np

# Fixed seed per purpose, shared by all configs.
SEED_WEIGHTS = 0
SEED_GRAPH = 1
SEED_FEATURES = 2
SEED_EDGE_WEIGHTS = 3
SEED_BIAS = 4
SEED_EDGE_FEATURES = 5


def stream(seed: int, substream: int = 0) -> np.random.Generator:
    """A Philox generator keyed by (seed, substream)."""
    key = np.array([np.uint64(seed), np.uint64(substream)], dtype=np.uint64)
    return np.random.Generator(np.random.Philox(key=key))


def f32_to_bf16_bits(x: np.ndarray) -> np.ndarray:
    """Round float32 to bfloat16 (round-to-nearest-even); returns uint16 bit patterns."""
    x = np.ascontiguousarray(x, dtype=np.float32)
    u = x.view(np.uint32)
    lsb = (u >> np.uint32(16)) & np.uint32(1)
    r = u + np.uint32(0x7FFF) + lsb
    out = (r >> np.uint32(16)).astype(np.uint16)
    nan = np.isnan(x)
    if nan.any():
        out[nan] = np.uint16(0x7FC0)
    return out


def bf16_bits_to_f32(b: np.ndarray) -> np.ndarray:
    """Widen bfloat16 bit patterns (uint16) to float32, exactly."""
    b = np.ascontiguousarray(b, dtype=np.uint16)
    return (b.astype(np.uint32) << np.uint32(16)).view(np.float32)


def normal_f32(rng: np.random.Generator, shape, chunk_rows: int = 1 << 20) -> np.ndarray:
    """float32 N(0,1) of the given 2-D shape, drawn in row chunks to bound temporaries."""
    n, f = shape
    out = np.empty((n, f), dtype=np.float32)
    for r0 in range(0, n, chunk_rows):
        r1 = min(n, r0 + chunk_rows)
        out[r0:r1] = rng.standard_normal((r1 - r0, f), dtype=np.float32)
    return out


def normal_bf16_bits(rng: np.random.Generator, shape, chunk_rows: int = 1 << 20) -> np.ndarray:
    """bfloat16 bit patterns of N(0,1) samples (float32 draws rounded to nearest even)."""
    n, f = shape
    out = np.empty((n, f), dtype=np.uint16)
    for r0 in range(0, n, chunk_rows):
        r1 = min(n, r0 + chunk_rows)
        out[r0:r1] = f32_to_bf16_bits(rng.standard_normal((r1 - r0, f), dtype=np.float32))
    return out
