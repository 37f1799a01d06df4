"""Seeded synthetic inputs (graphs, features, parameters) shared by the tests, the
benchmark and the CPU oracle's callers.  No GNN arithmetic lives here."""
from .configs import Layer, Workload, make, with_edge_features  # noqa: F401
