"""Host-side helpers around the binding: move a synthetic workload to the device and run it.
Marshalling only — no layer arithmetic happens here."""
from __future__ import annotations

from dataclasses import dataclass

import numpy as np
import torch

from . import binding as B


def features_to_device(x: np.ndarray, dtype: str, device="cuda", pinned=False) -> torch.Tensor:
    """float32 array, or uint16 bfloat16 bit patterns, -> device tensor of that dtype."""
    t = torch.from_numpy(x) if dtype == "f32" else torch.from_numpy(x.view(np.int16)).view(torch.bfloat16)
    if pinned:
        t = t.pin_memory()
    return t.to(device, non_blocking=pinned)


def param_to_device(a: np.ndarray, dtype: str, device="cuda") -> torch.Tensor:
    t = torch.from_numpy(np.ascontiguousarray(a, dtype=np.float32)).to(device)
    return t.to(torch.bfloat16) if dtype == "bf16" else t


def layer_to_device(layer, dtype: str, device="cuda") -> B.LayerDesc:
    f32 = lambda a: None if a is None else torch.from_numpy(np.ascontiguousarray(a, dtype=np.float32)).to(device)
    return B.LayerDesc(op=layer.op, act=layer.act, in_dim=layer.in_dim, out_dim=layer.out_dim,
                       W=param_to_device(layer.W, dtype, device), bias=f32(layer.bias), heads=layer.heads,
                       att_src=f32(layer.att_src), att_dst=f32(layer.att_dst), leaky_slope=float(layer.leaky_slope),
                       use_edge_weights=bool(layer.use_edge_weights), allow_reorder=bool(layer.allow_reorder),
                       edge_dim=int(getattr(layer, "edge_dim", 0) or 0), msg_dim=int(getattr(layer, "msg_dim", 0) or 0),
                       W_edge=None if getattr(layer, "W_edge", None) is None else param_to_device(layer.W_edge, dtype, device),
                       bias_edge=f32(getattr(layer, "bias_edge", None)), act_edge=getattr(layer, "act_edge", "none"),
                       att_edge=f32(getattr(layer, "att_edge", None)))


@dataclass
class DeviceWorkload:
    graph: B.Graph
    x: torch.Tensor
    layers: list
    workspace: torch.Tensor
    out: torch.Tensor
    n_rows: int
    n_split_owners: int

    def infer(self, stream=None) -> torch.Tensor:
        return B.it_infer(self.graph, self.layers, self.x, self.out, self.workspace, stream)


def upload(w, device="cuda", int32_indptr=False, threshold=None, with_workspace=True) -> DeviceWorkload:
    """Create the device graph (split at the workload's threshold), parameters, workspace, output.
    with_workspace=False: a second set of input / output buffers for a caller that shares one workspace and one set of
    layer parameters between them (layers and workspace are left empty)."""
    indptr = torch.from_numpy(w.indptr.astype(np.int32) if int32_indptr else w.indptr).to(device)
    indices = torch.from_numpy(w.indices).to(device)
    ew = None if w.edge_weights is None else torch.from_numpy(w.edge_weights).to(device)
    g = B.it_graph_create(indptr, indices, ew)
    if getattr(w, "edge_feat", None) is not None:
        B.it_graph_set_edge_features(g, features_to_device(w.edge_feat, w.dtype, device))
    thr = w.threshold if threshold is None else threshold
    n_rows, n_split = B.it_split_hubs(g, thr)
    x = features_to_device(w.x, w.dtype, device)
    if not with_workspace:
        out = torch.empty((w.n, w.layers[-1].out_dim), dtype=x.dtype, device=device)
        return DeviceWorkload(g, x, [], None, out, n_rows, n_split)
    layers = [layer_to_device(l, w.dtype, device) for l in w.layers]
    ws = torch.empty(B.it_workspace_bytes(g, layers), dtype=torch.uint8, device=device)
    out = torch.empty((w.n, w.layers[-1].out_dim), dtype=x.dtype, device=device)
    return DeviceWorkload(g, x, layers, ws, out, n_rows, n_split)
