"""ctypes binding of libinferturbo.so: the same entry points as include/inferturbo.h, with
argument marshalling only.  PyTorch supplies device memory and streams; every step of the
layer pass runs in the library's CUDA kernels.  There is no CPU path: loading fails loudly if
the library has not been built.
"""
from __future__ import annotations

import ctypes as C
import os
from dataclasses import dataclass

import torch

_PKG = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.environ.get("INFERTURBO_LIB") or os.path.join(_PKG, "libinferturbo.so")

IT_OK = 0
STATUS_NAMES = ["IT_OK", "IT_ERR_INVALID_ARG", "IT_ERR_BAD_GRAPH", "IT_ERR_UNSUPPORTED", "IT_ERR_WORKSPACE",
                "IT_ERR_OOM", "IT_ERR_CUDA", "IT_ERR_TIMEOUT"]
IT_F32, IT_BF16 = 0, 1
IT_I32, IT_I64 = 0, 1
GATHER_OPS = {"sum": 0, "mean": 1, "max": 2, "gat": 3, "min": 4, "dense": 5, "gcn": 6}
ACTS = {"none": 0, "relu": 1, "elu": 2}
IT_MAX_BUCKETS = 8
EXPORTS = ["it_graph_create", "it_split_hubs", "it_graph_get_split", "it_workspace_bytes", "it_layer_forward",
           "it_infer", "it_graph_destroy", "it_status_string", "it_last_error_message", "it_profile_begin",
           "it_profile_end", "it_kernel_launch_count", "it_layer_forward_static", "it_graph_check",
           "it_graph_set_edge_features", "it_debug_expire_wait", "it_graph_create_part", "it_layer_stages",
           "it_layer_transform", "it_layer_gather", "it_layer_update", "it_aggregate_finish", "it_debug_expire_wait_fused"]


class ItError(RuntimeError):
    def __init__(self, status: int, message: str):
        self.status = status
        self.status_name = STATUS_NAMES[status] if 0 <= status < len(STATUS_NAMES) else f"status {status}"
        super().__init__(f"{self.status_name}: {message}")


class it_layer_desc(C.Structure):
    _fields_ = [("op", C.c_int), ("act", C.c_int),
                ("in_dim", C.c_int32), ("out_dim", C.c_int32), ("heads", C.c_int32),
                ("feat_dtype", C.c_int), ("weight_dtype", C.c_int),
                ("W", C.c_void_p), ("bias", C.c_void_p), ("att_src", C.c_void_p), ("att_dst", C.c_void_p),
                ("leaky_slope", C.c_float), ("use_edge_weights", C.c_int32), ("allow_reorder", C.c_int32),
                ("edge_dim", C.c_int32), ("msg_dim", C.c_int32), ("act_edge", C.c_int),
                ("W_edge", C.c_void_p), ("bias_edge", C.c_void_p), ("att_edge", C.c_void_p)]


class it_stage_desc(C.Structure):
    _fields_ = [("table_dim", C.c_int32), ("table_dtype", C.c_int), ("score_dim", C.c_int32),
                ("table_is_input", C.c_int32), ("agg_dim", C.c_int32)]


_lib = None


def lib() -> C.CDLL:
    """Load the CUDA library (raises if it is missing: there is no fallback)."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise ImportError(f"{LIB_PATH} not found: build it with `python -m paper_2307_00228_b200.build`")
        L = C.CDLL(LIB_PATH)
        vp, i64, i32 = C.c_void_p, C.c_int64, C.c_int32
        L.it_graph_create.argtypes = [i64, i64, vp, C.c_int, vp, vp, vp, C.POINTER(vp)]
        L.it_split_hubs.argtypes = [vp, i64, vp, C.POINTER(i64), C.POINTER(i64)]
        L.it_graph_get_split.argtypes = [vp, C.POINTER(i64), C.POINTER(vp), C.POINTER(vp), C.POINTER(vp), C.POINTER(vp),
                                         C.POINTER(vp), C.POINTER(i32), C.POINTER(i64)]
        L.it_workspace_bytes.argtypes = [vp, C.POINTER(it_layer_desc), i32, C.POINTER(C.c_size_t)]
        L.it_layer_forward.argtypes = [vp, C.POINTER(it_layer_desc), vp, vp, vp, C.c_size_t, vp]
        L.it_infer.argtypes = [vp, C.POINTER(it_layer_desc), i32, vp, vp, vp, C.c_size_t, vp]
        L.it_graph_destroy.argtypes = [vp]
        L.it_graph_create_part.argtypes = [i64, i64, i64, vp, C.c_int, vp, vp, vp, C.POINTER(vp)]
        L.it_layer_stages.argtypes = [vp, C.POINTER(it_layer_desc), C.POINTER(it_stage_desc)]
        L.it_layer_transform.argtypes = [vp, C.POINTER(it_layer_desc), vp, vp, vp, vp, C.c_size_t, vp]
        L.it_layer_gather.argtypes = [vp, C.POINTER(it_layer_desc), vp, vp, i64, i32, vp, vp, C.c_size_t, vp]
        L.it_layer_update.argtypes = [vp, C.POINTER(it_layer_desc), vp, vp, vp, vp, C.c_size_t, vp]
        L.it_aggregate_finish.argtypes = [i64, i32, C.c_int, vp, vp, vp, vp]
        for name in ("it_graph_create_part", "it_layer_stages", "it_layer_transform", "it_layer_gather", "it_layer_update",
                     "it_aggregate_finish"):
            getattr(L, name).restype = C.c_int
        for name in EXPORTS[:7]:
            getattr(L, name).restype = C.c_int
        L.it_status_string.argtypes = [C.c_int]
        L.it_status_string.restype = C.c_char_p
        L.it_last_error_message.restype = C.c_char_p
        _lib = L
    return _lib


def _check(status: int):
    if status != IT_OK:
        raise ItError(status, lib().it_last_error_message().decode())


def _ptr(t):
    return None if t is None else C.c_void_p(t.data_ptr())


def _stream(stream=None):
    s = torch.cuda.current_stream() if stream is None else stream
    return C.c_void_p(s.cuda_stream)


def _dt(t: torch.dtype) -> int:
    if t == torch.float32:
        return IT_F32
    if t == torch.bfloat16:
        return IT_BF16
    raise TypeError(f"unsupported feature dtype {t}")


@dataclass
class LayerDesc:
    """Python mirror of it_layer_desc; tensors are CUDA tensors kept alive by this object."""
    op: str
    act: str
    in_dim: int
    out_dim: int
    W: torch.Tensor
    bias: torch.Tensor | None = None
    heads: int = 1
    att_src: torch.Tensor | None = None
    att_dst: torch.Tensor | None = None
    leaky_slope: float = 0.2
    use_edge_weights: bool = False
    allow_reorder: bool = True
    edge_dim: int = 0
    msg_dim: int = 0
    W_edge: torch.Tensor | None = None
    bias_edge: torch.Tensor | None = None
    act_edge: str = "none"
    att_edge: torch.Tensor | None = None

    def to_c(self) -> it_layer_desc:
        for t in (self.W, self.bias, self.att_src, self.att_dst, self.W_edge, self.bias_edge, self.att_edge):
            assert t is None or (t.is_cuda and t.is_contiguous())
        for t in (self.bias, self.att_src, self.att_dst, self.bias_edge, self.att_edge):
            assert t is None or t.dtype == torch.float32
        assert self.W_edge is None or self.W_edge.dtype == self.W.dtype
        d = it_layer_desc()
        d.op, d.act = GATHER_OPS[self.op], ACTS[self.act]
        d.in_dim, d.out_dim, d.heads = self.in_dim, self.out_dim, self.heads
        d.feat_dtype = d.weight_dtype = _dt(self.W.dtype)
        d.W = self.W.data_ptr()
        d.bias = None if self.bias is None else self.bias.data_ptr()
        d.att_src = None if self.att_src is None else self.att_src.data_ptr()
        d.att_dst = None if self.att_dst is None else self.att_dst.data_ptr()
        d.leaky_slope = self.leaky_slope
        d.use_edge_weights = int(self.use_edge_weights)
        d.allow_reorder = int(self.allow_reorder)
        d.edge_dim = int(self.edge_dim)
        d.msg_dim = int(self.msg_dim)
        d.act_edge = ACTS[self.act_edge]
        d.W_edge = None if self.W_edge is None else self.W_edge.data_ptr()
        d.bias_edge = None if self.bias_edge is None else self.bias_edge.data_ptr()
        d.att_edge = None if self.att_edge is None else self.att_edge.data_ptr()
        return d


def _c_layers(layers):
    arr = (it_layer_desc * len(layers))()
    for i, l in enumerate(layers):
        arr[i] = l.to_c() if isinstance(l, LayerDesc) else l
    return arr


class Graph:
    """Owner of an it_graph handle.  Keeps the borrowed CSR tensors alive."""

    def __init__(self, handle, n, e, keep):
        self.handle, self.n, self.e, self._keep = handle, n, e, keep

    def __del__(self):
        try:
            it_graph_destroy(self)
        except Exception:
            pass


def it_graph_create(indptr: torch.Tensor, indices: torch.Tensor, edge_weights: torch.Tensor | None = None,
                    stream=None, n_vertices: int | None = None, n_edges: int | None = None) -> Graph:
    assert indptr.is_cuda and indptr.is_contiguous() and indptr.dtype in (torch.int32, torch.int64)
    assert indices.dtype == torch.int32 and indices.is_contiguous() and (indices.is_cuda or indices.numel() == 0)
    assert edge_weights is None or (edge_weights.is_cuda and edge_weights.dtype == torch.float32 and edge_weights.is_contiguous())
    n = indptr.numel() - 1 if n_vertices is None else n_vertices
    e = indices.numel() if n_edges is None else n_edges
    out = C.c_void_p()
    _check(lib().it_graph_create(n, e, _ptr(indptr), IT_I64 if indptr.dtype == torch.int64 else IT_I32,
                                 _ptr(indices), _ptr(edge_weights), _stream(stream), C.byref(out)))
    return Graph(out, n, e, (indptr, indices, edge_weights))


def it_graph_create_part(indptr: torch.Tensor, indices: torch.Tensor, n_sources: int, edge_weights: torch.Tensor | None = None,
                         stream=None) -> Graph:
    """One part of a vertex-partitioned graph: the in-edges of len(indptr) - 1 local destinations, source ids
    naming rows of a table of n_sources rows."""
    assert indptr.is_cuda and indptr.is_contiguous() and indptr.dtype in (torch.int32, torch.int64)
    assert indices.dtype == torch.int32 and indices.is_contiguous() and (indices.is_cuda or indices.numel() == 0)
    assert edge_weights is None or (edge_weights.is_cuda and edge_weights.dtype == torch.float32 and edge_weights.is_contiguous())
    n, e = indptr.numel() - 1, indices.numel()
    out = C.c_void_p()
    _check(lib().it_graph_create_part(n, n_sources, e, _ptr(indptr), IT_I64 if indptr.dtype == torch.int64 else IT_I32,
                                      _ptr(indices), _ptr(edge_weights), _stream(stream), C.byref(out)))
    g = Graph(out, n, e, (indptr, indices, edge_weights))
    g.n_sources = n_sources
    return g


def it_layer_stages(g: Graph, layer) -> dict:
    """What the stage calls of this layer exchange: table_dim, table_dtype, score_dim, table_is_input, agg_dim."""
    d = it_stage_desc()
    _check(lib().it_layer_stages(g.handle, _c_layers([layer]), C.byref(d)))
    return {"table_dim": d.table_dim, "table_dtype": torch.float32 if d.table_dtype == IT_F32 else torch.bfloat16,
            "score_dim": d.score_dim, "table_is_input": bool(d.table_is_input), "agg_dim": d.agg_dim}


def _nbytes(t):
    return t.numel() * t.element_size()


def it_layer_transform(g: Graph, layer, h_self, table_out, scores_out, workspace, stream=None):
    _check(lib().it_layer_transform(g.handle, _c_layers([layer]), _ptr(h_self), _ptr(table_out), _ptr(scores_out),
                                    _ptr(workspace), _nbytes(workspace), _stream(stream)))


def it_layer_gather(g: Graph, layer, table, scores, first_vertex: int, raw_partial: bool, out, workspace, stream=None):
    _check(lib().it_layer_gather(g.handle, _c_layers([layer]), _ptr(table), _ptr(scores), first_vertex, int(raw_partial),
                                 _ptr(out), _ptr(workspace), _nbytes(workspace), _stream(stream)))


def it_layer_update(g: Graph, layer, h_self, agg, h_out, workspace, stream=None):
    _check(lib().it_layer_update(g.handle, _c_layers([layer]), _ptr(h_self), _ptr(agg), _ptr(h_out), _ptr(workspace),
                                 _nbytes(workspace), _stream(stream)))


def it_aggregate_finish(raw: torch.Tensor, scale: torch.Tensor, out: torch.Tensor, stream=None):
    """out[v, :] = raw[v, :] * scale[v] (0 where scale[v] = 0); raw fp32 [n, dim], scale fp32 [n]."""
    assert raw.dtype == torch.float32 and scale.dtype == torch.float32 and raw.is_contiguous() and out.is_contiguous()
    _check(lib().it_aggregate_finish(raw.shape[0], raw.shape[1], _dt(out.dtype), _ptr(raw), _ptr(scale), _ptr(out), _stream(stream)))
    return out


def it_graph_set_edge_features(g: Graph, edge_feat: torch.Tensor | None):
    """Attach [n_edges, edge_dim] edge features (CSR order), or detach them with None."""
    L = lib()
    L.it_graph_set_edge_features.restype = C.c_int
    L.it_graph_set_edge_features.argtypes = [C.c_void_p, C.c_void_p, C.c_int32, C.c_int]
    if edge_feat is None:
        _check(L.it_graph_set_edge_features(g.handle, None, 0, IT_F32))
        g._edge_feat = None
        return
    assert edge_feat.is_cuda and edge_feat.is_contiguous() and edge_feat.dim() == 2 and edge_feat.shape[0] == g.e
    _check(L.it_graph_set_edge_features(g.handle, _ptr(edge_feat), edge_feat.shape[1], _dt(edge_feat.dtype)))
    g._edge_feat = edge_feat   # borrowed by the library: keep it alive


def it_split_hubs(g: Graph, threshold: int, stream=None):
    """Returns (n_rows, n_split_owners)."""
    r, s = C.c_int64(), C.c_int64()
    _check(lib().it_split_hubs(g.handle, threshold, _stream(stream), C.byref(r), C.byref(s)))
    return r.value, s.value


class _DevArray:
    """Minimal __cuda_array_interface__ holder so torch can view library-owned device memory."""

    def __init__(self, ptr, count, typestr):
        self.__cuda_array_interface__ = {"shape": (count,), "typestr": typestr, "data": (ptr, False), "version": 2}


def _borrow(ptr, count, dtype, device):
    """Copy `count` elements at device address `ptr` into a new tensor (read-only peek for tests)."""
    if count == 0 or not ptr:
        return torch.empty(0, dtype=dtype, device=device)
    typestr = {torch.int64: "<i8", torch.int32: "<i4"}[dtype]
    return torch.as_tensor(_DevArray(ptr, count, typestr), device=device).clone()


def it_graph_get_split(g: Graph) -> dict:
    """Copies of the derived index arrays (device tensors) and the bucket bounds (host list)."""
    n_rows, nb = C.c_int64(), C.c_int32()
    sp, so, op, bo, br = (C.c_void_p() for _ in range(5))
    bounds = (C.c_int64 * IT_MAX_BUCKETS)()
    _check(lib().it_graph_get_split(g.handle, C.byref(n_rows), C.byref(sp), C.byref(so), C.byref(op), C.byref(bo),
                                    C.byref(br), C.byref(nb), bounds))
    R, dev = n_rows.value, g._keep[0].device
    torch.cuda.synchronize()
    return {
        "n_rows": R,
        "shadow_indptr": _borrow(sp.value, R + 1, torch.int64, dev),
        "shadow_owner": _borrow(so.value, R, torch.int32, dev),
        "owner_indptr": _borrow(op.value, g.n + 1, torch.int64, dev),
        "bucket_offsets": _borrow(bo.value, nb.value + 1, torch.int64, dev),
        "bucket_rows": _borrow(br.value, R, torch.int32, dev),
        "bucket_bounds": list(bounds)[:nb.value],
    }


def it_workspace_bytes(g: Graph, layers) -> int:
    out = C.c_size_t()
    arr = _c_layers(layers)
    _check(lib().it_workspace_bytes(g.handle, arr, len(layers), C.byref(out)))
    return out.value


def it_layer_forward(g: Graph, layer, h_in: torch.Tensor, h_out: torch.Tensor, workspace: torch.Tensor, stream=None):
    assert h_in.is_contiguous() and h_out.is_contiguous() and workspace.is_contiguous()
    arr = _c_layers([layer])
    _check(lib().it_layer_forward(g.handle, arr, _ptr(h_in), _ptr(h_out), _ptr(workspace),
                                  workspace.numel() * workspace.element_size(), _stream(stream)))
    return h_out


STATIC_WORKSPACE_BYTES = 32 << 20


def it_layer_forward_static(g: Graph, layer, h_in: torch.Tensor, h_out: torch.Tensor, stream=None):
    """it_layer_forward without a caller workspace, for callers that cannot allocate device
    memory: the scratch is a fixed STATIC_WORKSPACE_BYTES array inside the library, shared by
    all calls on a device (so calls that could overlap on the GPU must be serialised).  Layers
    that need more scratch raise ItError(IT_ERR_WORKSPACE).  Make the first call during set-up."""
    assert h_in.is_contiguous() and h_out.is_contiguous()
    L = lib()
    L.it_layer_forward_static.restype = C.c_int
    L.it_layer_forward_static.argtypes = [C.c_void_p, C.POINTER(it_layer_desc), C.c_void_p, C.c_void_p, C.c_void_p]
    arr = _c_layers([layer])
    _check(L.it_layer_forward_static(g.handle, arr, _ptr(h_in), _ptr(h_out), _stream(stream)))
    return h_out


def it_infer(g: Graph, layers, x: torch.Tensor, out: torch.Tensor, workspace: torch.Tensor, stream=None):
    assert x.is_contiguous() and out.is_contiguous() and workspace.is_contiguous()
    arr = _c_layers(layers)
    _check(lib().it_infer(g.handle, arr, len(layers), _ptr(x), _ptr(out), _ptr(workspace),
                          workspace.numel() * workspace.element_size(), _stream(stream)))
    return out


def it_graph_check(g: Graph, stream=None):
    """Synchronise the stream; raises ItError(IT_ERR_TIMEOUT) if a kernel gave up a bounded wait."""
    L = lib()
    L.it_graph_check.restype = C.c_int
    L.it_graph_check.argtypes = [C.c_void_p, C.c_void_p]
    _check(L.it_graph_check(g.handle, _stream(stream)))


def it_debug_expire_wait(g: Graph, x: torch.Tensor, out: torch.Tensor, workspace: torch.Tensor, stream=None):
    """Test hook: run the tensor-core apply with its producer off so that its bounded waits run out."""
    L = lib()
    L.it_debug_expire_wait.restype = C.c_int
    L.it_debug_expire_wait.argtypes = [C.c_void_p, C.c_int, C.c_void_p, C.c_void_p, C.c_void_p, C.c_size_t, C.c_void_p]
    _check(L.it_debug_expire_wait(g.handle, _dt(x.dtype), _ptr(x), _ptr(out), _ptr(workspace),
                                  workspace.numel() * workspace.element_size(), _stream(stream)))


def it_debug_expire_wait_fused(g: Graph, x: torch.Tensor, out: torch.Tensor, workspace: torch.Tensor, stream=None):
    """Test hook: the same for the kernel that runs two products back to back (bf16 [128, 64] in and out)."""
    L = lib()
    L.it_debug_expire_wait_fused.restype = C.c_int
    L.it_debug_expire_wait_fused.argtypes = [C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.c_size_t, C.c_void_p]
    _check(L.it_debug_expire_wait_fused(g.handle, _ptr(x), _ptr(out), _ptr(workspace),
                                        workspace.numel() * workspace.element_size(), _stream(stream)))


def it_graph_destroy(g: Graph):
    if g is not None and g.handle is not None and g.handle.value:
        lib().it_graph_destroy(g.handle)
        g.handle = None


class it_kernel_stat(C.Structure):
    _fields_ = [("name", C.c_char * 32), ("launches", C.c_int64), ("total_ms", C.c_double),
                ("algo_bytes", C.c_double), ("algo_flops", C.c_double)]


def it_profile_begin():
    lib().it_profile_begin.restype = C.c_int
    _check(lib().it_profile_begin())


def it_profile_end() -> list:
    """Per kernel kind: {'name', 'launches', 'total_ms', 'algo_bytes', 'algo_flops'}."""
    L = lib()
    L.it_profile_end.restype = C.c_int
    L.it_profile_end.argtypes = [C.POINTER(it_kernel_stat), C.c_int32, C.POINTER(C.c_int32)]
    arr = (it_kernel_stat * 32)()
    n = C.c_int32()
    _check(L.it_profile_end(arr, 32, C.byref(n)))
    return [{"name": arr[i].name.decode(), "launches": arr[i].launches, "total_ms": arr[i].total_ms,
             "algo_bytes": arr[i].algo_bytes, "algo_flops": arr[i].algo_flops} for i in range(min(n.value, 32))]


def it_kernel_launch_count() -> int:
    lib().it_kernel_launch_count.restype = C.c_int64
    return lib().it_kernel_launch_count()


def it_status_string(status: int) -> str:
    return lib().it_status_string(status).decode()


def it_last_error_message() -> str:
    return lib().it_last_error_message().decode()
