"""Python face of the CPU oracle (TEST INFRASTRUCTURE ONLY).

Thin ctypes wrappers over `it_oracle.c` plus the layer-by-layer driver that strings
them together the way the paper does: k layers = k passes over every vertex, each
vertex used once per layer, no sampling (Section "Alternative Backends and
Implementation Details", Execution: one iteration per layer, the k-layer result after k
of them).  Nothing here is shared with, or imported by, the CUDA library.

Storage points.  The method itself is exact, but a deployment stores layer inputs and
outputs in a narrow type.  `storage=None` keeps everything in fp64 (mode A).  With
`storage='f32'|'bf16'` (mode B) the oracle still accumulates in fp64 but rounds to the
storage type (nearest even) at the points where the layer contract says a tensor is
stored: the aggregate handed to apply, the transformed rows Z and the self term (GAT and
transform-before-aggregate) and the layer output.  The GAT scores are contract-fp32 and
are rounded to fp32.
"""
from __future__ import annotations

import ctypes as C
import os
import subprocess

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SO = os.path.join(_HERE, "libit_oracle.so")
_SRC = os.path.join(_HERE, "it_oracle.c")

OPS = {"sum": 0, "mean": 1, "max": 2, "min": 3}
ACTS = {"none": 0, "relu": 1, "elu": 2}


def build(force: bool = False) -> str:
    """Compile it_oracle.c into libit_oracle.so next to it (gcc, OpenMP)."""
    if force or not os.path.exists(_SO) or os.path.getmtime(_SO) < os.path.getmtime(_SRC):
        subprocess.check_call(["gcc", "-O2", "-fopenmp", "-fPIC", "-shared", "-std=c99",
                               "-o", _SO, _SRC, "-lm"])
    return _SO


_lib = None


def lib():
    global _lib
    if _lib is None:
        _lib = C.CDLL(build())
        _lib.ito_split_count.restype = C.c_int64
        _lib.ito_buckets.restype = C.c_int
    return _lib


def _p(a):
    return None if a is None else a.ctypes.data_as(C.c_void_p)


def _f64(a):
    return None if a is None else np.ascontiguousarray(a, dtype=np.float64)


def _i64(a):
    return np.ascontiguousarray(a, dtype=np.int64)


def _i32(a):
    return np.ascontiguousarray(a, dtype=np.int32)


# ----------------------------------------------------------------- rounding helpers

def round_bf16(x: np.ndarray) -> np.ndarray:
    """fp64 -> nearest bfloat16 (ties to even), returned as fp64.  Done directly on the
    fp64 bit pattern (keep 7 fraction bits) for values in bfloat16's normal range; tiny
    values go through fp32 first so subnormals and underflow behave like hardware."""
    x = np.ascontiguousarray(x, dtype=np.float64)
    u = x.view(np.uint64)
    drop = np.uint64(52 - 7)
    lsb = (u >> drop) & np.uint64(1)
    r = (u + ((np.uint64(1) << (drop - np.uint64(1))) - np.uint64(1)) + lsb) >> drop << drop
    out = r.view(np.float64).copy()
    small = np.abs(x) < 2.0 ** -120
    if small.any():
        f = x[small].astype(np.float32)
        b = f.view(np.uint32)
        b = ((b + np.uint32(0x7FFF) + ((b >> np.uint32(16)) & np.uint32(1))) >> np.uint32(16)) << np.uint32(16)
        out[small] = b.view(np.float32).astype(np.float64)
    big = np.abs(out) > 3.3895313892515355e38  # bfloat16 max
    out[big] = np.sign(out[big]) * np.inf
    out[np.isnan(x)] = np.nan
    return out


def round_f32(x: np.ndarray) -> np.ndarray:
    return np.asarray(x, dtype=np.float64).astype(np.float32).astype(np.float64)


def round_to(x: np.ndarray, storage: str | None) -> np.ndarray:
    if storage is None:
        return x
    if storage == "f32":
        return round_f32(x)
    if storage == "bf16":
        return round_bf16(x)
    raise ValueError(storage)


# ----------------------------------------------------------------- index side

def split_hubs(indptr, threshold: int):
    """Shadow rows of every vertex: (shadow_indptr int64[R+1], shadow_owner int32[R],
    owner_indptr int64[n+1])."""
    indptr = _i64(indptr)
    n = indptr.shape[0] - 1
    R = lib().ito_split_count(C.c_int64(n), _p(indptr), C.c_int64(threshold))
    sp = np.empty(R + 1, np.int64)
    so = np.empty(R, np.int32)
    op = np.empty(n + 1, np.int64)
    lib().ito_split_hubs(C.c_int64(n), _p(indptr), C.c_int64(threshold), _p(sp), _p(so), _p(op))
    return sp, so, op


def buckets(shadow_indptr, bounds):
    """Stable partition of shadow rows by length class: (bucket_offsets int64[nb+1],
    bucket_rows int32[R])."""
    sp = _i64(shadow_indptr)
    bounds = _i64(bounds)
    R = sp.shape[0] - 1
    off = np.empty(bounds.shape[0] + 1, np.int64)
    rows = np.empty(R, np.int32)
    rc = lib().ito_buckets(C.c_int64(R), _p(sp), C.c_int32(bounds.shape[0]), _p(bounds), _p(off), _p(rows))
    if rc != 0:
        raise ValueError("a row is longer than the last bucket bound")
    return off, rows


# ----------------------------------------------------------------- stages

def aggregate(indptr, indices, w, H, op: str):
    indptr, indices, w, H = _i64(indptr), _i32(indices), _f64(w), _f64(H)
    n, F = indptr.shape[0] - 1, H.shape[1]
    A = np.empty((n, F), np.float64)
    lib().ito_aggregate(C.c_int64(n), _p(indptr), _p(indices), _p(w), _p(H), C.c_int32(F),
                        C.c_int32(OPS[op]), _p(A))
    return A


def partial_gather(shadow_indptr, indices, w, H, op: str):
    sp, indices, w, H = _i64(shadow_indptr), _i32(indices), _f64(w), _f64(H)
    R, F = sp.shape[0] - 1, H.shape[1]
    P = np.empty((R, F), np.float64)
    lib().ito_partial_gather(C.c_int64(R), _p(sp), _p(indices), _p(w), _p(H), C.c_int32(F),
                             C.c_int32(OPS[op]), _p(P))
    return P


def combine(owner_indptr, indptr, P, op: str):
    op_, indptr, P = _i64(owner_indptr), _i64(indptr), _f64(P)
    n, F = indptr.shape[0] - 1, P.shape[1]
    A = np.empty((n, F), np.float64)
    lib().ito_combine(C.c_int64(n), _p(op_), _p(indptr), _p(P), C.c_int32(F), C.c_int32(OPS[op]), _p(A))
    return A


def aggregate_edges(segptr, EF, op: str):
    """Reduce of the edge-feature rows of every segment (in-edges of a vertex, or one shadow row)."""
    segptr, EF = _i64(segptr), _f64(EF)
    n, De = segptr.shape[0] - 1, EF.shape[1]
    AE = np.empty((n, De), np.float64)
    lib().ito_aggregate_edges(C.c_int64(n), _p(segptr), _p(EF), C.c_int32(De), C.c_int32(OPS[op]), _p(AE))
    return AE


def edge_messages(indices, w, H, EF, We, be, act: str):
    """m_j = w_j act(h_{u_j} We[:Fi] + e_j We[Fi:] + be) for every CSR entry j: [n_edges, Fm]."""
    indices, w, H, EF, We, be = _i32(indices), _f64(w), _f64(H), _f64(EF), _f64(We), _f64(be)
    Fi, De = H.shape[1], (0 if EF is None else EF.shape[1])
    assert We.shape[0] == Fi + De
    M = np.empty((indices.shape[0], We.shape[1]), np.float64)
    lib().ito_edge_messages(C.c_int64(indices.shape[0]), _p(indices), _p(w), _p(H), C.c_int32(Fi), _p(EF), C.c_int32(De),
                            _p(We), _p(be), C.c_int32(We.shape[1]), C.c_int32(ACTS[act]), _p(M))
    return M


def linear(X, W):
    X, W = _f64(X), _f64(W)
    out = np.empty((X.shape[0], W.shape[1]), np.float64)
    lib().ito_linear(C.c_int64(X.shape[0]), _p(X), C.c_int32(X.shape[1]), _p(W), C.c_int32(W.shape[1]), _p(out))
    return out


def sage_apply(H, A, W, bias, act: str):
    H, A, W, bias = _f64(H), _f64(A), _f64(W), _f64(bias)
    n, Fi, Fo = H.shape[0], H.shape[1], W.shape[1]
    assert W.shape[0] == 2 * Fi and A.shape == H.shape
    out = np.empty((n, Fo), np.float64)
    lib().ito_sage_apply(C.c_int64(n), _p(H), _p(A), C.c_int32(Fi), _p(W), _p(bias), C.c_int32(Fo),
                         C.c_int32(ACTS[act]), _p(out))
    return out


def bias_act(X, bias, act: str):
    X, bias = _f64(X), _f64(bias)
    out = np.empty_like(X)
    lib().ito_bias_act(C.c_int64(X.shape[0]), C.c_int32(X.shape[1]), _p(X), _p(bias), C.c_int32(ACTS[act]), _p(out))
    return out


def gat_scores(Z, att, heads: int):
    Z, att = _f64(Z), _f64(att)
    n, F = Z.shape
    s = np.empty((n, heads), np.float64)
    lib().ito_gat_scores(C.c_int64(n), _p(Z), C.c_int32(heads), C.c_int32(F // heads), _p(att), _p(s))
    return s


def gat_aggregate(indptr, indices, Z, s_src, s_dst, heads: int, slope: float, edge_logit=None):
    indptr, indices, Z, s_src, s_dst = _i64(indptr), _i32(indices), _f64(Z), _f64(s_src), _f64(s_dst)
    edge_logit = _f64(edge_logit)
    n, F = indptr.shape[0] - 1, Z.shape[1]
    assert edge_logit is None or edge_logit.shape == (indices.shape[0], heads)
    O = np.empty((n, F), np.float64)
    lib().ito_gat_aggregate(C.c_int64(n), _p(indptr), _p(indices), _p(Z), _p(s_src), _p(s_dst),
                            C.c_int32(heads), C.c_int32(F // heads), C.c_double(slope), _p(edge_logit), _p(O))
    return O


# ----------------------------------------------------------------- layers

def _sub_csr(indptr, indices, w, rows, ef=None):
    """CSR restricted to the destination vertices `rows` (source ids stay global).  With `ef` (edge features,
    one row per CSR entry) the matching rows are returned as a fourth value."""
    indptr = _i64(indptr)
    rows = _i64(rows)
    deg = indptr[rows + 1] - indptr[rows]
    sub = np.zeros(rows.shape[0] + 1, np.int64)
    np.cumsum(deg, out=sub[1:])
    pos = np.repeat(indptr[rows] - sub[:-1], deg) + np.arange(sub[-1], dtype=np.int64)
    out = (sub, _i32(indices)[pos], (None if w is None else np.asarray(w)[pos]))
    return out if ef is None else out + (np.asarray(ef)[pos],)


def _gathered(indptr, indices, w, H, op, threshold):
    """aggregate, optionally through shadow rows + partial gather + combine (the result is
    the same by associativity; Section "Optimization Strategies", Partial-Gather)."""
    if threshold and threshold > 0:
        sp, _, owner = split_hubs(indptr, threshold)
        return combine(owner, indptr, partial_gather(sp, indices, w, H, op), op)
    return aggregate(indptr, indices, w, H, op)


def _gathered_edges(indptr, EF, op, threshold):
    """The edge-feature part of the aggregate, optionally through shadow rows + combine."""
    if threshold and threshold > 0:
        sp, _, owner = split_hubs(indptr, threshold)
        return combine(owner, indptr, aggregate_edges(sp, EF, "sum" if op == "mean" else op), op)
    return aggregate_edges(indptr, EF, op)


def _edge_dim(layer) -> int:
    return int(getattr(layer, "edge_dim", 0) or 0)


def _msg_dim(layer) -> int:
    return int(getattr(layer, "msg_dim", 0) or 0)


def _message_aggregate(indptr, indices, w, H, ef, layer, storage, threshold):
    """Aggregate of the learned messages m_j = w_j act_e(h_u W_e[:in] + e_j W_e[in:] + b_e) of a layer with
    msg_dim > 0, over the in-edges of every vertex of `indptr`: [n, msg_dim].
    storage=None: the definition, edge by edge (ito_edge_messages).  With a storage type the same value is built the
    way the layer contract stores it: the per-source part P = H W_e[:in] and the per-edge part Q = e W_e[in:] + b_e
    are rounded where they are stored, and so is the finished message act_e(P[u] + Q[j]); without edge features the
    rounded table act_e(P + b_e) is the message itself.  The edge weight multiplies inside the reduce."""
    We, be = _f64(layer.W_edge), _f64(getattr(layer, "bias_edge", None))
    act_e = getattr(layer, "act_edge", "none")
    Fi = layer.in_dim
    op = "sum" if layer.op == "gcn" else layer.op
    if storage is None:
        M = edge_messages(indices, w, H, ef, We, be, act_e)
    else:
        need = np.unique(_i32(indices).astype(np.int64))
        P = np.full((H.shape[0], We.shape[1]), np.nan)
        if ef is None:
            P[need] = round_to(bias_act(linear(H[need], We[:Fi]), be, act_e), storage)
            M = P[_i32(indices).astype(np.int64)]
        else:
            P[need] = round_to(linear(H[need], We[:Fi]), storage)
            Q = round_to(bias_act(linear(ef, We[Fi:]), be, "none"), storage)
            M = round_to(bias_act(P[_i32(indices).astype(np.int64)] + Q, None, act_e), storage)
        if w is not None:
            M = M * _f64(w)[:, None]
    return _gathered_edges(indptr, M, op, threshold)


def _sources_of(indptr, indices, rows):
    """Sorted unique vertex ids that `rows` read: themselves and their in-neighbours."""
    sub, idx, _ = _sub_csr(indptr, indices, None, rows)
    return np.union1d(_i64(rows), idx.astype(np.int64))


def sage_layer(indptr, indices, edge_weights, H, layer, storage=None, threshold=0, reorder=False, rows=None,
               edge_feat=None):
    """One GraphSAGE layer.  `layer` has op, act, in_dim, out_dim, W [2*in, out], bias,
    use_edge_weights.  reorder=True evaluates the algebraically equal transform-before-
    aggregate form (sum and mean only): gather Z = H W_neigh instead of H.
    rows=None: every vertex.  rows=array: only those destination vertices (H is still indexed
    by global vertex id; rows of H that they do not read are never touched); returns
    [len(rows), out].
    layer.edge_dim > 0: the message is [w_e h_u | e_vu] (Eq. (1): M reads the edge features too), reduced
    entry by entry, and W has in_dim + edge_dim neighbour rows: [2*in + edge_dim, out].  Not reordered."""
    H = _f64(H)
    W = _f64(layer.W)
    Fi = layer.in_dim
    De = _edge_dim(layer)
    w = edge_weights if layer.use_edge_weights else None
    ef = _f64(edge_feat) if De else None
    if rows is None:
        Hself = H
    elif De:
        indptr, indices, w, ef = _sub_csr(indptr, indices, w, rows, ef)
        Hself = H[_i64(rows)]
    else:
        indptr, indices, w = _sub_csr(indptr, indices, w, rows)
        Hself = H[_i64(rows)]
    if _msg_dim(layer):   # learned per-edge messages: W is [in + msg_dim, out]
        if reorder:
            raise ValueError("layers with learned messages keep the plain order")
        assert W.shape[0] == Fi + _msg_dim(layer)
        A = round_to(_message_aggregate(indptr, indices, w, H, ef, layer, storage, threshold), storage)
        out = bias_act(linear(Hself, W[:Fi]) + linear(A, W[Fi:]), layer.bias, layer.act)
        return round_to(out, storage)
    if De:
        if reorder:
            raise ValueError("layers with edge features keep the plain order")
        assert ef.shape[1] == De and W.shape[0] == 2 * Fi + De
        A = np.concatenate([_gathered(indptr, indices, w, H, layer.op, threshold),
                            _gathered_edges(indptr, ef, layer.op, threshold)], axis=1)
        A = round_to(A, storage)
        out = bias_act(linear(Hself, W[:Fi]) + linear(A, W[Fi:]), layer.bias, layer.act)
        return round_to(out, storage)
    if reorder:
        if layer.op in ("max", "min"):
            raise ValueError("transform-before-aggregate is not valid for max or min")
        if rows is None:
            Z = round_to(linear(H, W[Fi:]), storage)
        else:   # transform only the rows that are read
            need = np.unique(indices.astype(np.int64))
            Z = np.full((H.shape[0], layer.out_dim), np.nan)
            Z[need] = round_to(linear(H[need], W[Fi:]), storage)
        S = linear(Hself, W[:Fi])
        if layer.bias is not None:
            S = S + _f64(layer.bias)[None, :]
        S = round_to(S, storage)   # the contract stores the self term like every other vertex table
        out = bias_act(S + _gathered(indptr, indices, w, Z, layer.op, threshold), None, layer.act)
    else:
        A = round_to(_gathered(indptr, indices, w, H, layer.op, threshold), storage)
        out = sage_apply(Hself, A, W, layer.bias, layer.act)
    return round_to(out, storage)


def gat_layer(indptr, indices, H, layer, storage=None, rows=None, edge_feat=None):
    """One GAT layer: z = h W; additive attention per head with LeakyReLU; softmax over the
    in-edges of each destination; heads concatenated; bias; activation.  `rows` as in
    sage_layer.  layer.edge_dim > 0: the edge's features enter its attention logit through
    att_edge [heads, edge_dim], e = LeakyReLU(a_src . z_u + a_dst . z_v + a_edge . e_vu)."""
    H = _f64(H)
    De = _edge_dim(layer)
    ef = _f64(edge_feat) if De else None
    if rows is None:
        z = linear(H, _f64(layer.W))
        s_src = gat_scores(z, layer.att_src, layer.heads)
        s_dst = gat_scores(z, layer.att_dst, layer.heads)
    else:
        need = _sources_of(indptr, indices, rows)
        if De:
            indptr, indices, _, ef = _sub_csr(indptr, indices, None, rows, ef)
        else:
            indptr, indices, _ = _sub_csr(indptr, indices, None, rows)
        z = np.full((H.shape[0], layer.out_dim), np.nan)
        z[need] = linear(H[need], _f64(layer.W))
        s_src = np.full((H.shape[0], layer.heads), np.nan)
        s_src[need] = gat_scores(z[need], layer.att_src, layer.heads)
        s_dst = gat_scores(z[_i64(rows)], layer.att_dst, layer.heads)
    c = linear(ef, _f64(layer.att_edge).T) if De else None   # [n_edges, heads]
    if storage is not None:
        s_src, s_dst = round_f32(s_src), round_f32(s_dst)
        if De:   # the contract stores ONE fp32 logit term per edge and head: source score + the edge's share
            c = round_f32(s_src[_i32(indices).astype(np.int64)] + round_f32(c))
            s_src = np.zeros_like(s_src)
    O = gat_aggregate(indptr, indices, round_to(z, storage), s_src, s_dst, layer.heads, layer.leaky_slope, edge_logit=c)
    return round_to(bias_act(O, layer.bias, layer.act), storage)


def dense_layer(H, layer, storage=None, rows=None):
    """A layer without a Gather stage: h' = act(h W + b), W [in, out].  This is the initialisation step of
    the first superstep (raw vertex states -> initial embeddings) and the prediction part attached after
    the last apply_node (Section "Implementation on Pregel")."""
    H = _f64(H)
    if rows is not None:
        H = H[_i64(rows)]
    return round_to(bias_act(linear(H, _f64(layer.W)), layer.bias, layer.act), storage)


def gcn_layer(indptr, indices, edge_weights, H, layer, storage=None, threshold=0, reorder=False, rows=None,
              edge_feat=None):
    """GCN in the message-passing form of Eq. (1): the message is the source state (times the edge weight,
    which carries the degree normalisation; self loops are edges of the graph), the reduce is a sum, and
    the update is dense on the aggregate alone: h'_v = act((sum_e w_e h_u) W + b), W [in, out].
    reorder=True evaluates the algebraically equal form that gathers Z = H W."""
    H = _f64(H)
    W = _f64(layer.W)
    w = edge_weights if layer.use_edge_weights else None
    De = _edge_dim(layer)
    if _msg_dim(layer):   # learned per-edge messages, summed; W is [msg_dim, out]
        if reorder:
            raise ValueError("layers with learned messages keep the plain order")
        ef = _f64(edge_feat) if De else None
        if rows is not None:
            if De:
                indptr, indices, w, ef = _sub_csr(indptr, indices, w, rows, ef)
            else:
                indptr, indices, w = _sub_csr(indptr, indices, w, rows)
        A = round_to(_message_aggregate(indptr, indices, w, H, ef, layer, storage, threshold), storage)
        return round_to(bias_act(linear(A, W), layer.bias, layer.act), storage)
    if De:   # message [w_e h_u | e_vu], summed; W is [in + edge_dim, out]
        if reorder:
            raise ValueError("layers with edge features keep the plain order")
        ef = _f64(edge_feat)
        if rows is not None:
            indptr, indices, w, ef = _sub_csr(indptr, indices, w, rows, ef)
        A = np.concatenate([_gathered(indptr, indices, w, H, "sum", threshold),
                            _gathered_edges(indptr, ef, "sum", threshold)], axis=1)
        return round_to(bias_act(linear(round_to(A, storage), W), layer.bias, layer.act), storage)
    if rows is not None:
        indptr, indices, w = _sub_csr(indptr, indices, w, rows)
    if reorder:
        if rows is None:
            Z = round_to(linear(H, W), storage)
        else:   # transform only the rows that are read
            need = np.unique(indices.astype(np.int64))
            Z = np.full((H.shape[0], layer.out_dim), np.nan)
            Z[need] = round_to(linear(H[need], W), storage)
        out = bias_act(_gathered(indptr, indices, w, Z, "sum", threshold), layer.bias, layer.act)
    else:
        A = round_to(_gathered(indptr, indices, w, H, "sum", threshold), storage)
        out = bias_act(linear(A, W), layer.bias, layer.act)
    return round_to(out, storage)


def layer_forward(indptr, indices, edge_weights, H, layer, storage=None, threshold=0, reorder=False, rows=None,
                  edge_feat=None):
    if layer.op == "gat":
        return gat_layer(indptr, indices, H, layer, storage, rows, edge_feat)
    if layer.op == "dense":
        return dense_layer(H, layer, storage, rows)
    if layer.op == "gcn":
        return gcn_layer(indptr, indices, edge_weights, H, layer, storage, threshold, reorder, rows, edge_feat)
    return sage_layer(indptr, indices, edge_weights, H, layer, storage, threshold, reorder, rows, edge_feat)


def layer_magnitude(indptr, indices, edge_weights, H, layer, rows=None, edge_feat=None):
    """The sum of the ABSOLUTE values of the terms that make up every output entry of `layer` (before its
    activation): the layer evaluated on |H|, |W|, |b|, |w_e| (|e_vu|), with a max / min pooling taken as the
    largest |w_e h_u|, and for GAT the true attention weights applied to |h| |W|.  This is the quantity D of a
    forward error bound |computed - exact| <= c u D for any order of evaluation (the terms of the reordered and
    of the split forms are the same terms), and D >= |exact|: it serves as the denominator floor when a device
    result is compared with the oracle.  Plain order, fp64, no storage rounding."""
    H = _f64(H)
    absw = None if edge_weights is None else np.abs(_f64(edge_weights))
    abse = None if edge_feat is None else np.abs(_f64(edge_feat))
    if layer.op == "gat":
        # attention weights from the true scores; messages replaced by |h| |W|
        if rows is None:
            need, sub_ip, sub_ix = None, indptr, indices
        else:
            need = _sources_of(indptr, indices, rows)
            sub_ip, sub_ix, _ = _sub_csr(indptr, indices, None, rows)
        sel = slice(None) if need is None else need
        z = linear(H[sel], _f64(layer.W))
        zabs = np.full((H.shape[0], layer.out_dim), np.nan)
        zabs[sel] = linear(np.abs(H[sel]), np.abs(_f64(layer.W)))
        s_src = np.full((H.shape[0], layer.heads), np.nan)
        s_src[sel] = gat_scores(z, layer.att_src, layer.heads)
        if rows is None:
            s_dst = gat_scores(z, layer.att_dst, layer.heads)
        else:
            s_dst = gat_scores(linear(H[_i64(rows)], _f64(layer.W)), layer.att_dst, layer.heads)
        c = None
        if _edge_dim(layer):
            ef = _f64(edge_feat)
            if rows is not None:
                ef = _sub_csr(indptr, indices, None, rows, ef)[3]
            c = linear(ef, _f64(layer.att_edge).T)
        D = gat_aggregate(sub_ip, sub_ix, zabs, s_src, s_dst, layer.heads, layer.leaky_slope, edge_logit=c)
        return D if layer.bias is None else D + np.abs(_f64(layer.bias))[None, :]

    class _Abs:   # the same layer on absolute values, no activation
        pass
    a = _Abs()
    a.op = "max" if layer.op in ("max", "min") else layer.op
    a.act = "none"
    a.in_dim, a.out_dim = layer.in_dim, layer.out_dim
    a.W = np.abs(_f64(layer.W))
    a.bias = None if layer.bias is None else np.abs(_f64(layer.bias))
    a.use_edge_weights = layer.use_edge_weights
    a.allow_reorder = False
    a.edge_dim = _edge_dim(layer)
    a.heads = 1
    a.msg_dim = _msg_dim(layer)
    if a.msg_dim:   # |act_e(x)| <= |x| for the activations offered, so the message is bounded by its terms' sum
        a.W_edge = np.abs(_f64(layer.W_edge))
        be = getattr(layer, "bias_edge", None)
        a.bias_edge = None if be is None else np.abs(_f64(be))
        a.act_edge = "none"
    return layer_forward(indptr, indices, absw, np.abs(H), a, storage=None, threshold=0, reorder=False, rows=rows,
                         edge_feat=abse)


def will_reorder(layer) -> bool:
    """The layer contract: transform first when it shrinks the rows that are gathered and
    the aggregate is linear."""
    return (bool(layer.allow_reorder) and layer.op in ("sum", "mean", "gcn") and layer.out_dim < layer.in_dim
            and _edge_dim(layer) == 0 and _msg_dim(layer) == 0)


def infer(indptr, indices, edge_weights, X, layers, storage=None, threshold=0, follow_reorder=False, edge_feat=None,
          magnitudes=False):
    """L layers in order over the whole graph; returns the list of every layer's output.  With magnitudes=True
    also the list of every layer's term magnitudes (layer_magnitude of the input that layer was given)."""
    H = _f64(X)
    outs, mags = [], []
    for layer in layers:
        if magnitudes:
            mags.append(layer_magnitude(indptr, indices, edge_weights, H, layer, edge_feat=edge_feat))
        H = layer_forward(indptr, indices, edge_weights, H, layer, storage, threshold,
                          reorder=follow_reorder and will_reorder(layer), edge_feat=edge_feat)
        outs.append(H)
    return (outs, mags) if magnitudes else outs


def infer_at(indptr, indices, edge_weights, X, layers, targets, storage=None, threshold=0, follow_reorder=False,
             edge_feat=None, magnitudes=False):
    """The L-layer result at the vertices `targets` only, computed from their L-hop
    in-neighbourhood (which is sufficient and necessary for an L-layer model, Section
    "K-hop Neighborhood and Sampling"): layer l is evaluated only where layer l+1 reads it.
    Everything else stays NaN, so a read outside the neighbourhood would poison the result.
    Returns [len(targets), out_dim] in the order of `targets`; with magnitudes=True also the term magnitudes of
    the last layer at the targets (layer_magnitude)."""
    targets = _i64(targets)
    need = [None] * (len(layers) + 1)
    need[len(layers)] = np.unique(targets)
    for l in range(len(layers) - 1, 0, -1):
        need[l] = _sources_of(indptr, indices, need[l + 1])
    H = _f64(X)
    n = H.shape[0]
    D = None
    for l, layer in enumerate(layers, start=1):
        if magnitudes and l == len(layers):
            D = np.full((n, layer.out_dim), np.nan)
            D[need[l]] = layer_magnitude(indptr, indices, edge_weights, H, layer, rows=need[l], edge_feat=edge_feat)
        out_rows = layer_forward(indptr, indices, edge_weights, H, layer, storage, threshold,
                                 reorder=follow_reorder and will_reorder(layer), rows=need[l], edge_feat=edge_feat)
        H = np.full((n, layer.out_dim), np.nan)
        H[need[l]] = out_rows
    return (H[targets], D[targets]) if magnitudes else H[targets]


def compact_neighbourhood(indptr, indices, edge_weights, targets, n_layers, edge_feat=None):
    """The part of the graph an n_layers-layer model reads to produce `targets`, relabelled to
    consecutive ids so that huge graphs can be checked without full-size fp64 arrays.
    Returns (vertex_ids, c_indptr, c_indices, c_weights, c_targets): vertex_ids are the global
    ids (sorted) of the compact vertices; a compact vertex keeps its in-edges only if some layer
    output of it is needed (the others are read as layer-0 inputs only).  With `edge_feat` the rows of
    the kept edges are appended as a sixth value."""
    targets = _i64(targets)
    need = np.unique(targets)
    for _ in range(n_layers - 1):
        need = _sources_of(indptr, indices, need)          # where layer 1 .. L-1 outputs are needed
    ids = _sources_of(indptr, indices, need)               # plus the layer-0 inputs they read
    if edge_feat is None:
        sub, idx, w = _sub_csr(indptr, indices, edge_weights, need)
        ef = None
    else:
        sub, idx, w, ef = _sub_csr(indptr, indices, edge_weights, need, edge_feat)
    deg = np.zeros(ids.shape[0], np.int64)
    pos_need = np.searchsorted(ids, need)
    deg[pos_need] = np.diff(sub)
    c_indptr = np.zeros(ids.shape[0] + 1, np.int64)
    np.cumsum(deg, out=c_indptr[1:])
    # rows of `need` are ascending in both numberings, so the concatenated edge lists keep their order
    c_indices = np.searchsorted(ids, idx.astype(np.int64)).astype(np.int32)
    out = (ids, c_indptr, c_indices, w, np.searchsorted(ids, targets))
    return out if edge_feat is None else out + (ef,)
