"""Pins for the CPU oracle: every check here compares the oracle with something that is
not the oracle — hand-worked values, closed forms, invariants, textbook special cases,
and a brute-force per-vertex computation tree written in pure Python."""
import json
import math
import os
from types import SimpleNamespace as NS

import numpy as np
import pytest

from oracle import oracle as O

GOLD = json.load(open(os.path.join(os.path.dirname(__file__), "golden", "w5.json")))


def L(op="sum", act="none", W=None, bias=None, heads=1, att_src=None, att_dst=None, slope=0.2,
      use_edge_weights=False, allow_reorder=True, edge_dim=0, W_edge=None, bias_edge=None, act_edge="none", att_edge=None):
    W = np.asarray(W, dtype=np.float64)
    in_dim = W.shape[0] if op == "gat" else ((W.shape[0] - edge_dim) if op in ("dense", "gcn") else (W.shape[0] - edge_dim) // 2)
    if W_edge is not None:   # learned messages: W_edge is [in + edge_dim, msg_dim], W is [in + msg_dim, out] (GCN: [msg_dim, out])
        W_edge = np.asarray(W_edge, dtype=np.float64)
        in_dim = W_edge.shape[0] - edge_dim
        return NS(op=op, act=act, in_dim=in_dim, out_dim=W.shape[1], W=W, edge_dim=edge_dim, msg_dim=W_edge.shape[1],
                  W_edge=W_edge, bias_edge=None if bias_edge is None else np.asarray(bias_edge, dtype=np.float64),
                  act_edge=act_edge, bias=None if bias is None else np.asarray(bias, dtype=np.float64), heads=1,
                  att_src=None, att_dst=None, leaky_slope=slope, use_edge_weights=use_edge_weights, allow_reorder=allow_reorder)
    return NS(op=op, act=act, in_dim=in_dim, out_dim=W.shape[1], W=W, edge_dim=edge_dim,
              bias=None if bias is None else np.asarray(bias, dtype=np.float64), heads=heads,
              att_src=None if att_src is None else np.asarray(att_src, dtype=np.float64),
              att_dst=None if att_dst is None else np.asarray(att_dst, dtype=np.float64),
              leaky_slope=slope, use_edge_weights=use_edge_weights, allow_reorder=allow_reorder,
              att_edge=None if att_edge is None else np.asarray(att_edge, dtype=np.float64))


def random_graph(rng, n, max_deg, p_zero=0.2):
    deg = rng.integers(0, max_deg + 1, size=n)
    deg[rng.random(n) < p_zero] = 0
    indptr = np.zeros(n + 1, np.int64)
    np.cumsum(deg, out=indptr[1:])
    indices = rng.integers(0, n, size=int(indptr[-1])).astype(np.int32)  # multi-edges and self-edges allowed
    return indptr, indices


# ------------------------------------------------------------------ hand-worked example

class TestW5:
    ip = np.array(GOLD["indptr"], np.int64)
    ix = np.array(GOLD["indices"], np.int32)
    x = np.array(GOLD["x"], np.float64)
    w = np.array(GOLD["w"], np.float64)

    @pytest.mark.parametrize("op", ["sum", "mean", "max"])
    def test_aggregates(self, op):
        assert np.array_equal(O.aggregate(self.ip, self.ix, None, self.x, op), np.array(GOLD[op], np.float64))

    def test_weighted_sum(self):
        assert np.array_equal(O.aggregate(self.ip, self.ix, self.w, self.x, "sum"), np.array(GOLD["weighted_sum"], np.float64))

    def test_split(self):
        sp, so, op = O.split_hubs(self.ip, GOLD["split_T"])
        assert sp.tolist() == GOLD["shadow_indptr"]
        assert so.tolist() == GOLD["shadow_owner"]
        assert op.tolist() == GOLD["owner_indptr"]
        ps = O.partial_gather(sp, self.ix, None, self.x, "sum")
        pm = O.partial_gather(sp, self.ix, None, self.x, "max")
        assert ps[:2].tolist() == GOLD["partial_sum_v0"]
        assert pm[:2].tolist() == GOLD["partial_max_v0"]
        for o in ("sum", "mean", "max"):
            P = O.partial_gather(sp, self.ix, None, self.x, o)
            assert np.array_equal(O.combine(op, self.ip, P, o), np.array(GOLD[o], np.float64))

    def test_two_layer_sage_mean(self):
        g1, g2 = GOLD["sage_mean_l1"], GOLD["sage_mean_l2"]
        l1 = L("mean", g1["act"], g1["W"], g1["b"])
        l2 = L("mean", g2["act"], g2["W"], g2["b"])
        for thr in (0, 2):
            for fr in (False, True):
                outs = O.infer(self.ip, self.ix, None, self.x, [l1, l2], threshold=thr, follow_reorder=fr)
                assert np.array_equal(outs[0], np.array(g1["out"], np.float64))
                assert np.array_equal(outs[1], np.array(g2["out"], np.float64))
        H1 = np.array(g1["out"], np.float64)
        Z = O.linear(H1, np.array(g2["W"], np.float64)[2:])
        assert Z.tolist() == g2["Z"]
        assert O.aggregate(self.ip, self.ix, None, Z, "mean").tolist() == g2["mean_Z"]

    def test_gat(self):
        g = GOLD["gat"]
        layer = L("gat", "none", g["W"], None, 1, g["att_src"], g["att_dst"], g["slope"])
        out = O.gat_layer(self.ip, self.ix, self.x, layer)
        assert np.abs(out - np.array(g["out"])).max() < g["out_tol"]
        # the printed alphas reproduce the printed outputs (fixture self-consistency, by hand rule)
        for v, al in g["alpha"].items():
            v = int(v)
            src = self.ix[self.ip[v]:self.ip[v + 1]]
            assert abs(sum(al) - 1) < 1e-6
            assert np.abs((np.array(al)[:, None] * self.x[src]).sum(0) - np.array(g["out"][v])).max() < 2e-6


# ------------------------------------------------------------------ brute-force computation tree

def py_act(x, act):
    if act == "relu":
        return x if x > 0 else 0.0
    if act == "elu":
        return x if x > 0 else math.exp(x) - 1.0
    return x


def tree_eval(v, depth, ip, ix, w, x, layers, memo=None, ef=None):
    """h_v^depth by direct recursion over the in-neighbourhood (Eq. (1)); pure Python floats.
    No memo: every path of the computation tree is evaluated, as a k-hop pipeline would."""
    if depth == 0:
        return [float(t) for t in x[v]]
    lay = layers[depth - 1]
    hv = tree_eval(v, depth - 1, ip, ix, w, x, layers, ef=ef)
    nb = [(int(ix[j]), (float(w[j]) if (w is not None and lay.use_edge_weights) else 1.0)) for j in range(ip[v], ip[v + 1])]
    hn = [tree_eval(u, depth - 1, ip, ix, w, x, layers, ef=ef) for u, _ in nb]
    Fi, Fo = lay.in_dim, lay.out_dim
    W = lay.W
    if lay.op == "gat":
        D = Fo // lay.heads
        zl = lambda h: [sum(h[k] * W[k][c] for k in range(Fi)) for c in range(Fo)]
        zv, zn = zl(hv), [zl(h) for h in hn]
        out = [0.0] * Fo
        for hd in range(lay.heads):
            sd = sum(lay.att_dst[hd][c] * zv[hd * D + c] for c in range(D))
            es = []
            for jj, z in zip(range(ip[v], ip[v + 1]), zn):
                e = sum(lay.att_src[hd][c] * z[hd * D + c] for c in range(D)) + sd
                if getattr(lay, "edge_dim", 0):
                    e += sum(lay.att_edge[hd][f] * float(ef[jj][f]) for f in range(lay.edge_dim))
                es.append(e if e > 0 else lay.leaky_slope * e)
            if es:
                m = max(es)
                ex = [math.exp(e - m) for e in es]
                tot = sum(ex)
                for z, p in zip(zn, ex):
                    for c in range(D):
                        out[hd * D + c] += p / tot * z[hd * D + c]
        return [py_act(out[c] + (lay.bias[c] if lay.bias is not None else 0.0), lay.act) for c in range(Fo)]
    De = getattr(lay, "edge_dim", 0)
    if getattr(lay, "msg_dim", 0):   # learned message: w_e act_e([h_u | e_vu] W_e + b_e)
        Fm = lay.msg_dim
        full = []
        for j, (_, wj), h in zip(range(ip[v], ip[v + 1]), nb, hn):
            cat = list(h) + [float(ef[j][f]) for f in range(De)]
            full.append([wj * py_act(sum(cat[k] * lay.W_edge[k][c] for k in range(Fi + De)) +
                                     (lay.bias_edge[c] if lay.bias_edge is not None else 0.0), lay.act_edge) for c in range(Fm)])
    else:
        Fm = Fi + De   # length of a message: [w_e h_u | e_vu]
        full = [[wj * h[f] for f in range(Fi)] + [float(ef[j][f]) for f in range(De)]
                for j, (_, wj), h in zip(range(ip[v], ip[v + 1]), nb, hn)]
    agg = [0.0] * Fm
    if full:
        for f in range(Fm):
            msgs = [m[f] for m in full]
            agg[f] = max(msgs) if lay.op == "max" else (min(msgs) if lay.op == "min" else sum(msgs))
            if lay.op == "mean":
                agg[f] /= len(msgs)
    out = []
    for c in range(Fo):
        t = lay.bias[c] if lay.bias is not None else 0.0
        if lay.op != "gcn":
            t += sum(hv[k] * W[k][c] for k in range(Fi))
        r0 = 0 if lay.op == "gcn" else Fi
        t += sum(agg[k] * W[r0 + k][c] for k in range(Fm))
        out.append(py_act(t, lay.act))
    return out


@pytest.mark.parametrize("op", ["sum", "mean", "max", "min", "gat"])
@pytest.mark.parametrize("depth", [1, 2, 3])
def test_layerwise_equals_computation_tree(op, depth):
    rng = np.random.default_rng(100 + depth)
    n = 14
    ip, ix = random_graph(rng, n, 3)
    w = rng.random(ix.shape[0])
    dims = [3, 4, 2, 3][:depth + 1]
    x = rng.standard_normal((n, dims[0]))
    layers = []
    for i in range(depth):
        fi, fo = dims[i], dims[i + 1]
        act = ["relu", "elu", "none"][i % 3]
        if op == "gat":
            fo = 4
            dims[i + 1] = 4
            layers.append(L("gat", act, rng.standard_normal((fi, fo)), rng.standard_normal(fo), 2,
                            rng.standard_normal((2, 2)), rng.standard_normal((2, 2)), 0.2))
        else:
            layers.append(L(op, act, rng.standard_normal((2 * fi, fo)), rng.standard_normal(fo),
                            use_edge_weights=(op != "mean")))
    full = O.infer(ip, ix, w, x, layers)[-1]
    split = O.infer(ip, ix, w, x, layers, threshold=2, follow_reorder=True)[-1]
    for v in range(n):
        ref = np.array(tree_eval(v, depth, ip, ix, w, x, layers))
        assert np.allclose(full[v], ref, rtol=1e-11, atol=1e-12), (op, depth, v)
        assert np.allclose(split[v], ref, rtol=1e-11, atol=1e-12), (op, depth, v)


def khop_in_neighbourhood(v, k, ip, ix):
    seen, frontier = {v}, {v}
    for _ in range(k):
        nxt = set()
        for t in frontier:
            nxt.update(int(u) for u in ix[ip[t]:ip[t + 1]])
        frontier = nxt - seen
        seen |= nxt
    return sorted(seen)


@pytest.mark.parametrize("op", ["mean", "max", "gat"])
def test_khop_neighbourhood_is_sufficient(op):
    """A k-layer model on the induced k-hop neighbourhood of v gives the full-graph value at v
    (Section "K-hop Neighborhood and Sampling"; the paper's consistency property)."""
    rng = np.random.default_rng(7)
    n, k = 60, 2
    ip, ix = random_graph(rng, n, 3)
    x = rng.standard_normal((n, 4))
    if op == "gat":
        layers = [L("gat", "elu", rng.standard_normal((4, 4)), rng.standard_normal(4), 2,
                    rng.standard_normal((2, 2)), rng.standard_normal((2, 2))) for _ in range(k)]
    else:
        layers = [L(op, "relu", rng.standard_normal((8, 4)), rng.standard_normal(4)) for _ in range(k)]
    full = O.infer(ip, ix, None, x, layers)[-1]
    for v in range(0, n, 7):
        keep = khop_in_neighbourhood(v, k, ip, ix)
        new_id = {u: i for i, u in enumerate(keep)}
        sub_ip, sub_ix = [0], []
        for u in keep:   # induced subgraph: every edge between kept vertices
            sub_ix += [new_id[int(s)] for s in ix[ip[u]:ip[u + 1]] if int(s) in new_id]
            sub_ip.append(len(sub_ix))
        # vertices at distance < k keep all their in-edges, which is what the value at v needs
        sub = O.infer(np.array(sub_ip, np.int64), np.array(sub_ix, np.int32), None, x[keep], layers)[-1]
        assert np.allclose(sub[new_id[v]], full[v], rtol=1e-12, atol=1e-13)


# ------------------------------------------------------------------ split / combine / buckets

def brute_split(deg, T):
    sp, so, op, pos = [], [], [], 0
    for v, d in enumerate(deg):
        n = 1 if (T <= 0 or d <= T) else -(-d // T)
        op.append(len(so))
        sizes = [d // n + (1 if g < d % n else 0) for g in range(n)]
        for s in sizes:
            sp.append(pos)
            so.append(v)
            pos += s
    op.append(len(so))
    sp.append(pos)
    return sp, so, op


@pytest.mark.parametrize("T", [0, 1, 2, 3, 7, 16, 1000])
def test_split_rule_closed_forms(T):
    rng = np.random.default_rng(T)
    deg = np.concatenate([rng.integers(0, 40, size=200), [0, 1, T, T + 1, 2 * T, 2 * T + 1, 997]]).astype(np.int64)
    deg = np.maximum(deg, 0)
    ip = np.zeros(deg.size + 1, np.int64)
    np.cumsum(deg, out=ip[1:])
    sp, so, op = O.split_hubs(ip, T)
    bs, bo, bp = brute_split(deg.tolist(), T)
    assert sp.tolist() == bs and so.tolist() == bo and op.tolist() == bp
    lens = np.diff(sp)
    for v, d in enumerate(deg):
        g = lens[op[v]:op[v + 1]]
        assert g.sum() == d
        assert g.max() - g.min() <= 1
        if T > 0:
            assert g.max() <= max(T, 0) or d == 0
            assert g.size == (1 if d <= T else math.ceil(d / T))
            if g.size > 1:
                assert (g.size - 1) * T < d   # smallest n that keeps every group <= T
        else:
            assert g.size == 1
        assert sp[op[v]] == ip[v] and sp[op[v + 1]] == ip[v + 1]
        assert np.all(np.diff(g) <= 0)        # the larger groups come first


@pytest.mark.parametrize("op", ["sum", "mean", "max", "min"])
def test_split_invariance(op):
    """Partial gather + combine does not change the result (associativity): bit-exact for
    max and for integer-valued inputs, to rounding for general floats."""
    rng = np.random.default_rng(3)
    ip, ix = random_graph(rng, 300, 90)
    w = rng.random(ix.shape[0])
    H = rng.standard_normal((300, 5))
    Hi = rng.integers(-8, 9, size=(300, 5)).astype(np.float64)
    wi = rng.integers(1, 4, size=ix.shape[0]).astype(np.float64)
    base, base_i = O.aggregate(ip, ix, w, H, op), O.aggregate(ip, ix, wi, Hi, op)
    for T in (1, 2, 5, 17, 64, 89, 90, 1000):
        sp, so, owner = O.split_hubs(ip, T)
        got = O.combine(owner, ip, O.partial_gather(sp, ix, w, H, op), op)
        got_i = O.combine(owner, ip, O.partial_gather(sp, ix, wi, Hi, op), op)
        if op in ("max", "min"):
            assert np.array_equal(got, base)
        else:
            assert np.allclose(got, base, rtol=1e-12, atol=1e-12)
        if op != "mean":
            assert np.array_equal(got_i, base_i)
        else:
            assert np.allclose(got_i, base_i, rtol=1e-15, atol=0)


def test_buckets_brute_force_and_stability():
    rng = np.random.default_rng(5)
    lens = np.concatenate([rng.integers(0, 50, size=500), [0, 0, 8, 9, 32, 33, 256, 257, 300]]).astype(np.int64)
    sp = np.zeros(lens.size + 1, np.int64)
    np.cumsum(lens, out=sp[1:])
    bounds = [0, 8, 32, 256, 300]
    off, rows = O.buckets(sp, bounds)
    assert off[0] == 0 and off[-1] == lens.size
    assert sorted(rows.tolist()) == list(range(lens.size))
    lo = -1
    for b, hi in enumerate(bounds):
        r = rows[off[b]:off[b + 1]]
        assert np.all(np.diff(r) > 0)                       # stable: ascending row id
        assert np.all((lens[r] > lo) & (lens[r] <= hi))
        assert r.tolist() == [i for i in range(lens.size) if lo < lens[i] <= hi]
        lo = hi
    with pytest.raises(ValueError):
        O.buckets(sp, [0, 8, 32])


# ------------------------------------------------------------------ textbook special cases

def dense_adjacency(ip, ix, w, n):
    A = np.zeros((n, n))
    for v in range(n):
        for j in range(ip[v], ip[v + 1]):
            A[v, ix[j]] += 1.0 if w is None else w[j]
    return A


def test_sum_layer_is_sparse_times_dense():
    """W_self = 0, W_neigh = I, no bias, no activation: the layer is (weighted adjacency) x H."""
    rng = np.random.default_rng(11)
    n, F = 50, 6
    ip, ix = random_graph(rng, n, 9)
    w = rng.random(ix.shape[0])
    H = rng.standard_normal((n, F))
    layer = L("sum", "none", np.vstack([np.zeros((F, F)), np.eye(F)]), None, use_edge_weights=True)
    out = O.sage_layer(ip, ix, w, H, layer)
    assert np.allclose(out, dense_adjacency(ip, ix, w, n) @ H, rtol=1e-13, atol=1e-13)
    layer.use_edge_weights = False
    out = O.sage_layer(ip, ix, w, H, layer)
    assert np.allclose(out, dense_adjacency(ip, ix, None, n) @ H, rtol=1e-13, atol=1e-13)


def test_self_and_neighbour_blocks_are_not_swapped():
    """Rows 0..in-1 of W multiply the vertex's own state, rows in..2in-1 the aggregate."""
    rng = np.random.default_rng(12)
    n, F = 30, 3
    ip, ix = random_graph(rng, n, 4)
    H = rng.standard_normal((n, F))
    Ws, Wn, b = rng.standard_normal((F, 2)), rng.standard_normal((F, 2)), rng.standard_normal(2)
    out = O.sage_layer(ip, ix, None, H, L("sum", "none", np.vstack([Ws, Wn]), b))
    assert np.allclose(out, H @ Ws + (dense_adjacency(ip, ix, None, n) @ H) @ Wn + b, rtol=1e-13, atol=1e-13)


def test_dense_layer_is_plain_matmul_bias_activation():
    """The layer without a Gather stage (initial transform, prediction part): numpy's act(H W + b)."""
    rng = np.random.default_rng(31)
    H, W, b = rng.standard_normal((60, 5)), rng.standard_normal((5, 3)), rng.standard_normal(3)
    for act, f in (("none", lambda y: y), ("relu", lambda y: np.maximum(y, 0)), ("elu", lambda y: np.where(y > 0, y, np.expm1(y)))):
        lay = L("dense", act, W, b)
        assert np.allclose(O.dense_layer(H, lay), f(H @ W + b), rtol=1e-13, atol=1e-13)
        rows = np.array([7, 3, 3, 59])
        assert np.array_equal(O.dense_layer(H, lay, rows=rows), O.dense_layer(H, lay)[rows])
        # through the layer dispatcher the graph is ignored
        ip, ix = random_graph(rng, 60, 4)
        assert np.array_equal(O.layer_forward(ip, ix, None, H, lay), O.dense_layer(H, lay))
    # a transposed weight matrix would not even have the right shape; a dropped bias is caught here
    assert not np.allclose(O.dense_layer(H, L("dense", "none", W, None)), H @ W + b)


def test_gcn_layer_is_normalised_adjacency_times_h_times_w():
    """GCN: act(A_hat H W + b) with the normalisation carried by the edge weights and self loops as edges;
    against the dense matrix product, and the textbook facts that a row-stochastic A_hat keeps constant
    features constant and that the symmetric normalisation of an undirected graph gives a symmetric A_hat."""
    rng = np.random.default_rng(32)
    n, Fi, Fo = 40, 5, 3
    ip, ix = random_graph(rng, n, 6)
    w = rng.random(ix.shape[0])
    H, W, b = rng.standard_normal((n, Fi)), rng.standard_normal((Fi, Fo)), rng.standard_normal(Fo)
    lay = L("gcn", "relu", W, b, use_edge_weights=True)
    A = dense_adjacency(ip, ix, w, n)
    want = np.maximum(A @ H @ W + b, 0)
    assert np.allclose(O.gcn_layer(ip, ix, w, H, lay), want, rtol=1e-12, atol=1e-12)
    assert np.allclose(O.gcn_layer(ip, ix, w, H, lay, reorder=True), want, rtol=1e-12, atol=1e-12)
    assert np.allclose(O.gcn_layer(ip, ix, w, H, lay, threshold=2), want, rtol=1e-12, atol=1e-12)
    rows = np.array([5, 0, 39, 17])
    assert np.allclose(O.gcn_layer(ip, ix, w, H, lay, rows=rows), want[rows], rtol=1e-12, atol=1e-12)
    assert np.allclose(O.gcn_layer(ip, ix, w, H, lay, rows=rows, reorder=True), want[rows], rtol=1e-12, atol=1e-12)
    # the vertex's own state enters only through a self-loop edge: no hidden self term
    lone = L("gcn", "none", np.eye(Fi), None, use_edge_weights=False)
    deg = np.diff(ip)
    assert np.all(O.gcn_layer(ip, ix, None, H, lone)[deg == 0] == 0)
    # row-stochastic weights (1 / in-degree): constant features stay constant where there is an in-edge
    wrow = np.repeat(1.0 / np.maximum(deg, 1), deg)
    const = np.full((n, Fi), 1.5)
    out = O.gcn_layer(ip, ix, wrow, const, L("gcn", "none", np.eye(Fi), None, use_edge_weights=True))
    assert np.allclose(out[deg > 0], 1.5, rtol=1e-14) and np.all(out[deg == 0] == 0)
    # symmetric normalisation of an undirected ring with self loops: A_hat = (A + I) / 3, symmetric
    m = 12
    src = np.array([[(v - 1) % m, v, (v + 1) % m] for v in range(m)]).ravel().astype(np.int32)
    rip = np.arange(0, 3 * m + 1, 3, dtype=np.int64)
    wsym = np.full(3 * m, 1.0 / 3.0)     # 1 / sqrt(d_u d_v) with d = 3 everywhere
    X = rng.standard_normal((m, 2))
    out = O.gcn_layer(rip, src, wsym, X, L("gcn", "none", np.eye(2), None, use_edge_weights=True))
    assert np.allclose(out, (np.roll(X, 1, 0) + X + np.roll(X, -1, 0)) / 3.0, rtol=1e-14, atol=1e-14)


def test_linear_and_activations_against_numpy():
    rng = np.random.default_rng(13)
    X, W, b = rng.standard_normal((40, 7)), rng.standard_normal((7, 5)), rng.standard_normal(5)
    assert np.allclose(O.linear(X, W), X @ W, rtol=1e-13, atol=1e-13)
    Y = X[:, :5] * 3
    assert np.array_equal(O.bias_act(Y, b, "relu"), np.maximum(Y + b, 0))
    assert np.allclose(O.bias_act(Y, b, "elu"), np.where(Y + b > 0, Y + b, np.expm1(Y + b)), rtol=1e-15)
    assert np.array_equal(O.bias_act(Y, None, "none"), Y)
    A = rng.standard_normal((40, 7))
    W2 = rng.standard_normal((14, 5))
    assert np.allclose(O.sage_apply(X, A, W2, b, "none"), np.hstack([X, A]) @ W2 + b, rtol=1e-13, atol=1e-13)


def test_mean_of_constant_is_constant_and_max_dominates_mean():
    rng = np.random.default_rng(14)
    n = 200
    ip, ix = random_graph(rng, n, 12)
    deg = np.diff(ip)
    H = np.full((n, 3), 2.5)
    m = O.aggregate(ip, ix, None, H, "mean")
    assert np.array_equal(m[deg > 0], H[deg > 0]) and np.all(m[deg == 0] == 0)
    H = rng.standard_normal((n, 3))
    mx, mn, sm = (O.aggregate(ip, ix, None, H, o) for o in ("max", "mean", "sum"))
    assert np.all(mx[deg > 0] >= mn[deg > 0] - 1e-15)
    assert np.allclose(sm, mn * deg[:, None], rtol=1e-13, atol=1e-13)
    assert np.all(mx[deg == 0] == 0)
    # max of all-negative messages stays negative (no spurious 0 from the initial value)
    mxn = O.aggregate(ip, ix, None, -np.abs(H) - 1, "max")
    assert np.all(mxn[deg > 0] < 0)


def test_min_pooling_against_numpy_and_against_max():
    """min pooling (the reduce of Eq. (1) may be sum, mean, max or min): per destination the plain numpy
    minimum over its gathered messages; equal to -max of the negated messages; an empty neighbourhood gives
    0; all-positive messages stay positive (no spurious 0 from the initial value)."""
    rng = np.random.default_rng(21)
    n = 150
    ip, ix = random_graph(rng, n, 10)
    deg = np.diff(ip)
    H = rng.standard_normal((n, 4))
    w = rng.random(ix.shape[0]) + 0.1
    for ww in (None, w):
        got = O.aggregate(ip, ix, ww, H, "min")
        for v in range(n):
            msgs = H[ix[ip[v]:ip[v + 1]]] * (1.0 if ww is None else ww[ip[v]:ip[v + 1], None])
            want = msgs.min(axis=0) if deg[v] else np.zeros(4)
            assert np.array_equal(got[v], want)
        assert np.array_equal(got, -O.aggregate(ip, ix, ww, -H, "max"))
    pos = O.aggregate(ip, ix, None, np.abs(H) + 1, "min")
    assert np.all(pos[deg > 0] > 0) and np.all(pos[deg == 0] == 0)
    mn, me = O.aggregate(ip, ix, None, H, "min"), O.aggregate(ip, ix, None, H, "mean")
    assert np.all(mn[deg > 0] <= me[deg > 0] + 1e-15)


def test_permutation_invariance_inside_segments():
    rng = np.random.default_rng(15)
    n = 120
    ip, ix = random_graph(rng, n, 10)
    w = rng.random(ix.shape[0])
    H = rng.standard_normal((n, 4))
    ix2, w2 = ix.copy(), w.copy()
    for v in range(n):
        p = rng.permutation(ip[v + 1] - ip[v]) + ip[v]
        ix2[ip[v]:ip[v + 1]], w2[ip[v]:ip[v + 1]] = ix[p], w[p]
    assert np.array_equal(O.aggregate(ip, ix, w, H, "max"), O.aggregate(ip, ix2, w2, H, "max"))
    assert np.allclose(O.aggregate(ip, ix, w, H, "sum"), O.aggregate(ip, ix2, w2, H, "sum"), rtol=1e-12, atol=1e-13)
    gl = L("gat", "none", rng.standard_normal((4, 4)), None, 2, rng.standard_normal((2, 2)), rng.standard_normal((2, 2)))
    assert np.allclose(O.gat_layer(ip, ix, H, gl), O.gat_layer(ip, ix2, H, gl), rtol=1e-12, atol=1e-13)


def test_gat_softmax_special_cases():
    rng = np.random.default_rng(16)
    n, F, heads = 150, 6, 3
    ip, ix = random_graph(rng, n, 8)
    deg = np.diff(ip)
    H = rng.standard_normal((n, F))
    W = rng.standard_normal((F, F))
    zero = np.zeros((heads, F // heads))
    # all-equal scores: attention is uniform, the reduce is a mean of z
    out = O.gat_layer(ip, ix, H, L("gat", "none", W, None, heads, zero, zero))
    assert np.allclose(out, O.aggregate(ip, ix, None, H @ W, "mean"), rtol=1e-12, atol=1e-13)
    # destination score is common to a segment, so it cannot change alpha when e > 0 everywhere
    a_s, a_d = rng.standard_normal((heads, F // heads)), rng.standard_normal((heads, F // heads))
    lay = L("gat", "none", W, None, heads, a_s, a_d, slope=1.0)       # slope 1: LeakyReLU is the identity
    lay0 = L("gat", "none", W, None, heads, a_s, zero, slope=1.0)
    assert np.allclose(O.gat_layer(ip, ix, H, lay), O.gat_layer(ip, ix, H, lay0), rtol=1e-10, atol=1e-12)
    # weights sum to one: constant z comes back unchanged where there is an in-edge, 0 elsewhere
    Hc = np.ones((n, F))
    out = O.gat_layer(ip, ix, Hc, L("gat", "none", np.eye(F), None, heads, a_s, a_d))
    assert np.allclose(out[deg > 0], 1.0, rtol=1e-13) and np.all(out[deg == 0] == 0)
    # single in-edge: alpha = 1
    one = np.flatnonzero(deg == 1)
    full = O.gat_layer(ip, ix, H, L("gat", "none", W, None, heads, a_s, a_d))
    assert one.size > 0 and np.allclose(full[one], (H @ W)[ix[ip[one]]], rtol=1e-13, atol=1e-14)
    # two in-edges: closed-form two-way softmax (a logistic of the score difference)
    two = np.flatnonzero(deg == 2)
    z = H @ W
    D = F // heads
    for v in two[:10]:
        u0, u1 = ix[ip[v]], ix[ip[v] + 1]
        for k in range(heads):
            sl = slice(k * D, (k + 1) * D)
            lrelu = lambda t: t if t > 0 else 0.2 * t
            e0 = lrelu(a_s[k] @ z[u0, sl] + a_d[k] @ z[v, sl])
            e1 = lrelu(a_s[k] @ z[u1, sl] + a_d[k] @ z[v, sl])
            a0 = 1.0 / (1.0 + math.exp(e1 - e0))
            assert np.allclose(full[v, sl], a0 * z[u0, sl] + (1 - a0) * z[u1, sl], rtol=1e-11, atol=1e-13)


def test_gat_softmax_is_shift_safe():
    """Large scores must not overflow: the max is subtracted before exp."""
    ip = np.array([0, 3], np.int64)
    ix = np.array([0, 0, 0], np.int32)
    lay = L("gat", "none", [[1000.0]], None, 1, [[1.0]], [[0.0]])
    out = O.gat_layer(ip, ix, np.array([[1.0]]), lay)
    assert np.isfinite(out).all() and abs(out[0, 0] - 1000.0) < 1e-9


def test_reorder_is_algebraically_equal():
    rng = np.random.default_rng(17)
    n = 100
    ip, ix = random_graph(rng, n, 20)
    w = rng.random(ix.shape[0])
    H = rng.standard_normal((n, 8))
    for op in ("sum", "mean"):
        lay = L(op, "relu", rng.standard_normal((16, 3)), rng.standard_normal(3), use_edge_weights=True)
        a = O.sage_layer(ip, ix, w, H, lay, reorder=False)
        b = O.sage_layer(ip, ix, w, H, lay, reorder=True, threshold=4)
        assert np.allclose(a, b, rtol=1e-11, atol=1e-12)
    with pytest.raises(ValueError):
        O.sage_layer(ip, ix, w, H, L("max", "relu", rng.standard_normal((16, 3))), reorder=True)
    assert O.will_reorder(L("sum", W=np.zeros((16, 3)))) and not O.will_reorder(L("max", W=np.zeros((16, 3))))
    assert O.will_reorder(L("gcn", W=np.zeros((8, 3)))) and not O.will_reorder(L("dense", W=np.zeros((8, 3))))
    assert not O.will_reorder(L("sum", W=np.zeros((16, 8)))) and not O.will_reorder(L("sum", W=np.zeros((16, 3)), allow_reorder=False))


# ------------------------------------------------------------------ rounding helpers

def test_round_bf16_matches_torch_and_ties_to_even():
    torch = pytest.importorskip("torch")
    rng = np.random.default_rng(18)
    x32 = np.concatenate([rng.standard_normal(20000).astype(np.float32) * 10.0 ** rng.integers(-30, 30, 20000).astype(np.float32),
                          np.array([0.0, -0.0, 1.0, 1.00390625, 1.01171875, 3.3e38, -3.3e38, 1e-40, 65504.0], np.float32)])
    ref = torch.from_numpy(x32).to(torch.bfloat16).to(torch.float64).numpy()
    got = O.round_bf16(x32.astype(np.float64))
    assert np.array_equal(got, ref)
    # exact ties in fp64 that fp32 cannot hold a hair away from: 1 + 2^-8 is a tie -> even (1.0);
    # 1 + 2^-8 + 2^-40 is above the tie -> 1 + 2^-7
    assert O.round_bf16(np.array([1 + 2.0 ** -8]))[0] == 1.0
    assert O.round_bf16(np.array([1 + 2.0 ** -8 + 2.0 ** -40]))[0] == 1 + 2.0 ** -7
    assert O.round_bf16(np.array([1 + 3 * 2.0 ** -8]))[0] == 1 + 2.0 ** -6
    assert O.round_f32(np.array([1 + 2.0 ** -30]))[0] == 1.0


def test_storage_mode_stays_close_to_exact_mode():
    rng = np.random.default_rng(19)
    n = 300
    ip, ix = random_graph(rng, n, 30)
    X = rng.standard_normal((n, 8))
    layers = [L("mean", "relu", rng.uniform(-.4, .4, (16, 8)), rng.uniform(-.1, .1, 8)),
              L("mean", "none", rng.uniform(-.4, .4, (16, 4)), rng.uniform(-.1, .1, 4))]
    a = O.infer(ip, ix, None, X, layers)[-1]
    for storage, tol in (("f32", 1e-6), ("bf16", 3e-2)):
        b = O.infer(ip, ix, None, X, layers, storage=storage, threshold=7, follow_reorder=True)[-1]
        assert np.abs(a - b).max() / np.sqrt((a ** 2).mean()) < tol
        assert not np.array_equal(a, b)


@pytest.mark.parametrize("op", ["sum", "mean", "max", "gat"])
def test_infer_at_targets_equals_full_graph_inference(op):
    """Evaluating only the L-hop in-neighbourhood of some targets gives the full-graph values
    there (and reads nothing else: untouched rows are NaN)."""
    rng = np.random.default_rng(21)
    n = 400
    ip, ix = random_graph(rng, n, 6)
    w = rng.random(ix.shape[0])
    X = rng.standard_normal((n, 8))
    if op == "gat":
        layers = [L("gat", "elu", rng.standard_normal((8, 8)) * .3, rng.standard_normal(8) * .1, 2,
                    rng.standard_normal((2, 4)) * .3, rng.standard_normal((2, 4)) * .3) for _ in range(2)]
    else:
        layers = [L(op, "relu", rng.standard_normal((16, 8)) * .3, rng.standard_normal(8) * .1, use_edge_weights=True),
                  L(op, "none", rng.standard_normal((16, 4)) * .3, rng.standard_normal(4) * .1, use_edge_weights=True)]
    targets = rng.permutation(n)[:25]
    for storage in (None, "bf16"):
        for thr in (0, 3):
            if op == "gat" and thr:
                continue
            full = O.infer(ip, ix, w, X, layers, storage=storage, threshold=thr, follow_reorder=True)[-1]
            part = O.infer_at(ip, ix, w, X, layers, targets, storage=storage, threshold=thr, follow_reorder=True)
            assert np.array_equal(part, full[targets])


def test_compact_neighbourhood_gives_the_same_values():
    rng = np.random.default_rng(23)
    n = 500
    ip, ix = random_graph(rng, n, 5)
    w = rng.random(ix.shape[0])
    X = rng.standard_normal((n, 6))
    layers = [L("sum", "relu", rng.standard_normal((12, 6)) * .3, rng.standard_normal(6) * .1, use_edge_weights=True),
              L("mean", "none", rng.standard_normal((12, 4)) * .3, rng.standard_normal(4) * .1)]
    targets = rng.permutation(n)[:20]
    full = O.infer(ip, ix, w, X, layers, threshold=3)[-1]
    ids, cip, cix, cw, ct = O.compact_neighbourhood(ip, ix, w, targets, len(layers))
    assert ids.shape[0] < n and np.all(np.diff(ids) > 0)
    part = O.infer_at(cip, cix, cw, X[ids], layers, ct, threshold=3)
    assert np.array_equal(part, full[targets])


# ------------------------------------------------------------------ edge features in the message (Eq. (1): e_{v,u})

class TestW5EdgeFeatures:
    g = GOLD["edge_features"]
    ip, ix, x = TestW5.ip, TestW5.ix, TestW5.x
    ef = np.array(GOLD["edge_features"]["ef"], np.float64)

    @pytest.mark.parametrize("op", ["sum", "mean", "max", "min"])
    def test_edge_aggregates(self, op):
        assert O.aggregate_edges(self.ip, self.ef, op).tolist() == self.g[op]

    def test_partials_and_combine(self):
        sp, _, owner = O.split_hubs(self.ip, GOLD["split_T"])
        assert O.aggregate_edges(sp, self.ef, "sum")[:2].tolist() == self.g["partial_sum_v0"]
        assert O.aggregate_edges(sp, self.ef, "max")[:2].tolist() == self.g["partial_max_v0"]
        for op in ("sum", "mean", "max", "min"):
            P = O.aggregate_edges(sp, self.ef, "sum" if op == "mean" else op)
            assert O.combine(owner, self.ip, P, op).tolist() == self.g[op]

    @pytest.mark.parametrize("op,key", [("sum", "sage_sum_out"), ("max", "sage_max_out")])
    def test_sage_layer_with_edge_features(self, op, key):
        layer = L(op, self.g["act"], self.g["W"], self.g["b"], edge_dim=1)
        for thr in (0, 2):
            out = O.sage_layer(self.ip, self.ix, None, self.x, layer, threshold=thr, edge_feat=self.ef)
            assert out.tolist() == self.g[key]


def test_edge_aggregate_is_a_segmented_reduce():
    """Against numpy's own segmented reductions over the non-empty segments."""
    rng = np.random.default_rng(31)
    ip, ix = random_graph(rng, 60, 9)
    ef = rng.standard_normal((ix.shape[0], 3))
    deg = np.diff(ip)
    nz = np.flatnonzero(deg > 0)
    starts = ip[nz]
    for op, ufunc in (("sum", np.add), ("max", np.maximum), ("min", np.minimum)):
        got = O.aggregate_edges(ip, ef, op)
        assert np.allclose(got[nz], ufunc.reduceat(ef, starts, axis=0), rtol=1e-13, atol=1e-13)
        assert np.all(got[deg == 0] == 0)
    mean = O.aggregate_edges(ip, ef, "mean")
    assert np.allclose(mean[nz], np.add.reduceat(ef, starts, axis=0) / deg[nz][:, None], rtol=1e-13, atol=1e-13)


@pytest.mark.parametrize("op", ["sum", "mean", "max", "min", "gcn"])
@pytest.mark.parametrize("depth", [1, 2])
def test_edge_feature_layers_equal_computation_tree(op, depth):
    rng = np.random.default_rng(300 + depth)
    n, De = 12, 2
    ip, ix = random_graph(rng, n, 3)
    w = rng.random(ix.shape[0])
    ef = rng.standard_normal((ix.shape[0], De))
    dims = [3, 4, 2][:depth + 1]
    x = rng.standard_normal((n, dims[0]))
    layers = []
    for i in range(depth):
        fi, fo = dims[i], dims[i + 1]
        rows = (fi if op == "gcn" else 2 * fi) + De
        layers.append(L(op, ["relu", "none"][i % 2], rng.standard_normal((rows, fo)), rng.standard_normal(fo),
                        use_edge_weights=(op != "mean"), edge_dim=De))
    full = O.infer(ip, ix, w, x, layers, edge_feat=ef)[-1]
    split = O.infer(ip, ix, w, x, layers, threshold=2, edge_feat=ef)[-1]
    at = O.infer_at(ip, ix, w, x, layers, np.arange(n), threshold=2, edge_feat=ef)
    for v in range(n):
        ref = np.array(tree_eval(v, depth, ip, ix, w, x, layers, ef=ef))
        assert np.allclose(full[v], ref, rtol=1e-11, atol=1e-12), (op, depth, v)
        assert np.allclose(split[v], ref, rtol=1e-11, atol=1e-12), (op, depth, v)
        assert np.allclose(at[v], ref, rtol=1e-11, atol=1e-12), (op, depth, v)


def test_edge_feature_special_cases():
    rng = np.random.default_rng(32)
    n, Fi, De, Fo = 40, 3, 2, 2
    ip, ix = random_graph(rng, n, 6)
    x = rng.standard_normal((n, Fi))
    ef = rng.standard_normal((ix.shape[0], De))
    W = rng.standard_normal((2 * Fi + De, Fo))
    b = rng.standard_normal(Fo)
    # all-zero edge features: the layer without them whose W drops the edge rows (sum / mean; max of zeros is zero too)
    for op in ("sum", "mean", "max"):
        with_zero = O.sage_layer(ip, ix, None, x, L(op, "relu", W, b, edge_dim=De), edge_feat=np.zeros_like(ef))
        without = O.sage_layer(ip, ix, None, x, L(op, "relu", W[:2 * Fi], b))
        assert np.allclose(with_zero, without, rtol=1e-13, atol=1e-13)
    # only the edge rows of W are non-zero and they are the identity: the output is the segment sum of the edge features
    W2 = np.zeros((2 * Fi + De, De))
    W2[2 * Fi:] = np.eye(De)
    out = O.sage_layer(ip, ix, None, x, L("sum", "none", W2, None, edge_dim=De), edge_feat=ef)
    dense = np.zeros((n, De))
    for v in range(n):
        for j in range(ip[v], ip[v + 1]):
            dense[v] += ef[j]
    assert np.allclose(out, dense, rtol=1e-13, atol=1e-13)
    # the vertex part and the edge part of W are not swapped: perturbing an edge row changes the output only
    # where there are in-edges
    W3 = W.copy()
    W3[2 * Fi] += 1.0
    d = O.sage_layer(ip, ix, None, x, L("sum", "none", W3, b, edge_dim=De), edge_feat=ef) - \
        O.sage_layer(ip, ix, None, x, L("sum", "none", W, b, edge_dim=De), edge_feat=ef)
    assert np.allclose(d[:, 0], O.aggregate_edges(ip, ef, "sum")[:, 0], rtol=1e-12, atol=1e-12)


def test_edge_feature_split_invariance_is_exact_for_max_and_integer_sums():
    rng = np.random.default_rng(33)
    ip, ix = random_graph(rng, 30, 40, p_zero=0.1)
    ef_int = rng.integers(-5, 6, size=(ix.shape[0], 3)).astype(np.float64)
    ef = rng.standard_normal((ix.shape[0], 3))
    for T in (1, 3, 7):
        sp, _, owner = O.split_hubs(ip, T)
        for op, e in (("max", ef), ("min", ef), ("sum", ef_int), ("mean", ef_int)):
            P = O.aggregate_edges(sp, e, "sum" if op == "mean" else op)
            assert np.array_equal(O.combine(owner, ip, P, op), O.aggregate_edges(ip, e, op)), (op, T)


def test_compact_neighbourhood_carries_edge_features():
    rng = np.random.default_rng(34)
    n, De = 50, 2
    ip, ix = random_graph(rng, n, 4)
    x = rng.standard_normal((n, 3))
    ef = rng.standard_normal((ix.shape[0], De))
    layers = [L("mean", "relu", rng.standard_normal((2 * 3 + De, 3)), rng.standard_normal(3), edge_dim=De),
              L("max", "none", rng.standard_normal((2 * 3 + De, 2)), None, edge_dim=De)]
    targets = np.array([3, 17, 41])
    full = O.infer(ip, ix, None, x, layers, edge_feat=ef)[-1]
    ids, cip, cix, cw, ct, cef = O.compact_neighbourhood(ip, ix, None, targets, 2, edge_feat=ef)
    got = O.infer_at(cip, cix, cw, x[ids], layers, ct, edge_feat=cef)
    assert np.allclose(got, full[targets], rtol=1e-12, atol=1e-12)


# ------------------------------------------------------------------ learned messages (apply_edge)

class TestW5EdgeMessages:
    g = GOLD["edge_messages"]
    ip = np.array(GOLD["indptr"], np.int64)
    ix = np.array(GOLD["indices"], np.int32)
    x = np.array(GOLD["x"], np.float64)
    w = np.array(GOLD["w"], np.float64)
    ef = np.array(GOLD["edge_features"]["ef"], np.float64)

    def test_messages(self):
        g = self.g
        assert O.edge_messages(self.ix, None, self.x, self.ef, g["W_e"], g["b_e"], g["act_e"]).tolist() == g["messages"]
        assert O.edge_messages(self.ix, self.w, self.x, self.ef, g["W_e"], g["b_e"], g["act_e"]).tolist() == g["weighted_messages"]

    @pytest.mark.parametrize("op", ["sum", "mean", "max"])
    def test_aggregates_of_messages(self, op):
        M = np.array(self.g["messages"], np.float64)
        assert O.aggregate_edges(self.ip, M, op).tolist() == self.g[op]
        sp, _, owner = O.split_hubs(self.ip, GOLD["split_T"])
        P = O.aggregate_edges(sp, M, "sum" if op == "mean" else op)
        if op == "sum":
            assert P[:2].tolist() == self.g["partial_sum_v0"]
        assert O.combine(owner, self.ip, P, op).tolist() == self.g[op]

    def test_layer(self):
        g = self.g
        lay = L("sum", g["act"], g["W"], g["b"], edge_dim=1, W_edge=g["W_e"], bias_edge=g["b_e"], act_edge=g["act_e"])
        for thr in (0, 2):
            for storage in (None, "f32"):
                out = O.layer_forward(self.ip, self.ix, None, self.x, lay, storage=storage, threshold=thr, edge_feat=self.ef)
                assert out.tolist() == g["sage_sum_out"], (thr, storage)
        wl = L("sum", "none", [[0, 0], [0, 0], [1, 0], [0, 1]], None, edge_dim=1, W_edge=g["W_e"], bias_edge=g["b_e"],
               act_edge=g["act_e"], use_edge_weights=True)
        assert O.layer_forward(self.ip, self.ix, self.w, self.x, wl, edge_feat=self.ef).tolist() == g["weighted_sum"]


@pytest.mark.parametrize("op", ["sum", "mean", "max", "min", "gcn"])
@pytest.mark.parametrize("depth", [1, 2])
@pytest.mark.parametrize("De", [0, 2])
def test_message_layers_equal_computation_tree(op, depth, De):
    rng = np.random.default_rng(400 + depth + 10 * De)
    n, Fm = 12, 3
    ip, ix = random_graph(rng, n, 3)
    w = rng.random(ix.shape[0])
    ef = rng.standard_normal((ix.shape[0], De)) if De else None
    dims = [3, 4, 2][:depth + 1]
    x = rng.standard_normal((n, dims[0]))
    layers = []
    for i in range(depth):
        fi, fo = dims[i], dims[i + 1]
        rows = Fm if op == "gcn" else fi + Fm
        layers.append(L(op, ["relu", "none"][i % 2], rng.standard_normal((rows, fo)), rng.standard_normal(fo),
                        use_edge_weights=(op != "mean"), edge_dim=De, W_edge=rng.standard_normal((fi + De, Fm)),
                        bias_edge=rng.standard_normal(Fm), act_edge=["elu", "relu"][i % 2]))
    full = O.infer(ip, ix, w, x, layers, edge_feat=ef)[-1]
    split = O.infer(ip, ix, w, x, layers, threshold=2, edge_feat=ef)[-1]
    at = O.infer_at(ip, ix, w, x, layers, np.arange(n), threshold=2, edge_feat=ef)
    stored = O.infer(ip, ix, w, x, layers, storage="f32", threshold=2, edge_feat=ef)[-1]
    for v in range(n):
        ref = np.array(tree_eval(v, depth, ip, ix, w, x, layers, ef=ef))
        assert np.allclose(full[v], ref, rtol=1e-11, atol=1e-12), (op, depth, v)
        assert np.allclose(split[v], ref, rtol=1e-11, atol=1e-12), (op, depth, v)
        assert np.allclose(at[v], ref, rtol=1e-11, atol=1e-12), (op, depth, v)
        assert np.allclose(stored[v], ref, rtol=2e-5, atol=2e-5), (op, depth, v)


def test_linear_messages_reduce_to_the_plain_aggregates():
    """Without an activation the sum of the messages is a closed form of the plain aggregates:
    sum_j w_j ([h_u | e_j] W_e + b_e) = (sum_j w_j h_u) W_e[:in] + (sum_j w_j e_j) W_e[in:] + (sum_j w_j) b_e."""
    rng = np.random.default_rng(41)
    n, Fi, De, Fm = 40, 3, 2, 4
    ip, ix = random_graph(rng, n, 6)
    x = rng.standard_normal((n, Fi))
    ef = rng.standard_normal((ix.shape[0], De))
    w = rng.random(ix.shape[0])
    We, be = rng.standard_normal((Fi + De, Fm)), rng.standard_normal(Fm)
    M = O.edge_messages(ix, w, x, ef, We, be, "none")
    got = O.aggregate_edges(ip, M, "sum")
    wsum = np.add.reduceat(np.concatenate([w, [0.0]]), np.minimum(ip[:-1], w.size)) * (np.diff(ip) > 0)
    want = O.aggregate(ip, ix, w, x, "sum") @ We[:Fi] + O.aggregate_edges(ip, ef * w[:, None], "sum") @ We[Fi:] + wsum[:, None] * be
    assert np.allclose(got, want, rtol=1e-12, atol=1e-12)
    # no edge features: the message depends on the source alone, so the aggregate is a plain gather of a table
    M0 = O.edge_messages(ix, None, x, None, We[:Fi], be, "relu")
    table = np.maximum(x @ We[:Fi] + be, 0.0)
    assert np.allclose(O.aggregate_edges(ip, M0, "max"), O.aggregate(ip, ix, None, table, "max"), rtol=1e-13, atol=1e-13)
    # the source part and the edge part of W_e are not swapped
    We2 = We.copy()
    We2[Fi] += 1.0
    d = O.edge_messages(ix, None, x, ef, We2, be, "none") - O.edge_messages(ix, None, x, ef, We, be, "none")
    assert np.allclose(d, np.repeat(ef[:, :1], Fm, axis=1), rtol=1e-12, atol=1e-12)


# ------------------------------------------------------------------ GAT with edge features in the logits

def gat_edge_layer(rng, fi, heads, hd, De, act="none"):
    return L("gat", act, rng.standard_normal((fi, heads * hd)), rng.standard_normal(heads * hd), heads=heads,
             att_src=rng.standard_normal((heads, hd)), att_dst=rng.standard_normal((heads, hd)), edge_dim=De,
             att_edge=rng.standard_normal((heads, De)))


@pytest.mark.parametrize("depth", [1, 2])
def test_gat_with_edge_logits_equals_computation_tree(depth):
    rng = np.random.default_rng(500 + depth)
    n, De = 12, 3
    ip, ix = random_graph(rng, n, 4)
    ef = rng.standard_normal((ix.shape[0], De))
    x = rng.standard_normal((n, 4))
    layers = [gat_edge_layer(rng, 4, 2, 2, De, act="elu"), gat_edge_layer(rng, 4, 1, 3, De)][:depth]
    full = O.infer(ip, ix, None, x, layers, edge_feat=ef)[-1]
    at = O.infer_at(ip, ix, None, x, layers, np.arange(n), edge_feat=ef)
    stored = O.infer(ip, ix, None, x, layers, storage="f32", edge_feat=ef)[-1]
    for v in range(n):
        ref = np.array(tree_eval(v, depth, ip, ix, None, x, layers, ef=ef))
        assert np.allclose(full[v], ref, rtol=1e-11, atol=1e-12), (depth, v)
        assert np.allclose(at[v], ref, rtol=1e-11, atol=1e-12), (depth, v)
        assert np.allclose(stored[v], ref, rtol=2e-5, atol=2e-5), (depth, v)


def test_gat_edge_logit_special_cases():
    rng = np.random.default_rng(51)
    n, De = 30, 2
    ip, ix = random_graph(rng, n, 5)
    x = rng.standard_normal((n, 4))
    ef = rng.standard_normal((ix.shape[0], De))
    lay = gat_edge_layer(rng, 4, 2, 3, De)
    plain = L("gat", "none", lay.W, lay.bias, heads=2, att_src=lay.att_src, att_dst=lay.att_dst)
    base = O.gat_layer(ip, ix, x, plain)
    # zero edge features, or a zero attention vector for them: the plain GAT layer
    assert np.array_equal(O.gat_layer(ip, ix, x, lay, edge_feat=np.zeros_like(ef)), base)
    zero_att = L("gat", "none", lay.W, lay.bias, heads=2, att_src=lay.att_src, att_dst=lay.att_dst, edge_dim=De, att_edge=np.zeros((2, De)))
    assert np.array_equal(O.gat_layer(ip, ix, x, zero_att, edge_feat=ef), base)
    # a softmax is unchanged by a shift of all its logits: with positive logits throughout (where the LeakyReLU is
    # the identity) an edge term that is the same for all in-edges of a destination changes nothing
    pos = L("gat", "none", lay.W, lay.bias, heads=2, att_src=np.zeros((2, 3)), att_dst=np.zeros((2, 3)), edge_dim=1, att_edge=np.ones((2, 1)))
    const = np.repeat(rng.random(n) + 1.0, np.diff(ip))[:, None]     # one value per destination
    flat = L("gat", "none", lay.W, lay.bias, heads=2, att_src=np.zeros((2, 3)), att_dst=np.zeros((2, 3)))
    assert np.allclose(O.gat_layer(ip, ix, x, pos, edge_feat=const), O.gat_layer(ip, ix, x, flat), rtol=1e-12, atol=1e-12)
    # two in-edges, logits from the edge features alone: alpha = sigmoid of their difference
    ip2, ix2 = np.array([0, 2, 2], np.int64), np.array([0, 1], np.int32)
    x2 = np.array([[1.0, 2.0], [3.0, -1.0]])
    lay2 = L("gat", "none", np.eye(2), None, heads=1, att_src=[[0, 0]], att_dst=[[0, 0]], edge_dim=1, att_edge=[[1.0]])
    e = np.array([[0.7], [1.9]])
    a0 = 1.0 / (1.0 + math.exp(1.9 - 0.7))
    out = O.gat_layer(ip2, ix2, x2, lay2, edge_feat=e)
    assert np.allclose(out[0], a0 * x2[0] + (1 - a0) * x2[1], rtol=1e-14)
    # a hugely negative edge term removes the edge from the softmax: the graph without that edge
    ef_big = np.zeros((ix.shape[0], 1))
    v = int(np.argmax(np.diff(ip)))
    ef_big[ip[v]] = -1e4
    drop = L("gat", "none", lay.W, lay.bias, heads=2, att_src=lay.att_src, att_dst=lay.att_dst, edge_dim=1, att_edge=np.ones((2, 1)))
    got = O.gat_layer(ip, ix, x, drop, edge_feat=ef_big)[v]
    ip3 = ip.copy(); ip3[v + 1:] -= 1
    ix3 = np.delete(ix, ip[v])
    assert np.allclose(got, O.gat_layer(ip3, ix3, x, plain)[v], rtol=1e-12, atol=1e-12)
