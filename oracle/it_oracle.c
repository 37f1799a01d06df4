/*
 * CPU oracle for one Gather-Apply-Scatter layer of full-graph GNN inference.
 *
 * TEST INFRASTRUCTURE ONLY.  This file is the plain definition of what a layer
 * computes, written out slowly in fp64 so that it can be checked against the paper
 * by eye.  It shares no code with the CUDA library and must never be used by it:
 * only the tests, the smoke check and the benchmark's CPU-baseline leg call it.
 *
 * What it follows (InferTurbo, arXiv 2307.00228):
 *   - Eq. (1): message m_{v,u} = M(h_v, h_u, e_{v,u}); update h_v' = U(h_v, R({m})).
 *   - Section "InferTurbo Abstraction": Gather (gather_nbrs + aggregate), Apply
 *     (apply_node), Scatter (apply_edge + scatter_nbrs); aggregate must be commutative
 *     and associative (sum / mean / max); GAT unions the messages in aggregate and
 *     does its attention-weighted reduce in apply_node.
 *   - Section "Optimization Strategies": partial-gather (aggregate what is available
 *     for one destination first, aggregate the partial results afterwards) and shadow
 *     nodes (the edges of a hub are cut into n equal groups, one mirror per group, the
 *     mirror id carries the group number).
 *
 * The graph is CSR by destination: the in-edges of vertex v are the entries
 * j in [indptr[v], indptr[v+1]); indices[j] is the source u_j; w[j] an optional scalar
 * edge weight (the minimal apply_edge: message = w_j * h_{u_j}).
 *
 * All floating-point inputs arrive already widened to double; all arithmetic is
 * double.  Loops over destinations may run under OpenMP (each destination is
 * independent); the order of operations inside a destination is fixed.
 *
 * Accuracy on the paper's real datasets (PPI, Products, MAG240M): parity unpinned
 * (those datasets and the trained weights are not available).
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

enum { ITO_SUM = 0, ITO_MEAN = 1, ITO_MAX = 2, ITO_MIN = 3 };
enum { ITO_ACT_NONE = 0, ITO_ACT_RELU = 1, ITO_ACT_ELU = 2 };

/* ------------------------------------------------------------------ index side */

/* Shadow-node rule applied to in-edge segments (the edges of a hub are cut into n groups of
 * equal size).  A vertex with in-degree d > T is split into n = ceil(d / T) groups; group g
 * takes the next contiguous run of base + (g < rem) edges, base = d / n, rem = d % n.
 * A vertex with d <= T (including d = 0) keeps exactly one row.  T <= 0: never split. */
static int64_t groups_of(int64_t d, int64_t T) {
    if (T <= 0 || d <= T) return 1;
    return (d + T - 1) / T;
}

int64_t ito_split_count(int64_t n, const int64_t *indptr, int64_t T) {
    int64_t rows = 0;
    for (int64_t v = 0; v < n; ++v) rows += groups_of(indptr[v + 1] - indptr[v], T);
    return rows;
}

/* shadow_indptr[R+1], shadow_owner[R], owner_indptr[n+1].  Row id = owner_indptr[v] + g. */
void ito_split_hubs(int64_t n, const int64_t *indptr, int64_t T, int64_t *shadow_indptr,
                    int32_t *shadow_owner, int64_t *owner_indptr) {
    int64_t r = 0;
    for (int64_t v = 0; v < n; ++v) {
        int64_t d = indptr[v + 1] - indptr[v];
        int64_t g_count = groups_of(d, T);
        int64_t base = d / g_count, rem = d % g_count;
        int64_t pos = indptr[v];
        owner_indptr[v] = r;
        for (int64_t g = 0; g < g_count; ++g) {
            shadow_indptr[r] = pos;
            shadow_owner[r] = (int32_t)v;
            pos += base + (g < rem ? 1 : 0);
            ++r;
        }
    }
    owner_indptr[n] = r;
    shadow_indptr[r] = indptr[n];
}

/* Degree buckets: row r of length len goes to the first bucket b with len <= bounds[b]
 * (bounds ascending; the last bound must cover every row).  Inside a bucket rows keep
 * ascending row id.  bucket_offsets[nb+1], bucket_rows[R].  Returns 0, or -1 if a row
 * fits no bucket. */
int ito_buckets(int64_t n_rows, const int64_t *shadow_indptr, int32_t nb, const int64_t *bounds,
                int64_t *bucket_offsets, int32_t *bucket_rows) {
    int64_t *count = (int64_t *)calloc((size_t)nb + 1, sizeof(int64_t));
    for (int64_t r = 0; r < n_rows; ++r) {
        int64_t len = shadow_indptr[r + 1] - shadow_indptr[r];
        int32_t b = 0;
        while (b < nb && len > bounds[b]) ++b;
        if (b == nb) { free(count); return -1; }
        count[b]++;
    }
    bucket_offsets[0] = 0;
    for (int32_t b = 0; b < nb; ++b) bucket_offsets[b + 1] = bucket_offsets[b] + count[b];
    for (int32_t b = 0; b < nb; ++b) count[b] = bucket_offsets[b];
    for (int64_t r = 0; r < n_rows; ++r) {
        int64_t len = shadow_indptr[r + 1] - shadow_indptr[r];
        int32_t b = 0;
        while (len > bounds[b]) ++b;
        bucket_rows[count[b]++] = (int32_t)r;
    }
    free(count);
    return 0;
}

/* ------------------------------------------------------------------ aggregate */

/* aggregate over the in-edges of every vertex (Eq. (1), reduce R; Section "InferTurbo
 * Abstraction", aggregate):
 *   sum : a_v    = sum_j w_j h_{u_j}
 *   mean: a_v    = (sum_j w_j h_{u_j}) / d_v        (d_v = number of in-edges)
 *   max : a_v[f] = max_j (w_j h_{u_j}[f])
 *   min : a_v[f] = min_j (w_j h_{u_j}[f])      (Section "Background", message passing: the reduce
 *                                               may be sum, mean, max or min pooling)
 * An empty in-neighbourhood gives a_v = 0.  H is [n_src, F] row-major, A is [n, F]. */
void ito_aggregate(int64_t n, const int64_t *indptr, const int32_t *indices, const double *w,
                   const double *H, int32_t F, int32_t op, double *A) {
#pragma omp parallel for schedule(dynamic, 256)
    for (int64_t v = 0; v < n; ++v) {
        double *a = A + v * F;
        int64_t j0 = indptr[v], j1 = indptr[v + 1];
        for (int32_t f = 0; f < F; ++f) a[f] = 0.0;
        for (int64_t j = j0; j < j1; ++j) {
            const double *h = H + (int64_t)indices[j] * F;
            double wj = w ? w[j] : 1.0;
            for (int32_t f = 0; f < F; ++f) {
                double m = wj * h[f];
                if (op == ITO_MAX) a[f] = (j == j0 || m > a[f]) ? m : a[f];
                else if (op == ITO_MIN) a[f] = (j == j0 || m < a[f]) ? m : a[f];
                else a[f] += m;
            }
        }
        if (op == ITO_MEAN && j1 > j0)
            for (int32_t f = 0; f < F; ++f) a[f] /= (double)(j1 - j0);
    }
}

/* aggregate of the edge features themselves (Eq. (1): the message function M may read the feature vector
 * e_{v,u} of the edge; here that part of the message is e_{v,u} as it is).  EF is [n_edges, De] row-major,
 * row j belonging to CSR entry j, so the in-edges of v own the consecutive rows indptr[v] .. indptr[v+1]-1:
 *   sum : ae_v    = sum_j e_j          mean: divided by the number of in-edges
 *   max : ae_v[f] = max_j e_j[f]       min : ae_v[f] = min_j e_j[f]
 * An empty in-neighbourhood gives 0.  `segptr` may also be the shadow-row pointer (partial results per group;
 * pass SUM for a mean then).  AE is [n_seg, De]. */
void ito_aggregate_edges(int64_t n_seg, const int64_t *segptr, const double *EF, int32_t De, int32_t op, double *AE) {
#pragma omp parallel for schedule(dynamic, 256)
    for (int64_t v = 0; v < n_seg; ++v) {
        double *a = AE + v * De;
        int64_t j0 = segptr[v], j1 = segptr[v + 1];
        for (int32_t f = 0; f < De; ++f) a[f] = 0.0;
        for (int64_t j = j0; j < j1; ++j) {
            const double *e = EF + j * De;
            for (int32_t f = 0; f < De; ++f) {
                if (op == ITO_MAX) a[f] = (j == j0 || e[f] > a[f]) ? e[f] : a[f];
                else if (op == ITO_MIN) a[f] = (j == j0 || e[f] < a[f]) ? e[f] : a[f];
                else a[f] += e[f];
            }
        }
        if (op == ITO_MEAN && j1 > j0)
            for (int32_t f = 0; f < De; ++f) a[f] /= (double)(j1 - j0);
    }
}

/* apply_edge with a learned message function (Eq. (1): m_{v,u} = M(h_v, h_u, e_{v,u}); Section "InferTurbo
 * Abstraction", Scatter stage: apply_edge makes the message of an edge out of the source's state and the edge's
 * features).  Here M is one dense layer on the concatenation of the two, scaled by the optional edge weight:
 *   m_j = w_j * act( h_{u_j} W_e[0:Fi, :] + e_j W_e[Fi:Fi+De, :] + b_e ),     W_e [Fi + De, Fm] row-major.
 * De may be 0 (no edge features; EF unused), b_e and w may be NULL.  M is [n_edges, Fm], row j for CSR entry j;
 * the Gather stage then reduces the rows of a destination with ito_aggregate_edges. */
static double activate(double x, int32_t act);
void ito_edge_messages(int64_t n_edges, const int32_t *indices, const double *w, const double *H, int32_t Fi,
                       const double *EF, int32_t De, const double *We, const double *be, int32_t Fm, int32_t act,
                       double *M) {
#pragma omp parallel for schedule(static)
    for (int64_t j = 0; j < n_edges; ++j) {
        const double *h = H + (int64_t)indices[j] * Fi;
        double *m = M + j * Fm;
        for (int32_t c = 0; c < Fm; ++c) m[c] = be ? be[c] : 0.0;
        for (int32_t k = 0; k < Fi; ++k)
            for (int32_t c = 0; c < Fm; ++c) m[c] += h[k] * We[(int64_t)k * Fm + c];
        for (int32_t k = 0; k < De; ++k)
            for (int32_t c = 0; c < Fm; ++c) m[c] += EF[j * De + k] * We[(int64_t)(Fi + k) * Fm + c];
        for (int32_t c = 0; c < Fm; ++c) m[c] = (w ? w[j] : 1.0) * activate(m[c], act);
    }
}

/* Partial gather: the same aggregate, but per shadow row (one group of a vertex's
 * in-edges).  Mean rows hold plain sums; the division happens once, in combine.
 * P is [R, F]. */
void ito_partial_gather(int64_t n_rows, const int64_t *shadow_indptr, const int32_t *indices,
                        const double *w, const double *H, int32_t F, int32_t op, double *P) {
    ito_aggregate(n_rows, shadow_indptr, indices, w, H, F, (op == ITO_MAX || op == ITO_MIN) ? op : ITO_SUM, P);
}

/* Combine: the receiver aggregates the partial results of one vertex "as usual", in
 * group order.  Empty groups can only occur for d = 0 (a single empty row), so a max
 * or a min never sees a spurious 0.  deg[v] = indptr[v+1]-indptr[v] of the unsplit graph. */
void ito_combine(int64_t n, const int64_t *owner_indptr, const int64_t *indptr, const double *P,
                 int32_t F, int32_t op, double *A) {
#pragma omp parallel for schedule(static)
    for (int64_t v = 0; v < n; ++v) {
        double *a = A + v * F;
        int64_t r0 = owner_indptr[v], r1 = owner_indptr[v + 1];
        for (int32_t f = 0; f < F; ++f) a[f] = P[r0 * F + f];
        for (int64_t r = r0 + 1; r < r1; ++r)
            for (int32_t f = 0; f < F; ++f) {
                double p = P[r * F + f];
                if (op == ITO_MAX) a[f] = p > a[f] ? p : a[f];
                else if (op == ITO_MIN) a[f] = p < a[f] ? p : a[f];
                else a[f] += p;
            }
        int64_t d = indptr[v + 1] - indptr[v];
        if (op == ITO_MEAN && d > 0)
            for (int32_t f = 0; f < F; ++f) a[f] /= (double)d;
    }
}

/* ------------------------------------------------------------------ apply */

static double activate(double x, int32_t act) {
    if (act == ITO_ACT_RELU) return x > 0.0 ? x : 0.0;
    if (act == ITO_ACT_ELU) return x > 0.0 ? x : expm1(x);
    return x;
}

/* out[v, :] = X[v, :] W, W is [K, Fo] row-major.  A plain dense product. */
void ito_linear(int64_t n, const double *X, int32_t K, const double *W, int32_t Fo, double *out) {
#pragma omp parallel for schedule(static)
    for (int64_t v = 0; v < n; ++v) {
        double *o = out + v * Fo;
        for (int32_t c = 0; c < Fo; ++c) o[c] = 0.0;
        for (int32_t k = 0; k < K; ++k) {
            double x = X[v * K + k];
            const double *wr = W + (int64_t)k * Fo;
            for (int32_t c = 0; c < Fo; ++c) o[c] += x * wr[c];
        }
    }
}

/* GraphSAGE apply_node: the vertex combines its former state with the gathered message,
 *   h'_v = act( h_v W[0:Fi, :] + a_v W[Fi:2Fi, :] + b ).
 * W is [2*Fi, Fo] row-major, bias may be NULL. */
void ito_sage_apply(int64_t n, const double *H, const double *A, int32_t Fi, const double *W,
                    const double *bias, int32_t Fo, int32_t act, double *out) {
#pragma omp parallel for schedule(static)
    for (int64_t v = 0; v < n; ++v) {
        double *o = out + v * Fo;
        for (int32_t c = 0; c < Fo; ++c) o[c] = bias ? bias[c] : 0.0;
        for (int32_t k = 0; k < Fi; ++k) {
            double h = H[v * Fi + k], a = A[v * Fi + k];
            const double *ws = W + (int64_t)k * Fo, *wn = W + (int64_t)(Fi + k) * Fo;
            for (int32_t c = 0; c < Fo; ++c) o[c] += h * ws[c] + a * wn[c];
        }
        for (int32_t c = 0; c < Fo; ++c) o[c] = activate(o[c], act);
    }
}

/* out = act(X + bias) elementwise over [n, F]; bias may be NULL. */
void ito_bias_act(int64_t n, int32_t F, const double *X, const double *bias, int32_t act,
                  double *out) {
#pragma omp parallel for schedule(static)
    for (int64_t v = 0; v < n; ++v)
        for (int32_t c = 0; c < F; ++c)
            out[v * F + c] = activate(X[v * F + c] + (bias ? bias[c] : 0.0), act);
}

/* ------------------------------------------------------------------ GAT */

/* Attention scores of every vertex: s[v, k] = att[k, :] . z_v^k, z_v^k the k-th block of
 * D = F / heads entries of Z[v, :]. */
void ito_gat_scores(int64_t n, const double *Z, int32_t heads, int32_t D, const double *att,
                    double *s) {
#pragma omp parallel for schedule(static)
    for (int64_t v = 0; v < n; ++v)
        for (int32_t k = 0; k < heads; ++k) {
            double acc = 0.0;
            for (int32_t c = 0; c < D; ++c) acc += att[k * D + c] * Z[v * heads * D + k * D + c];
            s[v * heads + k] = acc;
        }
}

/* GAT reduce (done in apply_node because it is not associative): per destination v and
 * head k,
 *   e_j     = LeakyReLU_slope( s_src[u_j, k] + s_dst[v, k] + c[j, k] )      (c: see below; 0 when absent)
 *   alpha_j = exp(e_j - max_j e_j) / sum_j exp(e_j - max_j e_j)
 *   o_v^k   = sum_j alpha_j z_{u_j}^k
 * Empty in-neighbourhood: o_v = 0.  Z is the message table [n_src, heads*D] (it may be a
 * rounded copy of the z the scores were computed from); O is [n, heads*D].
 * edge_logit (may be NULL) is [n_edges, heads]: the share of the edge's own features in the attention
 * logit, c[j, k] = att_edge[k] . e_j (Eq. (1): the message function may read e_{v,u}; with attention
 * the edge features enter the logit next to the two vertex terms). */
void ito_gat_aggregate(int64_t n, const int64_t *indptr, const int32_t *indices, const double *Z,
                       const double *s_src, const double *s_dst, int32_t heads, int32_t D,
                       double slope, const double *edge_logit, double *O) {
    int32_t F = heads * D;
#pragma omp parallel for schedule(dynamic, 256)
    for (int64_t v = 0; v < n; ++v) {
        int64_t j0 = indptr[v], j1 = indptr[v + 1];
        double *o = O + v * F;
        for (int32_t f = 0; f < F; ++f) o[f] = 0.0;
        for (int32_t k = 0; k < heads; ++k) {
            double emax = -INFINITY;
            for (int64_t j = j0; j < j1; ++j) {
                double e = s_src[(int64_t)indices[j] * heads + k] + s_dst[v * heads + k] + (edge_logit ? edge_logit[j * heads + k] : 0.0);
                e = e > 0.0 ? e : slope * e;
                if (e > emax) emax = e;
            }
            double denom = 0.0;
            for (int64_t j = j0; j < j1; ++j) {
                double e = s_src[(int64_t)indices[j] * heads + k] + s_dst[v * heads + k] + (edge_logit ? edge_logit[j * heads + k] : 0.0);
                e = e > 0.0 ? e : slope * e;
                denom += exp(e - emax);
            }
            for (int64_t j = j0; j < j1; ++j) {
                double e = s_src[(int64_t)indices[j] * heads + k] + s_dst[v * heads + k] + (edge_logit ? edge_logit[j * heads + k] : 0.0);
                e = e > 0.0 ? e : slope * e;
                double alpha = exp(e - emax) / denom;
                const double *z = Z + (int64_t)indices[j] * F + k * D;
                for (int32_t c = 0; c < D; ++c) o[k * D + c] += alpha * z[c];
            }
        }
    }
}
