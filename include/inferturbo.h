/*
 * inferturbo.h — C ABI of the B200 (sm_100a) layer-pass library.
 *
 * One Gather-Apply-Scatter layer pass of full-graph GNN inference over every vertex,
 * repeated layer after layer with no sampling (InferTurbo, arXiv 2307.00228).
 *
 * Conventions for every call
 *   - "device pointer" = memory on the current CUDA device, allocated by the caller.
 *     The library BORROWS caller arrays (never frees, never writes inputs) and OWNS
 *     only what it derives inside an it_graph (freed by it_graph_destroy).
 *   - `stream` is a cudaStream_t passed as void* (NULL = the default stream).  Work is
 *     enqueued on it; a call synchronises that stream only where it must read a status
 *     or a count back (it_graph_create, it_split_hubs).
 *   - Matrices are row-major and dense.  Feature rows (layer inputs and outputs, edge features) must be a
 *     multiple of 16 bytes; the pooling layers and GCN take any such width (rows other than 16, 32, ..., 512
 *     bytes are gathered in column chunks of those widths), GAT rows must be one of those widths.  The dense
 *     transform runs on the tensor cores when out_dim is a multiple of 16 and on the CUDA cores otherwise.
 *   - Errors are return codes only: nothing throws, aborts or traps the device.  On
 *     error no output is defined.  it_status_string() names a code;
 *     it_last_error_message() gives the detail of the calling thread's last failure.
 */
#ifndef INFERTURBO_H
#define INFERTURBO_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct it_graph it_graph; /* opaque, library-owned */

typedef enum {
  IT_OK = 0,
  IT_ERR_INVALID_ARG = 1, /* NULL pointer, negative size, bad enum, dims not supported by shape rules */
  IT_ERR_BAD_GRAPH = 2,   /* indptr not monotone / wrong ends, or a source id outside [0, n) */
  IT_ERR_UNSUPPORTED = 3, /* a valid request this build has no kernel for */
  IT_ERR_WORKSPACE = 4,   /* workspace NULL, misaligned or smaller than it_workspace_bytes() */
  IT_ERR_OOM = 5,         /* device allocation of library-owned arrays failed */
  IT_ERR_CUDA = 6,        /* a CUDA call or kernel launch failed */
  IT_ERR_TIMEOUT = 7      /* a bounded device-side wait gave up */
} it_status;

typedef enum { IT_F32 = 0, IT_BF16 = 1 } it_dtype;
typedef enum { IT_I32 = 0, IT_I64 = 1 } it_itype;
typedef enum {
  IT_GATHER_SUM = 0, IT_GATHER_MEAN = 1, IT_GATHER_MAX = 2, IT_GATHER_GAT = 3, IT_GATHER_MIN = 4,
  IT_GATHER_NONE = 5,   /* no Gather stage: a dense layer */
  IT_GATHER_GCN = 6     /* sum aggregate, update on the aggregate alone */
} it_gather_op;
typedef enum { IT_ACT_NONE = 0, IT_ACT_RELU = 1, IT_ACT_ELU = 2 } it_act;

#define IT_MAX_BUCKETS 8

/*
 * One GNN layer in the paper's stage vocabulary (Section "InferTurbo Abstraction"):
 * `op` is the aggregate of the Gather stage, W / bias / act are apply_node, and
 * use_edge_weights selects the minimal apply_edge (message = w_e * h_src).
 *
 * GraphSAGE (op = SUM | MEAN | MAX | MIN; the paper's message-passing paradigm lists all four poolings):
 *     a_v  = op_{e = (u -> v)} ( w_e * h_u )            (0 for a vertex with no in-edge;
 *                                                        MEAN divides by the edge count)
 *     h'_v = act( h_v * W[0:in_dim, :] + a_v * W[in_dim:2*in_dim, :] + bias )
 *   W is [2*in_dim, out_dim].
 * GAT (op = GAT; out_dim = heads * head_dim):
 *     z_u = h_u * W                                      W is [in_dim, out_dim]
 *     e   = LeakyReLU_slope( att_src[k] . z_u^k + att_dst[k] . z_v^k )    per head k
 *     h'_v = act( concat_k sum_e softmax_e(e) z_u^k + bias )
 *   The message-passing form is Eq. (1); the paper places GAT's reduce in apply_node
 *   because attention is not associative.
 *
 * Dense (op = NONE): h'_v = act( h_v * W + bias ), W is [in_dim, out_dim].  The paper's first superstep
 *   (raw vertex states -> initial embeddings) and the prediction part attached after the last
 *   apply_node (Section "Implementation on Pregel") are layers of this kind.
 * GCN (op = GCN): a_v = sum_e w_e * h_u (w_e = 1 without edge weights), h'_v = act( a_v * W + bias ),
 *   W is [in_dim, out_dim].  The degree normalisation is carried by the edge weights and a self loop is
 *   an edge of the graph like any other; the vertex's own state enters in no other way.
 *
 * Edge features (edge_dim > 0; pooling layers and GCN; for GAT see below): Eq. (1) lets the message function M read the feature
 *   vector e_{v,u} of the edge next to the source state.  The message here is the concatenation
 *       m_{v,u} = [ w_e * h_u | e_{v,u} ]                      (in_dim + edge_dim entries)
 *   reduced entry by entry with the layer's op (MEAN divides both parts by the edge count), so that
 *       GraphSAGE: h'_v = act( h_v * W[0:in_dim] + a_v * W[in_dim : 2*in_dim + edge_dim] + bias ),  W is [2*in_dim + edge_dim, out_dim]
 *       GCN:       h'_v = act( a_v * W + bias ),                                                  W is [in_dim + edge_dim, out_dim]
 *   Every message function that is linear in (h_u, e_{v,u}) and is followed by a sum or mean and a dense update
 *   folds into this form.  The vectors come from it_graph_set_edge_features; such layers are never reordered.
 *
 * GAT with edge features (op = GAT, edge_dim > 0): the edge's features enter its attention logit,
 *       e = LeakyReLU_slope( att_src[k] . z_u^k + att_dst[k] . z_v^k + att_edge[k] . e_{v,u} ),
 *   the messages stay z_u.  One fp32 logit term per edge and head (source score + edge share) and the message
 *   row of every edge are materialised in the workspace ([n_edges, heads] fp32 and [n_edges, out_dim] feat_dtype).
 *
 * Learned messages (msg_dim > 0; pooling layers and GCN): the general apply_edge of the Scatter stage (Section
 *   "InferTurbo Abstraction"; M of Eq. (1)) as one dense layer on the source state and the edge's features,
 *       m_{v,u} = w_e * act_edge( h_u * W_edge[0:in_dim] + e_{v,u} * W_edge[in_dim:in_dim+edge_dim] + bias_edge ),
 *   msg_dim entries, reduced entry by entry with the layer's op (w_e = 1 without edge weights; edge_dim may be 0), then
 *       GraphSAGE: h'_v = act( h_v * W[0:in_dim] + a_v * W[in_dim : in_dim + msg_dim] + bias ),  W is [in_dim + msg_dim, out_dim]
 *       GCN:       h'_v = act( a_v * W + bias ),                                             W is [msg_dim, out_dim]
 *   The source part h_u * W_edge[0:in_dim] is computed once per vertex and the edge part once per edge, both by the dense
 *   transform; they, and the finished messages, are stored in feat_dtype.  Never reordered.
 *
 * Storage contract: h_in, h_out (and the internal Z / aggregate tensors) are feat_dtype,
 * rounded to nearest even when written; all accumulation is fp32.  W is weight_dtype and
 * must equal feat_dtype.  bias, att_src, att_dst are fp32.  All are device pointers.
 */
typedef struct {
  it_gather_op op;
  it_act act;
  int32_t in_dim, out_dim, heads;       /* heads = 1 unless GAT */
  it_dtype feat_dtype, weight_dtype;
  const void *W;
  const float *bias;                    /* [out_dim], may be NULL */
  const float *att_src, *att_dst;       /* GAT only: [heads, out_dim / heads] */
  float leaky_slope;                    /* GAT only */
  int32_t use_edge_weights;             /* 0/1; needs a graph created with edge weights */
  int32_t allow_reorder;                /* 0/1: allow transform-before-aggregate (see it_layer_forward) */
  int32_t edge_dim;                     /* 0, or the length of the edge-feature vectors the messages carry (see below) */
  int32_t msg_dim;                      /* 0, or the length of a learned message (see "Learned messages") */
  it_act act_edge;                      /* learned messages: activation of the message function */
  const void *W_edge;                   /* learned messages: [in_dim + edge_dim, msg_dim], weight_dtype */
  const float *bias_edge;               /* learned messages: [msg_dim], may be NULL */
  const float *att_edge;                /* GAT with edge_dim > 0: [heads, edge_dim] fp32 */
} it_layer_desc;

/*
 * it_graph_create — accept a directed, weighted graph G = {V, E, X, E} (Section
 * "K-hop Neighborhood and Sampling") as CSR by destination: the in-edges of vertex v
 * are entries [indptr[v], indptr[v+1]) of `indices` (source ids) and `edge_weights`.
 * Multi-edges and self-edges are allowed; each entry is one message.
 *   n_vertices in [0, 2^31 - 2]; n_edges >= 0 (int64).
 *   indptr: device, n_vertices + 1 entries of indptr_type.  indices: device int32.
 *   edge_weights: device fp32 [n_edges] or NULL.
 * The CSR is validated on the device (indptr[0] = 0, non-decreasing, indptr[n] = n_edges,
 * 0 <= source < n): IT_ERR_BAD_GRAPH if not.  The arrays are borrowed until
 * it_graph_destroy.  The new graph starts unsplit (as after it_split_hubs(g, 0)).
 * Synchronises `stream`.
 */
it_status it_graph_create(int64_t n_vertices, int64_t n_edges, const void *indptr,
                          it_itype indptr_type, const int32_t *indices,
                          const float *edge_weights, void *stream, it_graph **out);

/*
 * it_graph_set_edge_features — attach the edge features E of G = {V, E, X, E} (Section "K-hop Neighborhood and
 * Sampling"; e_{v,u} of Eq. (1)): a device matrix [n_edges, edge_dim] of `dtype`, row j belonging to CSR entry j
 * (the same order as `indices` and `edge_weights`).  Borrowed until it_graph_destroy or the next call; NULL with
 * edge_dim = 0 detaches them.  A row must be a multiple of 16 bytes.  Nothing is launched.
 */
it_status it_graph_set_edge_features(it_graph *g, const void *edge_feat, int32_t edge_dim, it_dtype dtype);

/*
 * it_split_hubs — the shadow-node rule (Section "Optimization Strategies", Shadow Nodes: the
 * edges of a hub are cut into n groups of equal size, one mirror per group, the mirror's id
 * being the vertex id extended by the group number) applied to the in-edge segment of every
 * vertex whose in-degree d exceeds `threshold` T, so that each group can be gathered on its
 * own and the partial results combined (Partial-Gather, same section).
 *   n = 1 if d <= T (or T <= 0), else ceil(d / T) groups; group g takes the next
 *   d / n + (g < d % n) consecutive edges.  Row id = owner_indptr[v] + g.
 * Also builds the degree buckets: shadow rows partitioned stably by length class
 * (bounds from it_graph_get_split).  Rebuilds everything derived; edge arrays are not
 * permuted.  out_n_rows / out_n_split_owners may be NULL.  Synchronises `stream`.
 */
it_status it_split_hubs(it_graph *g, int64_t threshold, void *stream, int64_t *out_n_rows,
                        int64_t *out_n_split_owners);

/*
 * it_graph_get_split — borrowed device pointers to the derived index arrays (valid until
 * the next it_split_hubs / it_graph_destroy):
 *   shadow_indptr int64[R+1], shadow_owner int32[R], owner_indptr int64[n+1],
 *   bucket_offsets int64[n_buckets+1], bucket_rows int32[R] (ascending row id inside a
 *   bucket), and the bucket upper bounds copied to the HOST array bucket_bounds
 *   (IT_MAX_BUCKETS entries; row of length L is in the first bucket with L <= bound).
 * Any out pointer may be NULL.
 */
it_status it_graph_get_split(const it_graph *g, int64_t *n_rows, const int64_t **shadow_indptr,
                             const int32_t **shadow_owner, const int64_t **owner_indptr,
                             const int64_t **bucket_offsets, const int32_t **bucket_rows,
                             int32_t *n_buckets, int64_t *bucket_bounds);

/*
 * it_workspace_bytes — bytes of caller-provided device scratch that it_infer needs for
 * these layers on this graph (with its current split); it_layer_forward of any one of
 * them needs no more.  Layer pointers inside `layers` are not dereferenced.
 */
it_status it_workspace_bytes(const it_graph *g, const it_layer_desc *layers, int32_t n_layers,
                             size_t *out_bytes);

/*
 * it_layer_forward — one layer for every vertex: gather (per shadow row, by degree
 * bucket) -> combine the partial results of split vertices -> apply -> write h_out, which
 * the next layer reads ("scatter": on one device sending along out-edges is a store).
 *   h_in  [n, in_dim], h_out [n, out_dim], feat_dtype, device, must not overlap.
 *   workspace: device, 256-byte aligned, >= it_workspace_bytes(g, layer, 1).
 * If allow_reorder and op is SUM, MEAN or GCN and out_dim < in_dim, the neighbour transform is
 * done before the gather (Section "Inference" allows the order of a layer's computation to be
 * rearranged for speed): Z = h_in * W[in_dim:, :] is stored in feat_dtype and gathered instead of
 * h_in; the self term h_in * W[0:in_dim, :] + bias is stored in feat_dtype as well.
 * Asynchronous on `stream`.  Results are bit-identical from run to run.
 */
it_status it_layer_forward(const it_graph *g, const it_layer_desc *layer, const void *h_in,
                           void *h_out, void *workspace, size_t workspace_bytes, void *stream);

/*
 * it_infer — L layers in order (Section "InferTurbo on Graph Processing System": one layer
 * per iteration over all vertices, a k-layer model after k of them): the sequence of
 * it_layer_forward calls, intermediate layer outputs double-buffered inside the
 * workspace.  x [n, layers[0].in_dim]; out [n, layers[L-1].out_dim]; layers[i].out_dim must
 * equal layers[i+1].in_dim and all feat_dtype agree.  Bit-identical to calling
 * it_layer_forward layer by layer.  Where layer i + 1 transforms before it aggregates (its table is
 * H_i W), the output H_i of layer i feeds that transform and nothing else; for bf16 layers whose
 * widths are multiples of 64 the update of layer i and that transform then run as one kernel that
 * rounds each tile of H_i to bf16 as it would be stored and keeps it on the SM, so H_i is neither
 * written to nor read from device memory (same results, bit for bit).  Asynchronous on `stream`.
 */
it_status it_infer(const it_graph *g, const it_layer_desc *layers, int32_t n_layers, const void *x,
                   void *out, void *workspace, size_t workspace_bytes, void *stream);

/*
 * it_graph_create_part — one worker's part of a vertex-partitioned graph (Section "InferTurbo on Graph Processing
 * System": vertices are partitioned over the workers together with their edges, one layer per superstep, messages
 * exchanged in between).  The part holds the in-edges of `n_vertices` local destinations as a CSR of its own
 * (indptr has n_vertices + 1 entries); source ids name rows of a table of `n_sources` rows that the caller assembles
 * (all vertices of the graph for a destination partition; the local vertices for a source partition, see
 * it_layer_gather).  Validation, borrowing and errors as it_graph_create, with 0 <= source < n_sources.
 * it_layer_forward / it_infer take such a graph only when n_sources == n_vertices; otherwise use the stage calls.
 */
it_status it_graph_create_part(int64_t n_vertices, int64_t n_sources, int64_t n_edges, const void *indptr,
                               it_itype indptr_type, const int32_t *indices, const float *edge_weights, void *stream,
                               it_graph **out);

/*
 * The three stages of one layer as calls of their own, for callers that exchange data between them: several GPUs
 * that each own a range of the vertices, or one GPU that walks over parts of a graph too large to hold at once.
 * The names follow Section "InferTurbo Abstraction": what a vertex hands to its out-edges is produced by
 * it_layer_transform (the apply_edge half of Scatter, done once per source), it_layer_gather is the Gather stage
 * (gather_nbrs + aggregate; for GAT and transform-first layers it also finishes the vertex), it_layer_update is
 * apply_node.  it_layer_forward is exactly transform, gather, update on one graph with every table in the workspace.
 *
 * it_layer_stages tells what the layer exchanges:
 *   table_dim / table_dtype  one row per SOURCE vertex that the gather reads (the layer input itself when
 *                            table_is_input = 1: then it_layer_transform has nothing to do and need not be called)
 *   score_dim                fp32 values per vertex that travel with the table (GAT: 2 * heads, source scores
 *                            then destination scores), else 0
 *   agg_dim                  entries of the aggregate row that it_layer_gather hands to it_layer_update; 0 when the
 *                            gather writes the layer output itself and there is no update call
 */
typedef struct {
  int32_t table_dim;
  it_dtype table_dtype;
  int32_t score_dim;
  int32_t table_is_input;
  int32_t agg_dim;
} it_stage_desc;
it_status it_layer_stages(const it_graph *g, const it_layer_desc *layer, it_stage_desc *out);

/*
 * it_layer_transform — per local vertex, what its out-edges will carry: h_self [n, in_dim] -> table_out [n, table_dim]
 * (and scores_out [n, score_dim]).  Terms of the layer that stay with the vertex (the self term of a transform-first
 * layer) are kept in the workspace for it_layer_gather, so the same workspace must be passed to all three calls.
 */
it_status it_layer_transform(const it_graph *g, const it_layer_desc *layer, const void *h_self, void *table_out,
                             float *scores_out, void *workspace, size_t workspace_bytes, void *stream);

/*
 * it_layer_gather — the Gather stage over the in-edges of the local destinations.  table [n_sources, table_dim] is
 * indexed by the source ids of the graph; scores [n_sources, score_dim] likewise (GAT), the destination scores of
 * local vertex v being row first_vertex + v of it.  out is the aggregate [n, agg_dim] in feat_dtype, or the layer
 * output [n, out_dim] when agg_dim = 0.
 * raw_partial = 1 (layers with agg_dim > 0 whose table is the input, no edge features): the partial-gather of
 * Section "Optimization Strategies" for a partition of the SOURCES: out is fp32 [n, agg_dim] and holds the plain
 * sum (for mean too), max or min over the edges this part has, with the identity of the reduce (0, -inf, +inf)
 * where it has none; the caller reduces the parts' results (sum / max / min) and finishes with it_aggregate_finish.
 */
it_status it_layer_gather(const it_graph *g, const it_layer_desc *layer, const void *table, const float *scores,
                          int64_t first_vertex, int32_t raw_partial, void *out, void *workspace,
                          size_t workspace_bytes, void *stream);

/* it_layer_update — apply_node: h_self [n, in_dim] and agg [n, agg_dim] -> h_out [n, out_dim]. */
it_status it_layer_update(const it_graph *g, const it_layer_desc *layer, const void *h_self, const void *agg,
                          void *h_out, void *workspace, size_t workspace_bytes, void *stream);

/*
 * it_aggregate_finish — the receiver's side of a partial-gather over source partitions: raw [n, dim] fp32 (the
 * reduced partial results) -> out [n, dim] of `dtype`, out[v, :] = raw[v, :] * scale[v], and 0 where scale[v] = 0
 * (a vertex without in-edges, whose raw row still holds the identity of the reduce).  scale: fp32 [n]; 1 / in-degree
 * for mean, 1 otherwise.
 */
it_status it_aggregate_finish(int64_t n, int32_t dim, it_dtype dtype, const float *raw, const float *scale, void *out,
                              void *stream);

/*
 * it_layer_forward_static — it_layer_forward for callers that must not allocate device
 * memory (the paper has no counterpart: its workers allocate freely on CPU hosts).
 *
 * Who needs it: code that runs where cudaMalloc is unavailable or forbidden — inside a
 * latency-critical serving loop that has frozen its memory pool, inside a host callback, or in
 * a process whose device memory is handed out entirely by another component — and that
 * therefore cannot obtain the scratch `workspace` that it_layer_forward asks for.  Here the
 * scratch is a fixed array of IT_STATIC_WORKSPACE_BYTES that is part of the library image:
 * every GPU that loads the library holds those bytes until the process exits, whether or not
 * this call is ever made, which is why the limit is modest.
 *
 * Same arguments, results and errors as it_layer_forward, minus the workspace.  A layer whose
 * scratch need (it_workspace_bytes of that one layer) exceeds IT_STATIC_WORKSPACE_BYTES is
 * rejected with IT_ERR_WORKSPACE and nothing is launched.  The call itself performs no
 * cudaMalloc / cudaFree and calls no allocating routine; for that reason it refuses to run
 * (IT_ERR_UNSUPPORTED) while it_profile_begin instrumentation is active, since that creates
 * CUDA events on demand.  (it_graph_create / it_split_hubs do allocate: build the graph
 * during set-up.)
 *
 * The first call on each device looks up the device address of the array (with that device
 * current) and caches it, and the first launch of each kernel the library holds may make the
 * CUDA runtime load that kernel, which can allocate inside the driver.  So make one call per
 * layer shape and dtype during set-up, before any stream capture; calls after that leave the
 * device's memory as they found it.
 * All calls on a device share the one array.  It keeps the previous call's contents; nothing
 * in it needs to start at zero, because every kernel writes the part it later reads.  Two
 * calls whose kernels can overlap on the GPU (different streams without an ordering between
 * them) race on the array: serialise them.
 */
#define IT_STATIC_WORKSPACE_BYTES (32u << 20)
it_status it_layer_forward_static(const it_graph *g, const it_layer_desc *layer, const void *h_in,
                                  void *h_out, void *stream);

/*
 * it_graph_check — waits for `stream` and reports whether any kernel launched for this graph
 * since the last check gave up one of its bounded device-side waits (the tensor-core apply
 * waits on hardware barriers with an iteration limit instead of spinning for ever).
 * Returns IT_ERR_TIMEOUT in that case (and clears the condition): outputs written since the
 * last check are then not valid.  IT_OK otherwise.  No counterpart in the paper.
 */
it_status it_graph_check(it_graph *g, void *stream);

/*
 * it_debug_expire_wait — test hook for those bounded waits (no counterpart in the paper): launches the tensor-core
 * apply on a 128 x 64 operand of `dtype` with its copy producer switched off and a wait limit of a few thousand polls, so
 * that every wait inside the kernel runs out.  The kernel must then drain and return by itself; afterwards
 * it_graph_check reports IT_ERR_TIMEOUT once, and the library goes on working.  x: device [128, 64];
 * out: device [128, 64] (left undefined); workspace: device, 256-byte aligned, at least 64 KB.
 */
it_status it_debug_expire_wait(it_graph *g, it_dtype dtype, const void *x, void *out, void *workspace, size_t workspace_bytes,
                               void *stream);
/* The same hook for the kernel that it_infer uses where the update of one layer and the transform of the next run as one
 * (two products back to back, bf16): x and out are device [128, 64] bf16. */
it_status it_debug_expire_wait_fused(it_graph *g, const void *x, void *out, void *workspace, size_t workspace_bytes, void *stream);

/* Frees the library-owned arrays of the graph.  NULL is accepted. */
it_status it_graph_destroy(it_graph *g);

const char *it_status_string(it_status s);
const char *it_last_error_message(void);

/*
 * Instrumentation (no counterpart in the paper, which reports per-instance latency and IO
 * bytes of its cluster workers; this is the per-kernel equivalent).  Between it_profile_begin
 * and it_profile_end every kernel the library launches is bracketed by CUDA events on its
 * own stream.  it_profile_end waits for those events and returns, per kernel kind, the number
 * of launches, the summed device time, and the summed ALGORITHMIC bytes and flops of those
 * launches (what the method must move / compute: per edge one index, one optional weight and
 * one source row; per row its bounds and one output row; for the dense transform its operands
 * once and 2*M*K*N flops).  `stats` is a HOST array of `capacity` entries; *n_stats receives
 * the number of kinds seen.  it_kernel_launch_count: kernels launched by this process so far.
 */
typedef struct {
  char name[32];
  int64_t launches;
  double total_ms, algo_bytes, algo_flops;
} it_kernel_stat;
it_status it_profile_begin(void);
it_status it_profile_end(it_kernel_stat *stats, int32_t capacity, int32_t *n_stats);
int64_t it_kernel_launch_count(void);

#ifdef __cplusplus
}
#endif
#endif /* INFERTURBO_H */
