// it_layer_forward / it_infer / it_workspace_bytes: argument checks, workspace carving and the
// launch sequence of one layer.  All arithmetic lives in the kernels of the other files.
#include <mutex>

#include "common.cuh"

namespace {

enum LayerPlan { PLAN_SAGE = 0, PLAN_SAGE_REORDER = 1, PLAN_GAT = 2, PLAN_DENSE = 3, PLAN_GCN = 4, PLAN_GCN_REORDER = 5,
                 PLAN_MSG = 6 /* learned messages, GraphSAGE or GCN update */ };

struct LayerWs {
  LayerPlan plan;
  size_t off_counters;                              // IT_MAX_BUCKETS words from which the gather's warps claim their batches
  size_t off_B, off_partials, off_a, off_b, off_q;  // a: aggregate A | self term S | scores ; b: Z | P ; q: per-edge part Q / messages
  size_t bytes;
};

bool is_pooling(it_gather_op op) { return op == IT_GATHER_SUM || op == IT_GATHER_MEAN || op == IT_GATHER_MAX || op == IT_GATHER_MIN; }

it_status check_layer(const it_graph *g, const it_layer_desc *L) {
  IT_REQUIRE(L != nullptr, IT_ERR_INVALID_ARG, "layer is NULL");
  IT_REQUIRE(L->op >= IT_GATHER_SUM && L->op <= IT_GATHER_GCN, IT_ERR_INVALID_ARG, "bad gather op %d", (int)L->op);
  IT_REQUIRE(L->act >= IT_ACT_NONE && L->act <= IT_ACT_ELU, IT_ERR_INVALID_ARG, "bad activation %d", (int)L->act);
  IT_REQUIRE(L->feat_dtype == IT_F32 || L->feat_dtype == IT_BF16, IT_ERR_INVALID_ARG, "bad feat_dtype");
  IT_REQUIRE(L->weight_dtype == L->feat_dtype, IT_ERR_UNSUPPORTED, "weight_dtype must equal feat_dtype");
  IT_REQUIRE(L->in_dim > 0 && L->out_dim > 0, IT_ERR_INVALID_ARG, "dims must be positive");
  const int s = it_dtype_size(L->feat_dtype);
  IT_REQUIRE((L->in_dim * s) % 16 == 0 && (L->out_dim * s) % 16 == 0, IT_ERR_INVALID_ARG,
             "feature rows must be a multiple of 16 bytes (in %d, out %d, %d-byte elements)", L->in_dim, L->out_dim, s);
  if (L->op == IT_GATHER_GAT) {
    IT_REQUIRE(L->heads >= 1 && L->out_dim % L->heads == 0, IT_ERR_INVALID_ARG, "out_dim must be heads * head_dim");
    IT_REQUIRE(!L->use_edge_weights, IT_ERR_UNSUPPORTED, "GAT layers take no edge weights");
  } else {
    IT_REQUIRE(L->heads <= 1, IT_ERR_INVALID_ARG, "heads > 1 needs op = IT_GATHER_GAT");
    IT_REQUIRE(!L->use_edge_weights || g->edge_weights, IT_ERR_INVALID_ARG, "layer uses edge weights but the graph has none");
    IT_REQUIRE(L->op != IT_GATHER_NONE || !L->use_edge_weights, IT_ERR_INVALID_ARG, "a dense layer has no edges to weight");
  }
  IT_REQUIRE(L->edge_dim >= 0, IT_ERR_INVALID_ARG, "edge_dim is negative");
  if (L->edge_dim > 0) {
    IT_REQUIRE(L->op != IT_GATHER_NONE, IT_ERR_UNSUPPORTED, "a dense layer has no edges whose features it could take");
    IT_REQUIRE(g->edge_feat != nullptr, IT_ERR_INVALID_ARG, "layer uses edge features but the graph has none (it_graph_set_edge_features)");
    IT_REQUIRE(g->edge_dim == L->edge_dim && g->edge_dtype == L->feat_dtype, IT_ERR_INVALID_ARG,
               "layer expects edge features [%d] of its feat_dtype, the graph holds [%d]", L->edge_dim, g->edge_dim);
  }
  // rows that lie in edge order are addressed by a 32-bit edge id
  IT_REQUIRE((L->edge_dim == 0 && L->msg_dim == 0) || g->e <= (int64_t)INT32_MAX, IT_ERR_UNSUPPORTED,
             "layers with edge features or learned messages take graphs of at most 2^31 - 1 edges");
  IT_REQUIRE(L->msg_dim >= 0, IT_ERR_INVALID_ARG, "msg_dim is negative");
  if (L->msg_dim > 0) {
    IT_REQUIRE(is_pooling(L->op) || L->op == IT_GATHER_GCN, IT_ERR_UNSUPPORTED, "learned messages are taken by the pooling layers and GCN only");
    IT_REQUIRE((L->msg_dim * s) % 16 == 0, IT_ERR_INVALID_ARG, "a message row must be a multiple of 16 bytes (msg_dim %d)", L->msg_dim);
    IT_REQUIRE(L->act_edge >= IT_ACT_NONE && L->act_edge <= IT_ACT_ELU, IT_ERR_INVALID_ARG, "bad act_edge %d", (int)L->act_edge);
  }
  return IT_OK;
}

bool reorders(const it_layer_desc *L) {
  // with edge features the aggregate of the edge part would need its own transform, and a learned message is not
  // linear in the source state: such layers keep the plain order
  return L->allow_reorder && L->edge_dim == 0 && L->msg_dim == 0 &&
         (L->op == IT_GATHER_SUM || L->op == IT_GATHER_MEAN || L->op == IT_GATHER_GCN) && L->out_dim < L->in_dim;
}

LayerPlan plan_of(const it_layer_desc *L) {
  if (L->op == IT_GATHER_GAT) return PLAN_GAT;
  if (L->op == IT_GATHER_NONE) return PLAN_DENSE;
  if (L->msg_dim > 0) return PLAN_MSG;
  if (L->op == IT_GATHER_GCN) return reorders(L) ? PLAN_GCN_REORDER : PLAN_GCN;
  return reorders(L) ? PLAN_SAGE_REORDER : PLAN_SAGE;
}

// Row length of the aggregate that the gather hands to the update (0: the gather finishes the vertex itself).
int agg_dim_of(const it_layer_desc *L) {
  switch (plan_of(L)) {
    case PLAN_SAGE: case PLAN_GCN: return L->in_dim + L->edge_dim;
    case PLAN_MSG: return L->msg_dim;
    default: return 0;
  }
}

LayerWs plan_layer(const it_graph *g, const it_layer_desc *L) {
  LayerWs w;
  const size_t n = (size_t)g->n, s = (size_t)it_dtype_size(L->feat_dtype);
  const size_t fi = (size_t)L->in_dim, fo = (size_t)L->out_dim, fe = (size_t)L->edge_dim, fm = (size_t)L->msg_dim;
  const size_t kpad = 128;   // the tensor-core path pads the K of each operand to whole k-blocks (at most 63 + 63 rows)
  size_t off = 0;
  auto take = [&](size_t bytes) { size_t o = off; off += it_align_up(bytes); return o; };
  w.plan = plan_of(L);
  w.off_q = 0;
  w.off_counters = take(IT_MAX_BUCKETS * sizeof(int));
  switch (w.plan) {
    case PLAN_GAT:
      w.off_B = take((fi + kpad) * (fo + 2 * (size_t)L->heads) * 8);
      w.off_partials = take(it_gat_partial_bytes(g, L->out_dim, L->heads));
      w.off_a = take(n * 2 * (size_t)L->heads * 4);  // scores
      w.off_b = take(n * fo * s);                    // Z
      // edge features in the logits: per edge its message row and one logit term per head
      // ... or, without them, the source scores of every vertex on their own (read per edge at random: half the bytes
      // of the interleaved score rows, and small enough to stay in the L2)
      w.off_q = take(fe > 0 ? (size_t)g->e * fo * s + it_align_up((size_t)g->e * (size_t)L->heads * 4)
                            : (size_t)g->n_src * (size_t)L->heads * 4);
      break;
    case PLAN_DENSE:
      w.off_B = take((fi + kpad) * fo * 8);
      w.off_partials = w.off_a = w.off_b = off;
      break;
    case PLAN_GCN_REORDER:
      w.off_B = take((fi + fe + kpad) * fo * 8);
      w.off_partials = take((size_t)g->n_partial_rows * fo * 4);
      w.off_a = off;
      w.off_b = take(n * fo * s);  // Z
      break;
    case PLAN_GCN:
      w.off_B = take((fi + fe + kpad) * fo * 8);
      w.off_partials = take((size_t)g->n_partial_rows * (fi > fe ? fi : fe) * 4);
      w.off_a = take(n * (fi + fe) * s);  // A = [sum_e w_e h_u | sum_e e_vu]
      w.off_b = off;
      break;
    case PLAN_SAGE_REORDER:
      w.off_B = take((fi + kpad) * 2 * fo * 8);
      w.off_partials = take((size_t)g->n_partial_rows * fo * 4);
      w.off_a = take(n * fo * s);  // S (the self term, stored like the rows)
      w.off_b = take(n * fo * s);  // Z
      break;
    case PLAN_SAGE:
      w.off_B = take((2 * fi + fe + kpad) * fo * 8);
      w.off_partials = take((size_t)g->n_partial_rows * (fi > fe ? fi : fe) * 4);
      w.off_a = take(n * (fi + fe) * s);  // A = [aggregate of w_e h_u | aggregate of e_vu]
      w.off_b = off;
      break;
    case PLAN_MSG: {
      // the largest of the three weight matrices prepared in turn: W_edge[:in] (in x msg), W_edge[in:] (edge x msg), W ((in + msg) x out)
      size_t wb = (fi + kpad) * fm;
      if ((fe + kpad) * fm > wb) wb = (fe + kpad) * fm;
      if ((fi + fm + 2 * kpad) * fo > wb) wb = (fi + fm + 2 * kpad) * fo;
      w.off_B = take(wb * 8);
      w.off_partials = take((size_t)g->n_partial_rows * fm * 4);
      w.off_a = take(n * fm * s);                            // A: aggregate of the messages
      w.off_b = take(n * fm * s);                            // P: source part of the message, one row per vertex
      w.off_q = take(fe > 0 ? (size_t)g->e * fm * s : 0);    // Q, then the messages in place: one row per edge
      break;
    }
  }
  w.bytes = off;
  return w;
}

// The dense transform of a layer: on the tensor cores when the shape allows it, otherwise the
// fp32 CUDA-core kernel.  `ga` is filled for the CUDA-core kernel (for GAT: NB includes the
// 2*heads score columns and out2 = scores); the tensor-core kernel derives its own view.
it_status run_apply(const it_graph *g, const it_layer_desc *L, it_prep_kind kind, it_gemm_args ga, float *B,
                    float *scores, cudaStream_t st) {
  const int K = ga.K1 + (ga.X2 ? ga.K2 : 0);
  const bool want_scores = kind == IT_PREP_GAT;
  const int heads = L->heads > 0 ? L->heads : 1, hd = L->out_dim / heads;
  if (it_tc_supported(ga, heads, hd, want_scores)) {
    IT_TRY(it_launch_prep_weights_tc(kind, L, ga.n0 + ga.n1, ga.K1, ga.X2 ? ga.K2 : 0, B, st));
    return it_launch_gemm_tc(ga, B, L->att_src, L->att_dst, heads, hd, want_scores ? scores : nullptr, g->num_sms,
                             g->d_status, st);
  }
  ga.B = B;
  IT_TRY(it_launch_prep_weights(kind, L, K, B, st));
  return it_launch_gemm(ga, st);
}

// out [M, n_out] = act(X [M, K] * W [K, n_out] + bias): one plain dense product with W taken as it is.
it_status run_dense(const it_graph *g, const it_layer_desc *L, int64_t M, const void *X, int K, const void *W, int n_out,
                    const float *bias, it_act act, void *out, float *B, cudaStream_t st) {
  it_layer_desc d = *L;   // a view of the layer that names this product's weights
  d.op = IT_GATHER_NONE; d.in_dim = K; d.out_dim = n_out; d.W = W; d.heads = 1; d.edge_dim = 0; d.msg_dim = 0;
  it_gemm_args ga{};
  ga.M = M; ga.x_dtype = L->feat_dtype; ga.X1 = X; ga.K1 = K; ga.X2 = nullptr; ga.K2 = 0;
  ga.B = B; ga.NB = n_out;
  ga.n0 = n_out; ga.out0 = out; ga.dt0 = L->feat_dtype; ga.bias0 = bias; ga.act0 = act;
  ga.n1 = 0; ga.out1 = nullptr; ga.dt1 = L->feat_dtype; ga.out2 = nullptr;
  return run_apply(g, &d, IT_PREP_DENSE, ga, B, nullptr, st);
}

// The edge-feature half of the message [w_e h_u | e_vu]: the same reduce over the rows of the edge-feature
// matrix, which lie in edge order, written to columns [in_dim, in_dim + edge_dim) of the aggregate.
it_status gather_edge_part(it_gather_args gg, const it_layer_desc *L, void *A, int a_ld, cudaStream_t st) {
  if (L->edge_dim == 0) return IT_OK;
  gg.src = gg.g->edge_feat; gg.src_ld = 0; gg.per_edge_rows = 1; gg.use_edge_weights = 0; gg.dim = L->edge_dim;
  gg.dst = (char *)A + (size_t)L->in_dim * it_dtype_size(gg.dtype); gg.dst_ld = a_ld;
  return it_launch_gather(gg, st);
}

struct StageCtx {
  const it_graph *g;
  const it_layer_desc *L;
  LayerWs w;
  char *ws;
  float *B, *partials;
  cudaStream_t st;
};

it_status stage_ctx(const it_graph *g, const it_layer_desc *L, void *ws, size_t ws_bytes, cudaStream_t st, StageCtx *c) {
  c->g = g; c->L = L; c->w = plan_layer(g, L); c->ws = (char *)ws; c->st = st;
  IT_REQUIRE(ws_bytes >= c->w.bytes, IT_ERR_WORKSPACE, "workspace has %zu bytes, layer needs %zu", ws_bytes, c->w.bytes);
  IT_REQUIRE(L->W != nullptr, IT_ERR_INVALID_ARG, "W is NULL");
  c->B = reinterpret_cast<float *>(c->ws + c->w.off_B);
  c->partials = g->n_partial_rows > 0 ? reinterpret_cast<float *>(c->ws + c->w.off_partials) : nullptr;
  return IT_OK;
}

// ---- stage 1: what the out-edges of every local vertex carry (nothing to do when the table is the input itself)
it_status stage_transform(const StageCtx &c, const void *h_self, void *table_out, float *scores_out) {
  const it_graph *g = c.g;
  const it_layer_desc *L = c.L;
  const it_dtype dt = L->feat_dtype;
  it_gemm_args ga{};
  ga.M = g->n; ga.x_dtype = dt; ga.X1 = h_self; ga.K1 = L->in_dim; ga.X2 = nullptr; ga.K2 = 0; ga.B = c.B;
  switch (c.w.plan) {
    case PLAN_GAT:
      IT_REQUIRE(L->att_src && L->att_dst, IT_ERR_INVALID_ARG, "GAT layer needs att_src and att_dst");
      ga.NB = L->out_dim + 2 * L->heads;
      ga.n0 = 0; ga.out0 = nullptr; ga.dt0 = dt; ga.bias0 = nullptr; ga.act0 = IT_ACT_NONE;
      ga.n1 = L->out_dim; ga.out1 = table_out; ga.dt1 = dt; ga.out2 = scores_out;
      return run_apply(g, L, IT_PREP_GAT, ga, c.B, scores_out, c.st);
    case PLAN_GCN_REORDER:   // Z = H W
      ga.NB = L->out_dim;
      ga.n0 = 0; ga.out0 = nullptr; ga.dt0 = dt; ga.bias0 = nullptr; ga.act0 = IT_ACT_NONE;
      ga.n1 = L->out_dim; ga.out1 = table_out; ga.dt1 = dt; ga.out2 = nullptr;
      return run_apply(g, L, IT_PREP_DENSE, ga, c.B, nullptr, c.st);
    case PLAN_SAGE_REORDER:  // S = H W_self + b (stays with the vertex), Z = H W_neigh
      ga.NB = 2 * L->out_dim;
      ga.n0 = L->out_dim; ga.out0 = c.ws + c.w.off_a; ga.dt0 = dt; ga.bias0 = L->bias; ga.act0 = IT_ACT_NONE;
      ga.n1 = L->out_dim; ga.out1 = table_out; ga.dt1 = dt; ga.out2 = nullptr;
      return run_apply(g, L, IT_PREP_SAGE_REORDER, ga, c.B, nullptr, c.st);
    case PLAN_MSG:
      IT_REQUIRE(L->W_edge != nullptr, IT_ERR_INVALID_ARG, "W_edge is NULL");
      // the source part of the message, once per vertex; without edge features that is the whole message
      if (L->edge_dim == 0)
        return run_dense(g, L, g->n, h_self, L->in_dim, L->W_edge, L->msg_dim, L->bias_edge, L->act_edge, table_out, c.B, c.st);
      return run_dense(g, L, g->n, h_self, L->in_dim, L->W_edge, L->msg_dim, nullptr, IT_ACT_NONE, table_out, c.B, c.st);
    default:
      return IT_OK;
  }
}

// ---- stage 2: the Gather stage.  out: the aggregate [n, agg_dim] (plans with an update), else the layer output.
// `self_term`: where a transform-first GraphSAGE layer finds S (NULL: its place in the workspace, where stage_transform puts it).
it_status stage_gather(const StageCtx &c, const void *table, const float *scores, const float *scores_dst, bool raw, void *out,
                       const void *self_term = nullptr) {
  const it_graph *g = c.g;
  const it_layer_desc *L = c.L;
  const it_dtype dt = L->feat_dtype;
  if (c.w.plan == PLAN_DENSE) return IT_OK;
  if (c.w.plan == PLAN_GAT) {
    it_gat_args aa{};
    aa.g = g; aa.dtype = dt; aa.heads = L->heads; aa.head_dim = L->out_dim / L->heads; aa.z = table; aa.scores = scores;
    aa.scores_dst = scores_dst; aa.partials = c.partials; aa.counters = reinterpret_cast<int *>(c.ws + c.w.off_counters);
    aa.slope = L->leaky_slope; aa.bias = L->bias; aa.act = L->act; aa.dst = out;
    if (L->edge_dim > 0) {
      IT_REQUIRE(L->att_edge != nullptr, IT_ERR_INVALID_ARG, "GAT layer with edge features needs att_edge");
      void *Zj = c.ws + c.w.off_q;
      float *sc = reinterpret_cast<float *>(c.ws + c.w.off_q + it_align_up((size_t)g->e * (size_t)L->out_dim * (size_t)it_dtype_size(dt)));
      IT_TRY(it_launch_gat_edge_rows(g, dt, L->out_dim, L->heads, table, scores, L->att_edge, Zj, sc, c.st));
      aa.z = Zj; aa.per_edge_rows = 1; aa.src_scores = sc;
    } else {
      float *dense = reinterpret_cast<float *>(c.ws + c.w.off_q);
      IT_TRY(it_launch_compact_scores(g->n_src, L->heads, scores, dense, c.st));
      aa.src_scores = dense;
    }
    return it_launch_gat(aa, c.st);
  }
  it_gather_args gg{};
  gg.g = g; gg.op = L->op == IT_GATHER_GCN ? IT_GATHER_SUM : L->op; gg.use_edge_weights = L->use_edge_weights; gg.dtype = dt;
  gg.partials = c.partials; gg.counters = reinterpret_cast<int *>(c.ws + c.w.off_counters);
  switch (c.w.plan) {
    case PLAN_GCN_REORDER:   // h' = act(sum_e w_e z_u + b) in the gather's epilogue
      gg.dim = L->out_dim; gg.src = table; gg.dst = out; gg.epi = IT_EPI_BIAS_ACT; gg.self_term = nullptr; gg.bias = L->bias; gg.act = L->act;
      return it_launch_gather(gg, c.st);
    case PLAN_SAGE_REORDER:
      gg.dim = L->out_dim; gg.src = table; gg.dst = out; gg.epi = IT_EPI_ADD_ACT;
      gg.self_term = self_term ? self_term : c.ws + c.w.off_a; gg.self_dtype = dt; gg.act = L->act;
      return it_launch_gather(gg, c.st);
    case PLAN_MSG:
      gg.dim = L->msg_dim; gg.dst = out; gg.dst_ld = L->msg_dim; gg.epi = IT_EPI_STORE; gg.act = IT_ACT_NONE;
      if (L->edge_dim == 0) {   // the table holds the finished per-source message: a plain gather of it
        gg.src = table;
        return it_launch_gather(gg, c.st);
      } else {
        // the edge part Q = e W_edge[in:] + b_edge, once per edge; then m_j = act_edge(P[u_j] + Q[j]) in place; then the
        // reduce over the message rows, which lie in edge order
        void *Q = c.ws + c.w.off_q;
        const size_t es = (size_t)it_dtype_size(dt);
        const char *W_edge_part = (const char *)L->W_edge + (size_t)L->in_dim * L->msg_dim * es;
        IT_TRY(run_dense(g, L, g->e, g->edge_feat, L->edge_dim, W_edge_part, L->msg_dim, L->bias_edge, IT_ACT_NONE, Q, c.B, c.st));
        IT_TRY(it_launch_edge_messages(g, dt, L->msg_dim, table, Q, L->act_edge, c.st));
        gg.src = Q; gg.src_ld = 0; gg.per_edge_rows = 1;
        return it_launch_gather(gg, c.st);
      }
    default: {  // PLAN_SAGE, PLAN_GCN: A = aggregate of [w_e h_u | e_vu]
      const int a_ld = L->in_dim + L->edge_dim;   // row length of the aggregate handed to the update
      gg.dim = L->in_dim; gg.src = table; gg.dst = out; gg.dst_ld = a_ld; gg.epi = raw ? IT_EPI_RAW_F32 : IT_EPI_STORE;
      gg.self_term = nullptr; gg.bias = nullptr; gg.act = IT_ACT_NONE;
      IT_TRY(it_launch_gather(gg, c.st));
      return gather_edge_part(gg, L, out, a_ld, c.st);
    }
  }
}

// ---- stage 3: apply_node on the aggregate
it_status stage_update(const StageCtx &c, const void *h_self, const void *agg, void *h_out) {
  const it_graph *g = c.g;
  const it_layer_desc *L = c.L;
  const it_dtype dt = L->feat_dtype;
  const int a_ld = agg_dim_of(L);
  it_gemm_args ga{};
  ga.M = g->n; ga.x_dtype = dt; ga.B = c.B; ga.NB = L->out_dim;
  ga.n0 = L->out_dim; ga.out0 = h_out; ga.dt0 = dt; ga.bias0 = L->bias; ga.act0 = L->act;
  ga.n1 = 0; ga.out1 = nullptr; ga.dt1 = dt; ga.out2 = nullptr;
  switch (c.w.plan) {
    case PLAN_DENSE:   // no Gather stage: h' = act(h W + b)
      ga.X1 = h_self; ga.K1 = L->in_dim; ga.X2 = nullptr; ga.K2 = 0;
      return run_apply(g, L, IT_PREP_DENSE, ga, c.B, nullptr, c.st);
    case PLAN_GCN:     // h' = act(A W + b)
      ga.X1 = agg; ga.K1 = a_ld; ga.X2 = nullptr; ga.K2 = 0;
      return run_apply(g, L, IT_PREP_DENSE, ga, c.B, nullptr, c.st);
    case PLAN_SAGE:    // h' = act([h | A] W + b)
      ga.X1 = h_self; ga.K1 = L->in_dim; ga.X2 = agg; ga.K2 = a_ld;
      return run_apply(g, L, IT_PREP_SAGE, ga, c.B, nullptr, c.st);
    case PLAN_MSG:
      if (L->op == IT_GATHER_GCN) { ga.X1 = agg; ga.K1 = a_ld; ga.X2 = nullptr; ga.K2 = 0; }
      else { ga.X1 = h_self; ga.K1 = L->in_dim; ga.X2 = agg; ga.K2 = a_ld; }
      return run_apply(g, L, IT_PREP_DENSE, ga, c.B, nullptr, c.st);   // W [K1 + K2, out] taken as it is
    default:
      return IT_OK;
  }
}

it_status layer_forward_impl(const it_graph *g, const it_layer_desc *L, const void *h_in, void *h_out, char *ws,
                             size_t ws_bytes, cudaStream_t st) {
  IT_REQUIRE(g->n_src == g->n, IT_ERR_INVALID_ARG,
             "the graph is one part of a partition (%lld sources, %lld vertices): use it_layer_transform / it_layer_gather / it_layer_update",
             (long long)g->n_src, (long long)g->n);
  StageCtx c;
  IT_TRY(stage_ctx(g, L, ws, ws_bytes, st, &c));
  const int a_dim = agg_dim_of(L);
  const LayerPlan plan = c.w.plan;
  const bool table_is_input = plan == PLAN_SAGE || plan == PLAN_GCN || plan == PLAN_DENSE;
  // every table lives in the workspace: Z / P at off_b, scores / aggregate at off_a
  void *table = table_is_input ? const_cast<void *>(h_in) : (void *)(ws + c.w.off_b);
  float *scores = plan == PLAN_GAT ? reinterpret_cast<float *>(ws + c.w.off_a) : nullptr;
  IT_TRY(stage_transform(c, h_in, table, scores));
  void *agg = a_dim > 0 ? (void *)(ws + c.w.off_a) : h_out;
  IT_TRY(stage_gather(c, table, scores, scores, false, agg));
  return stage_update(c, h_in, agg, h_out);
}

// ---- the update of layer a and the transform of layer b = a + 1 as one kernel
// When layer b transforms before it aggregates, the output H of layer a is read by that transform and by nothing
// else, so the two dense products run back to back in one kernel that keeps each tile of H on the SM (rounded to the
// storage type exactly as it would have been stored): H is neither written nor read back.  Taken for bf16 layers
// whose shapes fit the kernel; everything else runs layer by layer.
#ifndef IT_FUSE_UPDATE_TRANSFORM
#define IT_FUSE_UPDATE_TRANSFORM 1
#endif

struct FusedPair {
  it_gemm2_args ga;        // pointers filled in by the caller
  it_prep_kind kind_a, kind_b;
  int nb_b;                // columns of layer b's prepared weights
  size_t s_bytes;          // bytes of S in front of Z in the buffer that would have held H (0: layer b keeps no self term)
};

bool fused_pair(const it_graph *g, const it_layer_desc *A, const it_layer_desc *Bn, FusedPair *out) {
  if (!IT_FUSE_UPDATE_TRANSFORM || g->n_src != g->n) return false;
  if (A->feat_dtype != IT_BF16 || Bn->feat_dtype != IT_BF16) return false;
  const LayerPlan pa = plan_of(A), pb = plan_of(Bn);
  if (pa != PLAN_SAGE && pa != PLAN_GCN && pa != PLAN_DENSE) return false;
  if (pb != PLAN_SAGE_REORDER && pb != PLAN_GCN_REORDER) return false;
  FusedPair f{};
  f.ga.M = g->n;
  const int a_ld = agg_dim_of(A);
  if (pa == PLAN_SAGE) { f.ga.K1 = A->in_dim; f.ga.K2 = a_ld; f.kind_a = IT_PREP_SAGE; }
  else if (pa == PLAN_GCN) { f.ga.K1 = a_ld; f.ga.K2 = 0; f.kind_a = IT_PREP_DENSE; }
  else { f.ga.K1 = A->in_dim; f.ga.K2 = 0; f.kind_a = IT_PREP_DENSE; }
  f.ga.N1 = A->out_dim; f.ga.bias1 = A->bias; f.ga.act1 = A->act;
  if (pb == PLAN_SAGE_REORDER) { f.ga.n0 = Bn->out_dim; f.ga.bias0 = Bn->bias; f.ga.n1 = Bn->out_dim; f.kind_b = IT_PREP_SAGE_REORDER; }
  else { f.ga.n0 = 0; f.ga.bias0 = nullptr; f.ga.n1 = Bn->out_dim; f.kind_b = IT_PREP_DENSE; }
  f.nb_b = f.ga.n0 + f.ga.n1;
  f.s_bytes = it_align_up((size_t)g->n * (size_t)f.ga.n0 * 2);
  // S and Z take the place of H, so together they must not be larger (alignment padding of S included)
  if (f.s_bytes + (size_t)g->n * (size_t)f.ga.n1 * 2 > it_align_up((size_t)g->n * (size_t)A->out_dim * 2)) return false;
  // probe the shape with placeholder pointers (X2 only says whether there is a second operand)
  it_gemm2_args probe = f.ga;
  probe.X1 = g; probe.X2 = f.ga.K2 > 0 ? (const void *)g : nullptr;
  if (!it_tc2_supported(probe)) return false;
  *out = f;
  return true;
}

struct InferWs { size_t layer_bytes, buf_bytes, off_buf0, off_buf1, off_B2, bytes; };

it_status plan_infer(const it_graph *g, const it_layer_desc *layers, int32_t n_layers, InferWs *out) {
  IT_REQUIRE(g != nullptr, IT_ERR_INVALID_ARG, "graph is NULL");
  IT_REQUIRE(layers != nullptr && n_layers >= 1, IT_ERR_INVALID_ARG, "need at least one layer");
  InferWs w{0, 0, 0, 0, 0, 0};
  size_t b2_bytes = 0;   // prepared weights of a layer whose transform runs fused with the previous layer's update
  for (int i = 0; i < n_layers; ++i) {
    IT_TRY(check_layer(g, &layers[i]));
    if (i > 0) {
      IT_REQUIRE(layers[i].in_dim == layers[i - 1].out_dim, IT_ERR_INVALID_ARG, "layer %d in_dim %d != layer %d out_dim %d", i,
                 layers[i].in_dim, i - 1, layers[i - 1].out_dim);
      IT_REQUIRE(layers[i].feat_dtype == layers[0].feat_dtype, IT_ERR_INVALID_ARG, "all layers must share feat_dtype");
    }
    size_t b = plan_layer(g, &layers[i]).bytes;
    if (b > w.layer_bytes) w.layer_bytes = b;
    if (i < n_layers - 1) {
      size_t hb = it_align_up((size_t)g->n * (size_t)layers[i].out_dim * (size_t)it_dtype_size(layers[i].feat_dtype));
      if (hb > w.buf_bytes) w.buf_bytes = hb;
    }
    if (i > 0) {
      const size_t wb = it_align_up(((size_t)layers[i].in_dim + 128) * 2 * (size_t)layers[i].out_dim * 8);
      if (wb > b2_bytes) b2_bytes = wb;
    }
  }
  w.off_buf0 = w.layer_bytes;
  w.off_buf1 = w.off_buf0 + (n_layers >= 2 ? w.buf_bytes : 0);
  w.off_B2 = w.off_buf1 + (n_layers >= 3 ? w.buf_bytes : 0);
  w.bytes = w.off_B2 + b2_bytes;
  *out = w;
  return IT_OK;
}

bool overlaps(const void *a, size_t na, const void *b, size_t nb) {
  const char *x = (const char *)a, *y = (const char *)b;
  return x < y + nb && y < x + na;
}

bool aligned16(const void *p) { return ((uintptr_t)p % 16) == 0; }

// What every forward call checks about the graph and its input / output matrices before anything is launched:
// the kernels move 16-byte slices of the rows, so a pointer that is not 16-byte aligned would fault on the device.
it_status check_io(const it_graph *g, const void *in, size_t in_bytes, const void *out, size_t out_bytes) {
  IT_REQUIRE(g->n == 0 || g->bucket_meta != nullptr, IT_ERR_BAD_GRAPH,
             "the graph has no row split (an it_split_hubs call failed): call it_split_hubs again before a forward pass");
  if (g->n == 0) return IT_OK;
  IT_REQUIRE(in != nullptr && out != nullptr, IT_ERR_INVALID_ARG, "input / output matrix is NULL");
  IT_REQUIRE(aligned16(in) && aligned16(out), IT_ERR_INVALID_ARG,
             "input and output matrices must be 16-byte aligned (got %p, %p)", in, out);
  IT_REQUIRE(!overlaps(in, in_bytes, out, out_bytes), IT_ERR_INVALID_ARG, "input and output matrices overlap");
  return IT_OK;
}

// Common checks of the stage calls.
it_status check_stage(const it_graph *g, const it_layer_desc *layer, void *workspace) {
  IT_REQUIRE(g != nullptr, IT_ERR_INVALID_ARG, "graph is NULL");
  IT_TRY(check_layer(g, layer));
  IT_REQUIRE(g->n == 0 || g->bucket_meta != nullptr, IT_ERR_BAD_GRAPH,
             "the graph has no row split (an it_split_hubs call failed): call it_split_hubs again before a forward pass");
  IT_REQUIRE(workspace != nullptr && ((uintptr_t)workspace % 256) == 0, IT_ERR_WORKSPACE, "workspace is NULL or not 256-byte aligned");
  return IT_OK;
}

}  // namespace

extern "C" it_status it_layer_stages(const it_graph *g, const it_layer_desc *layer, it_stage_desc *out) {
  IT_REQUIRE(g != nullptr && out != nullptr, IT_ERR_INVALID_ARG, "NULL argument");
  IT_TRY(check_layer(g, layer));
  const LayerPlan plan = plan_of(layer);
  out->table_dtype = layer->feat_dtype;
  out->score_dim = plan == PLAN_GAT ? 2 * layer->heads : 0;
  out->table_is_input = (plan == PLAN_SAGE || plan == PLAN_GCN || plan == PLAN_DENSE) ? 1 : 0;
  out->agg_dim = agg_dim_of(layer);
  out->table_dim = plan == PLAN_DENSE ? 0 : (out->table_is_input ? layer->in_dim : (plan == PLAN_MSG ? layer->msg_dim : layer->out_dim));
  return IT_OK;
}

extern "C" it_status it_layer_transform(const it_graph *g, const it_layer_desc *layer, const void *h_self, void *table_out,
                                        float *scores_out, void *workspace, size_t workspace_bytes, void *stream) {
  IT_TRY(check_stage(g, layer, workspace));
  if (g->n == 0) return IT_OK;
  const LayerPlan plan = plan_of(layer);
  if (plan == PLAN_SAGE || plan == PLAN_GCN || plan == PLAN_DENSE) return IT_OK;   // the table is the layer input itself
  IT_REQUIRE(h_self != nullptr && table_out != nullptr && aligned16(h_self) && aligned16(table_out), IT_ERR_INVALID_ARG,
             "h_self / table_out is NULL or not 16-byte aligned");
  IT_REQUIRE(plan != PLAN_GAT || (scores_out != nullptr && aligned16(scores_out)), IT_ERR_INVALID_ARG, "scores_out is NULL or not 16-byte aligned");
  StageCtx c;
  IT_TRY(stage_ctx(g, layer, workspace, workspace_bytes, (cudaStream_t)stream, &c));
  return stage_transform(c, h_self, table_out, scores_out);
}

extern "C" it_status it_layer_gather(const it_graph *g, const it_layer_desc *layer, const void *table, const float *scores,
                                     int64_t first_vertex, int32_t raw_partial, void *out, void *workspace,
                                     size_t workspace_bytes, void *stream) {
  IT_TRY(check_stage(g, layer, workspace));
  if (g->n == 0) return IT_OK;
  const LayerPlan plan = plan_of(layer);
  if (plan == PLAN_DENSE) return IT_OK;
  IT_REQUIRE(table != nullptr && out != nullptr && aligned16(table) && aligned16(out), IT_ERR_INVALID_ARG, "table / out is NULL or not 16-byte aligned");
  IT_REQUIRE(first_vertex >= 0 && first_vertex + g->n <= g->n_src || plan != PLAN_GAT, IT_ERR_INVALID_ARG,
             "first_vertex %lld + %lld local vertices exceeds the %lld rows of the score table", (long long)first_vertex, (long long)g->n, (long long)g->n_src);
  IT_REQUIRE(plan != PLAN_GAT || (scores != nullptr && aligned16(scores)), IT_ERR_INVALID_ARG, "scores is NULL or not 16-byte aligned");
  IT_REQUIRE(!raw_partial || ((plan == PLAN_SAGE || plan == PLAN_GCN) && layer->edge_dim == 0), IT_ERR_UNSUPPORTED,
             "raw partial results are produced by pooling / GCN layers that gather their input and carry no edge features");
  StageCtx c;
  IT_TRY(stage_ctx(g, layer, workspace, workspace_bytes, (cudaStream_t)stream, &c));
  const float *scores_dst = scores ? scores + (size_t)first_vertex * 2 * (size_t)layer->heads : nullptr;
  return stage_gather(c, table, scores, scores_dst, raw_partial != 0, out);
}

extern "C" it_status it_layer_update(const it_graph *g, const it_layer_desc *layer, const void *h_self, const void *agg,
                                     void *h_out, void *workspace, size_t workspace_bytes, void *stream) {
  IT_TRY(check_stage(g, layer, workspace));
  if (g->n == 0) return IT_OK;
  const int a_dim = agg_dim_of(layer);
  const LayerPlan plan = plan_of(layer);
  if (a_dim == 0 && plan != PLAN_DENSE) return IT_OK;   // the gather has written the layer output
  IT_REQUIRE(h_out != nullptr && aligned16(h_out), IT_ERR_INVALID_ARG, "h_out is NULL or not 16-byte aligned");
  const bool needs_self = plan == PLAN_DENSE || plan == PLAN_SAGE || (plan == PLAN_MSG && layer->op != IT_GATHER_GCN);
  IT_REQUIRE(!needs_self || (h_self != nullptr && aligned16(h_self)), IT_ERR_INVALID_ARG, "h_self is NULL or not 16-byte aligned");
  IT_REQUIRE(a_dim == 0 || (agg != nullptr && aligned16(agg)), IT_ERR_INVALID_ARG, "agg is NULL or not 16-byte aligned");
  StageCtx c;
  IT_TRY(stage_ctx(g, layer, workspace, workspace_bytes, (cudaStream_t)stream, &c));
  return stage_update(c, h_self, agg, h_out);
}

extern "C" it_status it_aggregate_finish(int64_t n, int32_t dim, it_dtype dtype, const float *raw, const float *scale, void *out,
                                         void *stream) {
  IT_REQUIRE(n >= 0 && dim > 0, IT_ERR_INVALID_ARG, "bad shape");
  IT_REQUIRE(dtype == IT_F32 || dtype == IT_BF16, IT_ERR_INVALID_ARG, "bad dtype");
  if (n == 0) return IT_OK;
  IT_REQUIRE(raw && scale && out && aligned16(raw) && aligned16(out), IT_ERR_INVALID_ARG, "raw / scale / out is NULL or not 16-byte aligned");
  return it_launch_aggregate_finish(n, dim, dtype, raw, scale, out, (cudaStream_t)stream);
}

extern "C" it_status it_workspace_bytes(const it_graph *g, const it_layer_desc *layers, int32_t n_layers,
                                        size_t *out_bytes) {
  IT_REQUIRE(out_bytes != nullptr, IT_ERR_INVALID_ARG, "out_bytes is NULL");
  InferWs w;
  IT_TRY(plan_infer(g, layers, n_layers, &w));
  *out_bytes = w.bytes > 0 ? w.bytes : 256;
  return IT_OK;
}

extern "C" it_status it_layer_forward(const it_graph *g, const it_layer_desc *layer, const void *h_in, void *h_out,
                                      void *workspace, size_t workspace_bytes, void *stream) {
  IT_REQUIRE(g != nullptr, IT_ERR_INVALID_ARG, "graph is NULL");
  IT_TRY(check_layer(g, layer));
  IT_REQUIRE(workspace != nullptr && ((uintptr_t)workspace % 256) == 0, IT_ERR_WORKSPACE, "workspace is NULL or not 256-byte aligned");
  const size_t s = (size_t)it_dtype_size(layer->feat_dtype);
  const size_t in_bytes = (size_t)g->n * layer->in_dim * s, out_bytes = (size_t)g->n * layer->out_dim * s;
  IT_TRY(check_io(g, h_in, in_bytes, h_out, out_bytes));
  IT_REQUIRE(g->n == 0 || (!overlaps(h_in, in_bytes, workspace, workspace_bytes) && !overlaps(h_out, out_bytes, workspace, workspace_bytes)),
             IT_ERR_INVALID_ARG, "h_in / h_out overlaps the workspace");
  return layer_forward_impl(g, layer, h_in, h_out, (char *)workspace, workspace_bytes, (cudaStream_t)stream);
}

// ----------------------------------------------------------------------------- no-allocation variant
// Scratch for it_layer_forward_static.  In host code this name is only a handle for
// cudaGetSymbolAddress, never a device address; kernels receive the looked-up pointer.
static __device__ __align__(256) unsigned char g_static_workspace[IT_STATIC_WORKSPACE_BYTES];

namespace {
constexpr int kMaxDevices = 64;
std::mutex g_static_mu;
void *g_static_ptr[kMaxDevices] = {nullptr};

// Device address of g_static_workspace on the current device (looked up once per device).
it_status static_workspace_ptr(void **out) {
  int dev = -1;
  IT_CUDA_TRY(cudaGetDevice(&dev));
  IT_REQUIRE(dev >= 0 && dev < kMaxDevices, IT_ERR_UNSUPPORTED, "device ordinal %d is beyond %d", dev, kMaxDevices);
  std::lock_guard<std::mutex> lk(g_static_mu);
  if (!g_static_ptr[dev]) {
    void *p = nullptr;
    IT_CUDA_TRY(cudaGetSymbolAddress(&p, g_static_workspace));
    IT_REQUIRE(p != nullptr && ((uintptr_t)p % 256) == 0, IT_ERR_CUDA, "built-in scratch has no usable device address");
    g_static_ptr[dev] = p;
  }
  *out = g_static_ptr[dev];
  return IT_OK;
}
}  // namespace

extern "C" it_status it_layer_forward_static(const it_graph *g, const it_layer_desc *layer, const void *h_in,
                                             void *h_out, void *stream) {
  IT_REQUIRE(g != nullptr, IT_ERR_INVALID_ARG, "graph is NULL");
  IT_TRY(check_layer(g, layer));
  const size_t s = (size_t)it_dtype_size(layer->feat_dtype);
  IT_TRY(check_io(g, h_in, (size_t)g->n * layer->in_dim * s, h_out, (size_t)g->n * layer->out_dim * s));
  IT_REQUIRE(!it_profile_is_on(), IT_ERR_UNSUPPORTED,
             "it_layer_forward_static does not run while instrumentation is on (it would create CUDA events)");
  const size_t need = plan_layer(g, layer).bytes;
  IT_REQUIRE(need <= (size_t)IT_STATIC_WORKSPACE_BYTES, IT_ERR_WORKSPACE,
             "layer needs %zu bytes of scratch, the built-in array holds %zu; use it_layer_forward with a caller workspace",
             need, (size_t)IT_STATIC_WORKSPACE_BYTES);
  void *ws = nullptr;
  IT_TRY(static_workspace_ptr(&ws));
  return layer_forward_impl(g, layer, h_in, h_out, (char *)ws, (size_t)IT_STATIC_WORKSPACE_BYTES, (cudaStream_t)stream);
}

extern "C" it_status it_infer(const it_graph *g, const it_layer_desc *layers, int32_t n_layers, const void *x, void *out,
                              void *workspace, size_t workspace_bytes, void *stream) {
  InferWs w;
  IT_TRY(plan_infer(g, layers, n_layers, &w));
  IT_REQUIRE(workspace != nullptr && ((uintptr_t)workspace % 256) == 0, IT_ERR_WORKSPACE, "workspace is NULL or not 256-byte aligned");
  IT_REQUIRE(workspace_bytes >= w.bytes, IT_ERR_WORKSPACE, "workspace has %zu bytes, it_infer needs %zu", workspace_bytes, w.bytes);
  const size_t es = (size_t)it_dtype_size(layers[0].feat_dtype);
  const size_t x_bytes = (size_t)g->n * layers[0].in_dim * es, out_bytes = (size_t)g->n * layers[n_layers - 1].out_dim * es;
  IT_TRY(check_io(g, x, x_bytes, out, out_bytes));
  IT_REQUIRE(g->n == 0 || (!overlaps(x, x_bytes, workspace, workspace_bytes) && !overlaps(out, out_bytes, workspace, workspace_bytes)),
             IT_ERR_INVALID_ARG, "x / out overlaps the workspace");
  char *ws = (char *)workspace;
  void *buf[2] = {ws + w.off_buf0, ws + w.off_buf1};
  const void *cur = x;
  cudaStream_t st = (cudaStream_t)stream;
  for (int i = 0; i < n_layers; ++i) {
    void *dst = (i == n_layers - 1) ? out : buf[i & 1];
    FusedPair f;
    if (g->n > 0 && i + 1 < n_layers && fused_pair(g, &layers[i], &layers[i + 1], &f)) {
      // layer i up to its aggregate; its update with the transform of layer i + 1, S and Z landing where H would have
      // been stored; then the rest of layer i + 1
      const it_layer_desc *A = &layers[i], *Bn = &layers[i + 1];
      StageCtx ca, cb;
      IT_TRY(stage_ctx(g, A, ws, w.layer_bytes, st, &ca));
      void *agg = agg_dim_of(A) > 0 ? (void *)(ws + ca.w.off_a) : nullptr;
      if (agg) IT_TRY(stage_gather(ca, cur, nullptr, nullptr, false, agg));
      void *B2 = ws + w.off_B2;
      IT_TRY(it_launch_prep_weights_tc(f.kind_a, A, f.ga.N1, f.ga.K1, f.ga.K2, ca.B, st));
      IT_TRY(it_launch_prep_weights_tc(f.kind_b, Bn, f.nb_b, f.ga.N1, 0, B2, st));
      char *S = (char *)dst, *Z = (char *)dst + f.s_bytes;
      if (plan_of(A) == PLAN_GCN) { f.ga.X1 = agg; f.ga.X2 = nullptr; }
      else { f.ga.X1 = cur; f.ga.X2 = f.ga.K2 > 0 ? agg : nullptr; }
      f.ga.out0 = S; f.ga.out1 = Z;
      IT_TRY(it_launch_gemm2_tc(f.ga, ca.B, B2, g->num_sms, g->d_status, st));
      void *dst2 = (i + 1 == n_layers - 1) ? out : buf[(i + 1) & 1];
      IT_TRY(stage_ctx(g, Bn, ws, w.layer_bytes, st, &cb));
      IT_TRY(stage_gather(cb, Z, nullptr, nullptr, false, dst2, S));
      cur = dst2;
      ++i;
      continue;
    }
    IT_TRY(layer_forward_impl(g, &layers[i], cur, dst, ws, w.layer_bytes, st));
    cur = dst;
  }
  return IT_OK;
}
