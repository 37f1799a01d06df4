// it_layer_forward / it_infer / it_workspace_bytes: argument checks, workspace carving and the
// launch sequence of one layer.  All arithmetic lives in the kernels of the other files.
#include <mutex>

#include "common.cuh"

namespace {

enum LayerPlan { PLAN_SAGE = 0, PLAN_SAGE_REORDER = 1, PLAN_GAT = 2, PLAN_DENSE = 3, PLAN_GCN = 4, PLAN_GCN_REORDER = 5 };

struct LayerWs {
  LayerPlan plan;
  size_t off_B, off_partials, off_a, off_b;  // a: aggregate A | self term S | scores ; b: Z
  size_t bytes;
};

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
    IT_REQUIRE(L->op != IT_GATHER_GAT && L->op != IT_GATHER_NONE, IT_ERR_UNSUPPORTED, "edge features are taken by the pooling layers and GCN only");
    IT_REQUIRE(g->edge_feat != nullptr, IT_ERR_INVALID_ARG, "layer uses edge features but the graph has none (it_graph_set_edge_features)");
    IT_REQUIRE(g->edge_dim == L->edge_dim && g->edge_dtype == L->feat_dtype, IT_ERR_INVALID_ARG,
               "layer expects edge features [%d] of its feat_dtype, the graph holds [%d]", L->edge_dim, g->edge_dim);
  }
  return IT_OK;
}

bool reorders(const it_layer_desc *L) {
  // with edge features the aggregate of the edge part would need its own transform: such layers keep the plain order
  return L->allow_reorder && L->edge_dim == 0 && (L->op == IT_GATHER_SUM || L->op == IT_GATHER_MEAN || L->op == IT_GATHER_GCN) && L->out_dim < L->in_dim;
}

LayerWs plan_layer(const it_graph *g, const it_layer_desc *L) {
  LayerWs w;
  const size_t n = (size_t)g->n, s = (size_t)it_dtype_size(L->feat_dtype);
  const size_t fi = (size_t)L->in_dim, fo = (size_t)L->out_dim, fe = (size_t)L->edge_dim;
  const size_t kpad = 128;   // the tensor-core path pads the K of each operand to whole k-blocks (at most 63 + 63 rows)
  size_t off = 0;
  auto take = [&](size_t bytes) { size_t o = off; off += it_align_up(bytes); return o; };
  if (L->op == IT_GATHER_GAT) {
    w.plan = PLAN_GAT;
    w.off_B = take((fi + kpad) * (fo + 2 * (size_t)L->heads) * 8);
    w.off_partials = take(it_gat_partial_bytes(g, L->out_dim, L->heads));
    w.off_a = take(n * 2 * (size_t)L->heads * 4);  // scores
    w.off_b = take(n * fo * s);                    // Z
  } else if (L->op == IT_GATHER_NONE) {
    w.plan = PLAN_DENSE;
    w.off_B = take((fi + kpad) * fo * 8);
    w.off_partials = w.off_a = w.off_b = off;
  } else if (L->op == IT_GATHER_GCN) {
    w.off_B = take((fi + fe + kpad) * fo * 8);
    if (reorders(L)) {
      w.plan = PLAN_GCN_REORDER;
      w.off_partials = take((size_t)g->n_partial_rows * fo * 4);
      w.off_a = off;
      w.off_b = take(n * fo * s);  // Z
    } else {
      w.plan = PLAN_GCN;
      w.off_partials = take((size_t)g->n_partial_rows * (fi > fe ? fi : fe) * 4);
      w.off_a = take(n * (fi + fe) * s);  // A = [sum_e w_e h_u | sum_e e_vu]
      w.off_b = off;
    }
  } else if (reorders(L)) {
    w.plan = PLAN_SAGE_REORDER;
    w.off_B = take((fi + kpad) * 2 * fo * 8);
    w.off_partials = take((size_t)g->n_partial_rows * fo * 4);
    w.off_a = take(n * fo * 4);  // S (fp32)
    w.off_b = take(n * fo * s);  // Z
  } else {
    w.plan = PLAN_SAGE;
    w.off_B = take((2 * fi + fe + kpad) * fo * 8);
    w.off_partials = take((size_t)g->n_partial_rows * (fi > fe ? fi : fe) * 4);
    w.off_a = take(n * (fi + fe) * s);  // A = [aggregate of w_e h_u | aggregate of e_vu]
    w.off_b = off;
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

// The edge-feature half of the message [w_e h_u | e_vu]: the same reduce over the rows of the edge-feature
// matrix, which lie in edge order, written to columns [in_dim, in_dim + edge_dim) of the aggregate.
it_status gather_edge_part(it_gather_args gg, const it_layer_desc *L, void *A, int a_ld, cudaStream_t st) {
  if (L->edge_dim == 0) return IT_OK;
  gg.src = gg.g->edge_feat; gg.src_ld = 0; gg.per_edge_rows = 1; gg.use_edge_weights = 0; gg.dim = L->edge_dim;
  gg.dst = (char *)A + (size_t)L->in_dim * it_dtype_size(gg.dtype); gg.dst_ld = a_ld;
  return it_launch_gather(gg, st);
}

it_status layer_forward_impl(const it_graph *g, const it_layer_desc *L, const void *h_in, void *h_out, char *ws,
                             size_t ws_bytes, cudaStream_t st) {
  const LayerWs w = plan_layer(g, L);
  IT_REQUIRE(ws_bytes >= w.bytes, IT_ERR_WORKSPACE, "workspace has %zu bytes, layer needs %zu", ws_bytes, w.bytes);
  IT_REQUIRE(L->W != nullptr, IT_ERR_INVALID_ARG, "W is NULL");
  float *B = reinterpret_cast<float *>(ws + w.off_B);
  float *partials = g->n_partial_rows > 0 ? reinterpret_cast<float *>(ws + w.off_partials) : nullptr;
  const it_dtype dt = L->feat_dtype;

  if (w.plan == PLAN_GAT) {
    IT_REQUIRE(L->att_src && L->att_dst, IT_ERR_INVALID_ARG, "GAT layer needs att_src and att_dst");
    float *scores = reinterpret_cast<float *>(ws + w.off_a);
    void *Z = ws + w.off_b;
    it_gemm_args ga{};
    ga.M = g->n; ga.x_dtype = dt; ga.X1 = h_in; ga.K1 = L->in_dim; ga.X2 = nullptr; ga.K2 = 0;
    ga.B = B; ga.NB = L->out_dim + 2 * L->heads;
    ga.n0 = 0; ga.out0 = nullptr; ga.dt0 = dt; ga.bias0 = nullptr; ga.act0 = IT_ACT_NONE;
    ga.n1 = L->out_dim; ga.out1 = Z; ga.dt1 = dt; ga.out2 = scores;
    IT_TRY(run_apply(g, L, IT_PREP_GAT, ga, B, scores, st));
    it_gat_args aa{};
    aa.g = g; aa.dtype = dt; aa.heads = L->heads; aa.head_dim = L->out_dim / L->heads; aa.z = Z; aa.scores = scores; aa.partials = partials;
    aa.slope = L->leaky_slope; aa.bias = L->bias; aa.act = L->act; aa.dst = h_out;
    return it_launch_gat(aa, st);
  }

  if (w.plan == PLAN_DENSE) {   // no Gather stage: h' = act(h W + b)
    it_gemm_args ga{};
    ga.M = g->n; ga.x_dtype = dt; ga.X1 = h_in; ga.K1 = L->in_dim; ga.X2 = nullptr; ga.K2 = 0;
    ga.B = B; ga.NB = L->out_dim;
    ga.n0 = L->out_dim; ga.out0 = h_out; ga.dt0 = dt; ga.bias0 = L->bias; ga.act0 = L->act;
    ga.n1 = 0; ga.out1 = nullptr; ga.dt1 = dt; ga.out2 = nullptr;
    return run_apply(g, L, IT_PREP_DENSE, ga, B, nullptr, st);
  }

  it_gather_args gg{};
  gg.g = g; gg.op = L->op == IT_GATHER_GCN ? IT_GATHER_SUM : L->op; gg.use_edge_weights = L->use_edge_weights; gg.dtype = dt;
  gg.partials = partials;
  const int a_ld = L->in_dim + L->edge_dim;   // row length of the aggregate handed to apply
  if (w.plan == PLAN_GCN_REORDER) {   // Z = H W, then h' = act(sum_e w_e z_u + b) in the gather's epilogue
    void *Z = ws + w.off_b;
    it_gemm_args ga{};
    ga.M = g->n; ga.x_dtype = dt; ga.X1 = h_in; ga.K1 = L->in_dim; ga.X2 = nullptr; ga.K2 = 0;
    ga.B = B; ga.NB = L->out_dim;
    ga.n0 = 0; ga.out0 = nullptr; ga.dt0 = dt; ga.bias0 = nullptr; ga.act0 = IT_ACT_NONE;
    ga.n1 = L->out_dim; ga.out1 = Z; ga.dt1 = dt; ga.out2 = nullptr;
    IT_TRY(run_apply(g, L, IT_PREP_DENSE, ga, B, nullptr, st));
    gg.dim = L->out_dim; gg.src = Z; gg.dst = h_out; gg.epi = IT_EPI_BIAS_ACT; gg.self_term = nullptr; gg.bias = L->bias; gg.act = L->act;
    return it_launch_gather(gg, st);
  }
  if (w.plan == PLAN_GCN) {   // A = sum_e [w_e h_u | e_vu], then h' = act(A W + b)
    void *A = ws + w.off_a;
    gg.dim = L->in_dim; gg.src = h_in; gg.dst = A; gg.dst_ld = a_ld; gg.epi = IT_EPI_STORE; gg.self_term = nullptr; gg.bias = nullptr; gg.act = IT_ACT_NONE;
    IT_TRY(it_launch_gather(gg, st));
    IT_TRY(gather_edge_part(gg, L, A, a_ld, st));
    it_gemm_args ga{};
    ga.M = g->n; ga.x_dtype = dt; ga.X1 = A; ga.K1 = a_ld; ga.X2 = nullptr; ga.K2 = 0;
    ga.B = B; ga.NB = L->out_dim;
    ga.n0 = L->out_dim; ga.out0 = h_out; ga.dt0 = dt; ga.bias0 = L->bias; ga.act0 = L->act;
    ga.n1 = 0; ga.out1 = nullptr; ga.dt1 = dt; ga.out2 = nullptr;
    return run_apply(g, L, IT_PREP_DENSE, ga, B, nullptr, st);
  }
  if (w.plan == PLAN_SAGE_REORDER) {
    float *S = reinterpret_cast<float *>(ws + w.off_a);
    void *Z = ws + w.off_b;
    it_gemm_args ga{};
    ga.M = g->n; ga.x_dtype = dt; ga.X1 = h_in; ga.K1 = L->in_dim; ga.X2 = nullptr; ga.K2 = 0;
    ga.B = B; ga.NB = 2 * L->out_dim;
    ga.n0 = L->out_dim; ga.out0 = S; ga.dt0 = IT_F32; ga.bias0 = L->bias; ga.act0 = IT_ACT_NONE;
    ga.n1 = L->out_dim; ga.out1 = Z; ga.dt1 = dt; ga.out2 = nullptr;
    IT_TRY(run_apply(g, L, IT_PREP_SAGE_REORDER, ga, B, nullptr, st));
    gg.dim = L->out_dim; gg.src = Z; gg.dst = h_out; gg.epi = IT_EPI_ADD_ACT; gg.self_term = S; gg.act = L->act;
    return it_launch_gather(gg, st);
  }
  void *A = ws + w.off_a;
  gg.dim = L->in_dim; gg.src = h_in; gg.dst = A; gg.dst_ld = a_ld; gg.epi = IT_EPI_STORE; gg.self_term = nullptr; gg.act = IT_ACT_NONE;
  IT_TRY(it_launch_gather(gg, st));
  IT_TRY(gather_edge_part(gg, L, A, a_ld, st));
  it_gemm_args ga{};
  ga.M = g->n; ga.x_dtype = dt; ga.X1 = h_in; ga.K1 = L->in_dim; ga.X2 = A; ga.K2 = a_ld;
  ga.B = B; ga.NB = L->out_dim;
  ga.n0 = L->out_dim; ga.out0 = h_out; ga.dt0 = dt; ga.bias0 = L->bias; ga.act0 = L->act;
  ga.n1 = 0; ga.out1 = nullptr; ga.dt1 = dt; ga.out2 = nullptr;
  return run_apply(g, L, IT_PREP_SAGE, ga, B, nullptr, st);
}

struct InferWs { size_t layer_bytes, buf_bytes, off_buf0, off_buf1, bytes; };

it_status plan_infer(const it_graph *g, const it_layer_desc *layers, int32_t n_layers, InferWs *out) {
  IT_REQUIRE(g != nullptr, IT_ERR_INVALID_ARG, "graph is NULL");
  IT_REQUIRE(layers != nullptr && n_layers >= 1, IT_ERR_INVALID_ARG, "need at least one layer");
  InferWs w{0, 0, 0, 0, 0};
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
  }
  w.off_buf0 = w.layer_bytes;
  w.off_buf1 = w.off_buf0 + (n_layers >= 2 ? w.buf_bytes : 0);
  w.bytes = w.off_buf1 + (n_layers >= 3 ? w.buf_bytes : 0);
  *out = w;
  return IT_OK;
}

bool overlaps(const void *a, size_t na, const void *b, size_t nb) {
  const char *x = (const char *)a, *y = (const char *)b;
  return x < y + nb && y < x + na;
}

// What every forward call checks about the graph and its input / output matrices before anything is launched:
// the kernels move 16-byte slices of the rows, so a pointer that is not 16-byte aligned would fault on the device.
it_status check_io(const it_graph *g, const void *in, size_t in_bytes, const void *out, size_t out_bytes) {
  IT_REQUIRE(g->n == 0 || g->bucket_meta != nullptr, IT_ERR_BAD_GRAPH,
             "the graph has no row split (an it_split_hubs call failed): call it_split_hubs again before a forward pass");
  if (g->n == 0) return IT_OK;
  IT_REQUIRE(in != nullptr && out != nullptr, IT_ERR_INVALID_ARG, "input / output matrix is NULL");
  IT_REQUIRE(((uintptr_t)in % 16) == 0 && ((uintptr_t)out % 16) == 0, IT_ERR_INVALID_ARG,
             "input and output matrices must be 16-byte aligned (got %p, %p)", in, out);
  IT_REQUIRE(!overlaps(in, in_bytes, out, out_bytes), IT_ERR_INVALID_ARG, "input and output matrices overlap");
  return IT_OK;
}

}  // namespace

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
  for (int i = 0; i < n_layers; ++i) {
    void *dst = (i == n_layers - 1) ? out : buf[i & 1];
    IT_TRY(layer_forward_impl(g, &layers[i], cur, dst, ws, w.layer_bytes, (cudaStream_t)stream));
    cur = dst;
  }
  return IT_OK;
}
