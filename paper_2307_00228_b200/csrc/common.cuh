// Shared declarations of the layer-pass library (host + device helpers, the graph handle,
// the launch entry points of each kernel file).  sm_100a only.
#pragma once

#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>
#include <stdio.h>

#include "inferturbo.h"

#define IT_NUM_SMS_FALLBACK 148

// ----------------------------------------------------------------------------- errors
void it_set_error(const char *fmt, ...);

#define IT_CUDA_TRY(expr)                                                            \
  do {                                                                               \
    cudaError_t _e = (expr);                                                         \
    if (_e != cudaSuccess) {                                                         \
      it_set_error("%s failed: %s (%s:%d)", #expr, cudaGetErrorString(_e), __FILE__, \
                   __LINE__);                                                        \
      return (_e == cudaErrorMemoryAllocation) ? IT_ERR_OOM : IT_ERR_CUDA;           \
    }                                                                                \
  } while (0)

#define IT_TRY(expr)               \
  do {                             \
    it_status _s = (expr);         \
    if (_s != IT_OK) return _s;    \
  } while (0)

#define IT_REQUIRE(cond, code, ...) \
  do {                              \
    if (!(cond)) {                  \
      it_set_error(__VA_ARGS__);    \
      return (code);                \
    }                               \
  } while (0)

// ----------------------------------------------------------------------------- instrumentation
enum it_kernel_id {
  IT_K_VALIDATE = 0, IT_K_SPLIT_SCAN, IT_K_SPLIT_FILL, IT_K_BUCKET_SCAN, IT_K_PREP, IT_K_GATHER_CTA, IT_K_GATHER_FLAT,
  IT_K_GATHER_EMPTY, IT_K_COMBINE, IT_K_GEMM_FP32, IT_K_GEMM_TC, IT_K_GAT_CTA, IT_K_GAT_FLAT, IT_K_GAT_EMPTY,
  IT_K_EDGE_MSG, IT_K_AGG_FINISH, IT_K_GEMM2_TC,
  IT_K_COUNT
};
// Wraps one kernel launch: counts it and, while profiling is on, brackets it with events on `st`.
struct it_prof_scope {
  it_prof_scope(int kid, double algo_bytes, double algo_flops, cudaStream_t st);
  ~it_prof_scope();
  int slot_;
  cudaStream_t st_;
};
bool it_profile_is_on();
#define IT_LAUNCH(kid, bytes, flops, st, ...) \
  do {                                        \
    it_prof_scope _scope((kid), (bytes), (flops), (st)); \
    __VA_ARGS__;                              \
  } while (0)

// ----------------------------------------------------------------------------- graph handle
// One shadow row as the gather kernels read it: first edge, edge count, and where the
// aggregate goes (vertex id >= 0 for an unsplit row, ~slot in the partial buffer otherwise).
struct __align__(16) it_row_meta {
  int64_t j0;
  int32_t len;
  int32_t dest;
};

struct it_graph {
  int64_t n = 0, e = 0;
  int64_t n_src = 0;   // rows of the table the source ids name (= n unless the graph is one part of a partition)
  const void *indptr = nullptr;
  it_itype indptr_type = IT_I64;
  const int32_t *indices = nullptr;
  const float *edge_weights = nullptr;
  const void *edge_feat = nullptr;   // [e, edge_dim] rows in CSR order (borrowed), set by it_graph_set_edge_features
  int32_t edge_dim = 0;
  it_dtype edge_dtype = IT_F32;
  int device = 0;
  int num_sms = IT_NUM_SMS_FALLBACK;

  // derived by the split (library-owned, device)
  int64_t threshold = 0;
  int64_t n_rows = 0;           // R
  int64_t n_split_owners = 0;   // vertices with more than one shadow row
  int64_t n_partial_rows = 0;   // shadow rows that belong to split owners
  int64_t *shadow_indptr = nullptr;  // [R+1]
  int32_t *shadow_owner = nullptr;   // [R]
  int64_t *owner_indptr = nullptr;   // [n+1]
  int32_t *row_dest = nullptr;       // [R]  v >= 0: row is the whole segment of v; < 0: ~index into the partial buffer
  int32_t *split_owners = nullptr;   // [n_split_owners] ascending vertex ids
  int32_t n_buckets = 0;
  int64_t bucket_bounds[IT_MAX_BUCKETS] = {0};
  int64_t h_bucket_offsets[IT_MAX_BUCKETS + 1] = {0};
  int64_t h_bucket_edges[IT_MAX_BUCKETS] = {0};  // edges held by the rows of each bucket
  int64_t *bucket_offsets = nullptr;  // device [n_buckets+1]
  int32_t *bucket_rows = nullptr;     // [R]
  int *d_status = nullptr;            // device word: set to 1 by a kernel whose bounded wait gave up
  int32_t *bucket_owner = nullptr;    // [R] in bucket order: the vertex each row belongs to
  it_row_meta *bucket_meta = nullptr; // [R] in bucket order: what a gather needs to know about one row, in one 16-byte load
};

static inline size_t it_align_up(size_t x, size_t a = 256) { return (x + a - 1) / a * a; }

// ELU on the device.  The negative branch is exp(x) - 1 with the hardware exponential (absolute error below 1e-6,
// a handful of instructions where expm1f costs a few dozen in the end-of-row code of every short row); close to
// zero, where that difference cancels, the three-term series x + x^2/2 + x^3/6 takes over (relative error below
// 2e-6 at the switch point x = -1/32 and falling towards 0), so the result is relatively accurate everywhere.
#ifndef IT_FAST_ELU
#define IT_FAST_ELU 1
#endif
#ifdef __CUDACC__
__device__ __forceinline__ float it_elu(float x) {
#if IT_FAST_ELU
  const float series = x * fmaf(x, fmaf(x, 1.f / 6.f, 0.5f), 1.f);
  return x > 0.f ? x : (x > -0.03125f ? series : __expf(x) - 1.f);
#else
  return x > 0.f ? x : expm1f(x);
#endif
}
#endif
static inline int it_dtype_size(it_dtype t) { return t == IT_F32 ? 4 : 2; }

// ----------------------------------------------------------------------------- gather.cu
// What a gather / combine kernel does with the finished aggregate of vertex v.
enum it_epilogue_kind {
  IT_EPI_STORE = 0,      // dst[v, :] = agg                      (feat dtype)
  IT_EPI_ADD_ACT = 1,    // dst[v, :] = act(self[v, :] + agg)    (self fp32 or feat dtype, dst feat dtype)
  IT_EPI_BIAS_ACT = 2,   // dst[v, :] = act(bias + agg)          (bias fp32 [dim] or NULL)
  IT_EPI_RAW_F32 = 3     // dst[v, :] = the raw reduce in fp32: plain sum (mean undivided), max or min, and the identity of
                         // the reduce (0, -inf, +inf) for a row without edges: one part's share of a partial-gather
};

struct it_gather_args {
  const it_graph *g;
  it_gather_op op;         // SUM / MEAN / MAX
  int use_edge_weights;
  it_dtype dtype;          // of src rows and of dst rows
  int dim;                 // elements of a row that are gathered (any multiple of 16 bytes)
  const void *src;         // rows that are gathered: row u starts at src + u * src_ld elements
  int src_ld;              // 0 means dim
  int per_edge_rows;       // 1: src is [n_edges, dim] and row j belongs to edge j (edge features); 0: rows are looked up by source vertex
  float *partials;         // [n_partial_rows, dim] fp32 scratch (may be NULL when nothing is split)
  int *counters;           // IT_MAX_BUCKETS device words of scratch from which warps claim their batches (NULL: fixed strides)
  void *dst;               // row v starts at dst + v * dst_ld elements and takes dim of them
  int dst_ld;              // 0 means dim
  it_epilogue_kind epi;
  const void *self_term;   // IT_EPI_ADD_ACT only: row v starts at self_term + v * self_ld elements of self_dtype
  it_dtype self_dtype;     // IT_F32, or the dtype of the rows (the self term of a transform-first layer is stored like the rows)
  int self_ld;             // 0 means dim
  const float *bias;       // [dim] fp32 or NULL, IT_EPI_BIAS_ACT only
  it_act act;              // IT_EPI_ADD_ACT and IT_EPI_BIAS_ACT
};
it_status it_launch_gather(const it_gather_args &a, cudaStream_t stream);

// ----------------------------------------------------------------------------- gat.cu
struct it_gat_args {
  const it_graph *g;
  it_dtype dtype;
  int heads, head_dim;
  const void *z;          // [n, heads*head_dim] messages
  const float *scores;    // [n_src, 2*heads]: source scores of the vertex, then its destination scores
  const float *scores_dst;   // the same layout, row v = local destination v (scores + first_vertex * 2*heads for a part; NULL: scores)
  int per_edge_rows;      // 1: z is [n_edges, dim] and src_scores [n_edges, heads], row j belonging to edge j (edge features in the logits)
  const float *src_scores;   // [rows, heads], dense: the source-side logit term that is read per edge (row = source vertex, or the
                             // edge itself with per_edge_rows); NULL: the first half of the rows of `scores`
  float *partials;        // it_gat_partial_bytes() of fp32 scratch for the groups of split vertices (may be NULL if none)
  int *counters;          // IT_MAX_BUCKETS device words of scratch from which warps claim their batches (NULL: fixed strides)
  float slope;
  const float *bias;      // may be NULL
  it_act act;
  void *dst;              // [n, heads*head_dim]
};
it_status it_launch_gat(const it_gat_args &a, cudaStream_t stream);
size_t it_gat_partial_bytes(const it_graph *g, int dim, int heads);

// ----------------------------------------------------------------------------- apply.cu
// C[M, NB] = X1[M, K1] * B[0:K1, :] + X2[M, K2] * B[K1:K1+K2, :]   (X2 may be NULL, K2 = 0)
// B is an fp32 [K1+K2, NB] matrix assembled by it_launch_prep_weights.  Column ranges of C
// go to up to three destinations:
//   [0, n0)        -> out0 (dtype dt0) = act0(C + bias0)
//   [n0, n0+n1)    -> out1 (dtype dt1), raw
//   [n0+n1, NB)    -> out2 (fp32), raw, row stride n2 = NB - n0 - n1
struct it_gemm_args {
  int64_t M;
  it_dtype x_dtype;
  const void *X1; int K1;
  const void *X2; int K2;
  const float *B; int NB;
  int n0; void *out0; it_dtype dt0; const float *bias0; it_act act0;
  int n1; void *out1; it_dtype dt1;
  void *out2;
  uint32_t spin_limit;   // tensor-core path: polls after which a barrier wait gives up (0 = the default)
  int no_loads;          // tensor-core path, test hook: issue no operand copies
};
it_status it_launch_gemm(const it_gemm_args &a, cudaStream_t stream);

enum it_prep_kind { IT_PREP_SAGE = 0, IT_PREP_SAGE_REORDER = 1, IT_PREP_GAT = 2, IT_PREP_DENSE = 3 };   // DENSE: B = W [in, out] as it is
// Assemble the fp32 B matrix for a layer (K = its row count): SAGE and dense / GCN: a copy of W [K, out]; REORDER [in, 2*out] =
// [W_self | W_neigh]; GAT [in, out + 2*heads] = [W | W a_src | W a_dst].
it_status it_launch_prep_weights(it_prep_kind kind, const it_layer_desc *layer, int K, float *B,
                                 cudaStream_t stream);

// ----------------------------------------------------------------------------- apply_tc.cu
// The same product on the tensor cores (tcgen05 + TMEM + TMA).  Needs operand rows that are multiples of 16
// bytes (K1, K2 are padded to whole 128-byte k-blocks with zeros) and n0, n0 + n1 multiples of 16; computes the n0 + n1 columns and, for GAT, the
// attention scores [M, 2*heads] in its epilogue (a.B, a.NB and a.out2 are not used).  B is the
// matrix written by it_launch_prep_weights_tc: bf16 [NB, Kp] or fp32 [2, NB, Kp] (hi, lo), K-major, Kp = padded K1 + padded K2.
bool it_tc_supported(const it_gemm_args &a, int heads, int head_dim, bool want_scores);
it_status it_launch_prep_weights_tc(it_prep_kind kind, const it_layer_desc *layer, int NB, int K1, int K2, void *B,
                                    cudaStream_t stream);
it_status it_launch_gemm_tc(const it_gemm_args &a, const void *B, const float *att_src, const float *att_dst,
                            int heads, int head_dim, float *scores, int num_sms, int *status, cudaStream_t stream);

// The update of one layer and the transform of the next as one kernel (bf16 only): H = act1([X1 | X2] B1 + bias1) is
// rounded to bf16 and multiplied by B2 without leaving the SM; columns [0, n0) of H B2, plus bias0, go to out0 and
// columns [n0, n0 + n1) to out1.  N1 (columns of H), n0 and n1 must be multiples of 64.
struct it_gemm2_args {
  int64_t M;
  const void *X1; int K1;
  const void *X2; int K2;
  int N1; const float *bias1; it_act act1;
  int n0; void *out0; const float *bias0;
  int n1; void *out1;
  uint32_t spin_limit;   // polls after which a barrier wait gives up (0 = the default)
  int no_loads;          // test hook: issue no operand copies
};
bool it_tc2_supported(const it_gemm2_args &a);
it_status it_launch_gemm2_tc(const it_gemm2_args &a, const void *B1, const void *B2, int num_sms, int *status, cudaStream_t stream);

// ----------------------------------------------------------------------------- message.cu
// Learned messages, edge by edge: M[j, :] = act(P[indices[j], :] + M[j, :]) in place (M arrives holding the per-edge
// part Q), rows of `dim` elements of `dtype` (a multiple of 16 bytes).
it_status it_launch_edge_messages(const it_graph *g, it_dtype dtype, int dim, const void *P, void *M, it_act act, cudaStream_t stream);
// GAT with edge features: Zj[j, :] = Z[indices[j], :] and sc[j, h] = scores[indices[j], h] + att_edge[h, :] . ef[j, :].
it_status it_launch_gat_edge_rows(const it_graph *g, it_dtype dtype, int dim, int heads, const void *Z, const float *scores,
                                  const float *att_edge, void *Zj, float *sc, cudaStream_t stream);
// dense[v, :] = scores[v, 0:heads]: the source scores on their own, 16 bytes per vertex for 4 heads instead of a 32-byte
// row shared with the destination scores (the reduce reads one per edge, at random).
it_status it_launch_compact_scores(int64_t n, int heads, const float *scores, float *dense, cudaStream_t stream);
// out[v, :] = raw[v, :] * scale[v] (0 where scale[v] = 0), fp32 -> dtype.
it_status it_launch_aggregate_finish(int64_t n, int dim, it_dtype dtype, const float *raw, const float *scale, void *out, cudaStream_t stream);
