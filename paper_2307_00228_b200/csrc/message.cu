// Elementwise kernels around the gather:
//   * the learned message of every edge, m_j = act(P[u_j] + Q[j]) (the source part P was computed once per vertex, the
//     edge part Q once per edge, both by the dense transform), written over Q so that the per-edge-row gather can
//     reduce it;
//   * for GAT layers whose logits read the edge features: the message row of every edge (a copy of its source's row)
//     and its logit term per head (source score + the edge's share), so that the reduce can walk rows in edge order;
//   * the receiver's finish of a partial-gather over source partitions (scale, zero the vertices without in-edges,
//     round to the storage type).
// All are HBM-bound streams of 16-byte slices; the only irregular access is the source row of an edge.
#include "common.cuh"

namespace {

constexpr int MSG_THREADS = 256;
constexpr int MSG_UNROLL = 4;   // slices in flight per thread

__device__ __forceinline__ float msg_act(float x, int act) {
  if (act == IT_ACT_RELU) return fmaxf(x, 0.f);
  if (act == IT_ACT_ELU) return it_elu(x);
  return x;
}

// 16 bytes of a row: four fp32 or eight bf16 values
template <typename T>
__device__ __forceinline__ uint4 add_act_slice(const uint4 &p, const uint4 &q, int act) {
  const uint32_t pw[4] = {p.x, p.y, p.z, p.w}, qw[4] = {q.x, q.y, q.z, q.w};
  uint32_t o[4];
  if constexpr (sizeof(T) == 4) {
#pragma unroll
    for (int i = 0; i < 4; ++i) o[i] = __float_as_uint(msg_act(__uint_as_float(pw[i]) + __uint_as_float(qw[i]), act));
  } else {
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      const float lo = msg_act(__uint_as_float(pw[i] << 16) + __uint_as_float(qw[i] << 16), act);
      const float hi = msg_act(__uint_as_float(pw[i] & 0xffff0000u) + __uint_as_float(qw[i] & 0xffff0000u), act);
      __nv_bfloat162 h = __floats2bfloat162_rn(lo, hi);
      o[i] = *reinterpret_cast<uint32_t *>(&h);
    }
  }
  return make_uint4(o[0], o[1], o[2], o[3]);
}

// slices: 16-byte slices per row; total = n_edges * slices
template <typename T>
__global__ void __launch_bounds__(MSG_THREADS) edge_messages_kernel(const int32_t *__restrict__ indices, const uint4 *__restrict__ P,
                                                                    uint4 *__restrict__ M, int64_t total, int slices, int act) {
  const int64_t stride = (int64_t)gridDim.x * MSG_THREADS;
  for (int64_t t0 = (int64_t)blockIdx.x * MSG_THREADS + threadIdx.x; t0 < total; t0 += stride * MSG_UNROLL) {
    uint4 p[MSG_UNROLL], q[MSG_UNROLL];
#pragma unroll
    for (int u = 0; u < MSG_UNROLL; ++u) {
      const int64_t t = t0 + u * stride;
      if (t < total) {
        const int64_t j = t / slices;
        const int c = (int)(t - j * slices);
        const int64_t src = __ldg(indices + j);
        p[u] = __ldg(P + src * slices + c);
        q[u] = __ldcs(M + t);
      }
    }
#pragma unroll
    for (int u = 0; u < MSG_UNROLL; ++u) {
      const int64_t t = t0 + u * stride;
      if (t < total) __stcs(M + t, add_act_slice<T>(p[u], q[u], act));
    }
  }
}

// GAT with edge features: the message row of every edge (a copy of its source's row, so that the reduce can walk rows
// in edge order) ...
__global__ void __launch_bounds__(MSG_THREADS) gat_edge_rows_kernel(const int32_t *__restrict__ indices, const uint4 *__restrict__ Z,
                                                                    uint4 *__restrict__ Zj, int64_t total, int slices) {
  const int64_t stride = (int64_t)gridDim.x * MSG_THREADS;
  for (int64_t t0 = (int64_t)blockIdx.x * MSG_THREADS + threadIdx.x; t0 < total; t0 += stride * MSG_UNROLL) {
    uint4 z[MSG_UNROLL];
#pragma unroll
    for (int u = 0; u < MSG_UNROLL; ++u) {
      const int64_t t = t0 + u * stride;
      if (t < total) {
        const int64_t j = t / slices;
        z[u] = __ldg(Z + (int64_t)__ldg(indices + j) * slices + (t - j * slices));
      }
    }
#pragma unroll
    for (int u = 0; u < MSG_UNROLL; ++u) {
      const int64_t t = t0 + u * stride;
      if (t < total) __stcs(Zj + t, z[u]);
    }
  }
}
// ... and its logit term per head: the source's score plus the edge's own share att_edge[h] . e_j
template <typename T>
__global__ void __launch_bounds__(MSG_THREADS) gat_edge_scores_kernel(const int32_t *__restrict__ indices, const float *__restrict__ scores,
                                                                      const T *__restrict__ ef, const float *__restrict__ att_edge,
                                                                      float *__restrict__ sc, int64_t n_edges, int heads, int edge_dim) {
  const int64_t total = n_edges * heads, stride = (int64_t)gridDim.x * MSG_THREADS;
  for (int64_t t = (int64_t)blockIdx.x * MSG_THREADS + threadIdx.x; t < total; t += stride) {
    const int64_t j = t / heads;
    const int h = (int)(t - j * heads);
    float acc = 0.f;
    for (int k = 0; k < edge_dim; ++k) {
      float e;
      if constexpr (sizeof(T) == 4) e = __ldg(reinterpret_cast<const float *>(ef) + j * edge_dim + k);
      else e = __bfloat162float(ef[j * edge_dim + k]);
      acc = fmaf(__ldg(att_edge + h * edge_dim + k), e, acc);
    }
    sc[t] = __ldg(scores + (int64_t)__ldg(indices + j) * (2 * heads) + h) + acc;
  }
}

__global__ void __launch_bounds__(MSG_THREADS) compact_scores_kernel(const float *__restrict__ scores, float *__restrict__ dense,
                                                                     int64_t total, int heads) {
  const int64_t stride = (int64_t)gridDim.x * MSG_THREADS;
  for (int64_t t = (int64_t)blockIdx.x * MSG_THREADS + threadIdx.x; t < total; t += stride) {
    const int64_t v = t / heads;
    dense[t] = __ldcs(scores + v * 2 * heads + (t - v * heads));
  }
}

// one thread per four consecutive entries of a row
template <typename T>
__global__ void __launch_bounds__(MSG_THREADS) aggregate_finish_kernel(const float4 *__restrict__ raw, const float *__restrict__ scale,
                                                                       T *__restrict__ out, int64_t total4, int quads) {
  const int64_t stride = (int64_t)gridDim.x * MSG_THREADS;
  for (int64_t t = (int64_t)blockIdx.x * MSG_THREADS + threadIdx.x; t < total4; t += stride) {
    const int64_t v = t / quads;
    const float s = __ldg(scale + v);
    float4 x = __ldcs(raw + t);
    if (s == 0.f) x = make_float4(0.f, 0.f, 0.f, 0.f);
    else { x.x *= s; x.y *= s; x.z *= s; x.w *= s; }
    if constexpr (sizeof(T) == 4) {
      reinterpret_cast<float4 *>(out)[t] = x;
    } else {
      __nv_bfloat162 a = __floats2bfloat162_rn(x.x, x.y), b = __floats2bfloat162_rn(x.z, x.w);
      reinterpret_cast<uint2 *>(out)[t] = make_uint2(*reinterpret_cast<uint32_t *>(&a), *reinterpret_cast<uint32_t *>(&b));
    }
  }
}

}  // namespace

it_status it_launch_edge_messages(const it_graph *g, it_dtype dtype, int dim, const void *P, void *M, it_act act, cudaStream_t st) {
  const int es = it_dtype_size(dtype);
  IT_REQUIRE(dim > 0 && (dim * es) % 16 == 0, IT_ERR_INVALID_ARG, "edge messages: a row of %d bytes is not a multiple of 16", dim * es);
  if (g->e == 0) return IT_OK;
  const int slices = dim * es / 16;
  const int64_t total = g->e * slices;
  const int64_t want = (total + (int64_t)MSG_THREADS * MSG_UNROLL - 1) / ((int64_t)MSG_THREADS * MSG_UNROLL);
  const int64_t cap = (int64_t)g->num_sms * 16;
  const unsigned blocks = (unsigned)(want < cap ? want : cap);
  // per edge: its index, one row of P (read), one row of Q (read) and the message (written)
  const double bytes = (double)g->e * (4.0 + 3.0 * dim * es);
  if (dtype == IT_F32)
    IT_LAUNCH(IT_K_EDGE_MSG, bytes, 0, st, edge_messages_kernel<float><<<blocks, MSG_THREADS, 0, st>>>(
        g->indices, reinterpret_cast<const uint4 *>(P), reinterpret_cast<uint4 *>(M), total, slices, (int)act));
  else
    IT_LAUNCH(IT_K_EDGE_MSG, bytes, 0, st, edge_messages_kernel<__nv_bfloat16><<<blocks, MSG_THREADS, 0, st>>>(
        g->indices, reinterpret_cast<const uint4 *>(P), reinterpret_cast<uint4 *>(M), total, slices, (int)act));
  IT_CUDA_TRY(cudaGetLastError());
  return IT_OK;
}

it_status it_launch_gat_edge_rows(const it_graph *g, it_dtype dtype, int dim, int heads, const void *Z, const float *scores,
                                  const float *att_edge, void *Zj, float *sc, cudaStream_t st) {
  if (g->e == 0) return IT_OK;
  const int es = it_dtype_size(dtype);
  const int slices = dim * es / 16;
  const int64_t total = g->e * slices;
  const int64_t cap = (int64_t)g->num_sms * 16;
  int64_t want = (total + (int64_t)MSG_THREADS * MSG_UNROLL - 1) / ((int64_t)MSG_THREADS * MSG_UNROLL);
  unsigned blocks = (unsigned)(want < cap ? want : cap);
  IT_LAUNCH(IT_K_EDGE_MSG, (double)g->e * (4.0 + 2.0 * dim * es), 0, st,
            gat_edge_rows_kernel<<<blocks, MSG_THREADS, 0, st>>>(g->indices, reinterpret_cast<const uint4 *>(Z), reinterpret_cast<uint4 *>(Zj), total, slices));
  want = (g->e * heads + MSG_THREADS - 1) / MSG_THREADS;
  blocks = (unsigned)(want < cap ? want : cap);
  const double sbytes = (double)g->e * (4.0 + (double)g->edge_dim * es + 8.0 * heads);
  if (dtype == IT_F32)
    IT_LAUNCH(IT_K_EDGE_MSG, sbytes, 0, st, gat_edge_scores_kernel<float><<<blocks, MSG_THREADS, 0, st>>>(
        g->indices, scores, reinterpret_cast<const float *>(g->edge_feat), att_edge, sc, g->e, heads, g->edge_dim));
  else
    IT_LAUNCH(IT_K_EDGE_MSG, sbytes, 0, st, gat_edge_scores_kernel<__nv_bfloat16><<<blocks, MSG_THREADS, 0, st>>>(
        g->indices, scores, reinterpret_cast<const __nv_bfloat16 *>(g->edge_feat), att_edge, sc, g->e, heads, g->edge_dim));
  IT_CUDA_TRY(cudaGetLastError());
  return IT_OK;
}

it_status it_launch_compact_scores(int64_t n, int heads, const float *scores, float *dense, cudaStream_t st) {
  if (n == 0) return IT_OK;
  const int64_t total = n * heads;
  const int64_t want = (total + MSG_THREADS - 1) / MSG_THREADS, cap = (int64_t)IT_NUM_SMS_FALLBACK * 32;
  IT_LAUNCH(IT_K_EDGE_MSG, (double)n * heads * 12.0, 0, st,
            compact_scores_kernel<<<(unsigned)(want < cap ? want : cap), MSG_THREADS, 0, st>>>(scores, dense, total, heads));
  IT_CUDA_TRY(cudaGetLastError());
  return IT_OK;
}

it_status it_launch_aggregate_finish(int64_t n, int dim, it_dtype dtype, const float *raw, const float *scale, void *out, cudaStream_t st) {
  IT_REQUIRE(dim > 0 && dim % 4 == 0, IT_ERR_INVALID_ARG, "aggregate finish: dim %d is not a multiple of 4", dim);
  if (n == 0) return IT_OK;
  const int quads = dim / 4;
  const int64_t total4 = n * quads;
  const int64_t want = (total4 + MSG_THREADS - 1) / MSG_THREADS;
  const int64_t cap = (int64_t)IT_NUM_SMS_FALLBACK * 32;
  const unsigned blocks = (unsigned)(want < cap ? want : cap);
  const double bytes = (double)n * (4.0 + dim * (4.0 + it_dtype_size(dtype)));
  if (dtype == IT_F32)
    IT_LAUNCH(IT_K_AGG_FINISH, bytes, 0, st, aggregate_finish_kernel<float><<<blocks, MSG_THREADS, 0, st>>>(
        reinterpret_cast<const float4 *>(raw), scale, reinterpret_cast<float *>(out), total4, quads));
  else
    IT_LAUNCH(IT_K_AGG_FINISH, bytes, 0, st, aggregate_finish_kernel<__nv_bfloat16><<<blocks, MSG_THREADS, 0, st>>>(
        reinterpret_cast<const float4 *>(raw), scale, reinterpret_cast<__nv_bfloat16 *>(out), total4, quads));
  IT_CUDA_TRY(cudaGetLastError());
  return IT_OK;
}
