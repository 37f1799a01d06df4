// Gather (aggregate over the in-edges of one shadow row) and combine (fold the partial
// results of a split vertex).  HBM-bound: one 16-byte load per lane per edge, several edges
// in flight per lane, fp32 accumulation in a fixed order (results are bit-reproducible; no
// floating-point atomics anywhere).
//
// Work decomposition.  A feature row of `dim` elements is LPR = dim * sizeof(T) / 16 lanes
// wide.  A *group* of GROUP lanes (LPR <= GROUP <= 32) owns one shadow row at a time and
// works on SLOTS = GROUP / LPR edges at once; slot s takes edges s, s + SLOTS, ... of the
// row, and the slots are folded with shuffles at the end.  Which GROUP a row gets depends on
// its degree bucket: short rows -> GROUP = LPR (several rows per warp), medium rows -> one
// warp per row, long rows (up to the split threshold) -> one CTA per row.
#include "common.cuh"

namespace {

constexpr int GATHER_THREADS = 256;
constexpr int UNROLL = 8;

template <typename T> struct Row16;
template <> struct Row16<float> {
  static constexpr int VEC = 4;
  __device__ static __forceinline__ void load(const float *p, float (&v)[4]) {
    float4 x = __ldg(reinterpret_cast<const float4 *>(p));
    v[0] = x.x; v[1] = x.y; v[2] = x.z; v[3] = x.w;
  }
  __device__ static __forceinline__ void store(float *p, const float (&v)[4]) {
    *reinterpret_cast<float4 *>(p) = make_float4(v[0], v[1], v[2], v[3]);
  }
};
template <> struct Row16<__nv_bfloat16> {
  static constexpr int VEC = 8;
  __device__ static __forceinline__ void load(const __nv_bfloat16 *p, float (&v)[8]) {
    uint4 x = __ldg(reinterpret_cast<const uint4 *>(p));
    const uint32_t w[4] = {x.x, x.y, x.z, x.w};
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      v[2 * i] = __uint_as_float(w[i] << 16);
      v[2 * i + 1] = __uint_as_float(w[i] & 0xffff0000u);
    }
  }
  __device__ static __forceinline__ void store(__nv_bfloat16 *p, const float (&v)[8]) {
    uint32_t w[4];
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      __nv_bfloat162 h = __floats2bfloat162_rn(v[2 * i], v[2 * i + 1]);
      w[i] = *reinterpret_cast<uint32_t *>(&h);
    }
    *reinterpret_cast<uint4 *>(p) = make_uint4(w[0], w[1], w[2], w[3]);
  }
};

__device__ __forceinline__ float act_apply(float x, int act) {
  if (act == IT_ACT_RELU) return fmaxf(x, 0.f);
  if (act == IT_ACT_ELU) return x > 0.f ? x : expm1f(x);
  return x;
}

struct GatherParams {
  const int64_t *__restrict__ shadow_indptr;
  const int32_t *__restrict__ indices;
  const float *__restrict__ weights;
  const int32_t *__restrict__ bucket_rows;
  const int32_t *__restrict__ row_dest;
  const void *__restrict__ src;
  float *__restrict__ partials;
  void *__restrict__ dst;
  const float *__restrict__ self_term;
  int64_t row_lo, row_hi;  // range inside bucket_rows
  int dim;
  int is_mean, epi, act;
};

// Aggregate edges [j0, j1) into acc[] (per lane: its 16-byte column slice, for its slot).
// All GROUP lanes of the group call this together with the same j0, j1.
template <typename T, int LPR, int GROUP, bool IS_MAX, bool WEIGHTED>
__device__ __forceinline__ void gather_edges(const GatherParams &p, int64_t j0, int64_t j1, unsigned group_mask,
                                             int t /*lane in group*/, float (&acc)[Row16<T>::VEC]) {
  constexpr int VEC = Row16<T>::VEC;
  constexpr int SLOTS = GROUP / LPR;
  const int slot = t / LPR;
  const int col = (t % LPR) * VEC;
  const T *__restrict__ src = reinterpret_cast<const T *>(p.src);
  for (int64_t base = j0; base < j1; base += GROUP) {
    const int64_t mine = base + t;
    int32_t my_idx = 0;
    float my_w = 1.f;
    if (mine < j1) {
      my_idx = __ldg(p.indices + mine);
      if (WEIGHTED) my_w = __ldg(p.weights + mine);
    }
    const int cnt = (int)((j1 - base) < (int64_t)GROUP ? (j1 - base) : (int64_t)GROUP);
    for (int k0 = 0; k0 < cnt; k0 += SLOTS * UNROLL) {
      float v[UNROLL][VEC];
      float w[UNROLL];
      bool ok[UNROLL];
#pragma unroll
      for (int u = 0; u < UNROLL; ++u) {
        const int e = k0 + u * SLOTS + slot;
        const int32_t s = __shfl_sync(group_mask, my_idx, e & (GROUP - 1), GROUP);
        w[u] = WEIGHTED ? __shfl_sync(group_mask, my_w, e & (GROUP - 1), GROUP) : 1.f;
        ok[u] = e < cnt;
        if (ok[u]) Row16<T>::load(src + (int64_t)s * p.dim + col, v[u]);
      }
#pragma unroll
      for (int u = 0; u < UNROLL; ++u) {
        if (ok[u]) {
#pragma unroll
          for (int i = 0; i < VEC; ++i) {
            if (IS_MAX) acc[i] = fmaxf(acc[i], WEIGHTED ? w[u] * v[u][i] : v[u][i]);
            else acc[i] = WEIGHTED ? fmaf(w[u], v[u][i], acc[i]) : acc[i] + v[u][i];
          }
        }
      }
    }
  }
}

// Fold the SLOTS partial accumulators of a group into slot 0 (fixed order).
template <int LPR, int GROUP, bool IS_MAX, int VEC>
__device__ __forceinline__ void fold_slots(unsigned group_mask, float (&acc)[VEC]) {
#pragma unroll
  for (int o = GROUP / 2; o >= LPR; o >>= 1) {
#pragma unroll
    for (int i = 0; i < VEC; ++i) {
      float y = __shfl_xor_sync(group_mask, acc[i], o, GROUP);
      acc[i] = IS_MAX ? fmaxf(acc[i], y) : acc[i] + y;
    }
  }
}

// Write the aggregate of shadow row r (held by the LPR lanes of slot 0).
template <typename T, bool IS_MAX>
__device__ __forceinline__ void finish_row(const GatherParams &p, int32_t r, int64_t len, int col,
                                           float (&acc)[Row16<T>::VEC]) {
  constexpr int VEC = Row16<T>::VEC;
  if (IS_MAX && len == 0) {
#pragma unroll
    for (int i = 0; i < VEC; ++i) acc[i] = 0.f;
  }
  const int32_t dest = __ldg(p.row_dest + r);
  if (dest < 0) {  // a group of a split vertex: raw partial, finished by the combine kernel
    float *q = p.partials + (int64_t)(~dest) * p.dim + col;
#pragma unroll
    for (int i = 0; i < VEC; i += 4)
      *reinterpret_cast<float4 *>(q + i) = make_float4(acc[i], acc[i + 1], acc[i + 2], acc[i + 3]);
    return;
  }
  if (p.is_mean && len > 0) {
    const float inv = 1.f / (float)len;
#pragma unroll
    for (int i = 0; i < VEC; ++i) acc[i] *= inv;
  }
  const int64_t off = (int64_t)dest * p.dim + col;
  if (p.epi == IT_EPI_ADD_ACT) {
#pragma unroll
    for (int i = 0; i < VEC; i += 4) {
      float4 s = __ldg(reinterpret_cast<const float4 *>(p.self_term + off + i));
      acc[i] = act_apply(acc[i] + s.x, p.act);
      acc[i + 1] = act_apply(acc[i + 1] + s.y, p.act);
      acc[i + 2] = act_apply(acc[i + 2] + s.z, p.act);
      acc[i + 3] = act_apply(acc[i + 3] + s.w, p.act);
    }
  }
  Row16<T>::store(reinterpret_cast<T *>(p.dst) + off, acc);
}

// One group of GROUP lanes per shadow row; groups stride over the bucket's row list.
template <typename T, int LPR, int GROUP, bool IS_MAX, bool WEIGHTED>
__global__ void __launch_bounds__(GATHER_THREADS) gather_group_kernel(GatherParams p) {
  constexpr int VEC = Row16<T>::VEC;
  const int lane = threadIdx.x & 31;
  const int t = lane % GROUP;
  const unsigned group_mask = (GROUP == 32) ? 0xffffffffu : (((1u << (GROUP & 31)) - 1u) << (lane - t));
  const int64_t groups_total = (int64_t)gridDim.x * (GATHER_THREADS / GROUP);
  const int64_t group_id = (int64_t)blockIdx.x * (GATHER_THREADS / GROUP) + threadIdx.x / GROUP;
  for (int64_t i = p.row_lo + group_id; i < p.row_hi; i += groups_total) {
    const int32_t r = __ldg(p.bucket_rows + i);
    const int64_t j0 = __ldg(p.shadow_indptr + r), j1 = __ldg(p.shadow_indptr + r + 1);
    float acc[VEC];
#pragma unroll
    for (int k = 0; k < VEC; ++k) acc[k] = IS_MAX ? -INFINITY : 0.f;
    gather_edges<T, LPR, GROUP, IS_MAX, WEIGHTED>(p, j0, j1, group_mask, t, acc);
    fold_slots<LPR, GROUP, IS_MAX, VEC>(group_mask, acc);
    if (t < LPR) finish_row<T, IS_MAX>(p, r, j1 - j0, t * VEC, acc);
  }
}

// One CTA per long shadow row: warp w takes the w-th contiguous chunk (a multiple of 32
// edges), the warp results are folded in warp order through shared memory.
template <typename T, int LPR, bool IS_MAX, bool WEIGHTED>
__global__ void __launch_bounds__(GATHER_THREADS) gather_cta_kernel(GatherParams p) {
  constexpr int VEC = Row16<T>::VEC;
  constexpr int WARPS = GATHER_THREADS / 32;
  __shared__ float red[WARPS][LPR * VEC];
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  for (int64_t i = p.row_lo + blockIdx.x; i < p.row_hi; i += gridDim.x) {
    const int32_t r = __ldg(p.bucket_rows + i);
    const int64_t j0 = __ldg(p.shadow_indptr + r), j1 = __ldg(p.shadow_indptr + r + 1);
    const int64_t len = j1 - j0;
    int64_t chunk = (len + WARPS - 1) / WARPS;
    chunk = (chunk + 31) / 32 * 32;
    int64_t a = j0 + warp * chunk, b = a + chunk;
    if (a > j1) a = j1;
    if (b > j1) b = j1;
    float acc[VEC];
#pragma unroll
    for (int k = 0; k < VEC; ++k) acc[k] = IS_MAX ? -INFINITY : 0.f;
    gather_edges<T, LPR, 32, IS_MAX, WEIGHTED>(p, a, b, 0xffffffffu, lane, acc);
    fold_slots<LPR, 32, IS_MAX, VEC>(0xffffffffu, acc);
    __syncthreads();  // red[] free again
    if (lane < LPR) {
#pragma unroll
      for (int k = 0; k < VEC; ++k) red[warp][lane * VEC + k] = acc[k];
    }
    __syncthreads();
    if (warp == 0 && lane < LPR) {
#pragma unroll
      for (int w = 1; w < WARPS; ++w) {
#pragma unroll
        for (int k = 0; k < VEC; ++k) {
          float y = red[w][lane * VEC + k];
          acc[k] = IS_MAX ? fmaxf(acc[k], y) : acc[k] + y;
        }
      }
      finish_row<T, IS_MAX>(p, r, len, lane * VEC, acc);
    }
  }
}

// Combine: one group of LPR32 = dim / 4 lanes (fp32 partial rows) ... one warp per split owner.
// Partial rows of owner k are rows [p0, p0 + n_k) of the partial buffer, folded in group order.
struct CombineParams {
  const int32_t *__restrict__ split_owners;
  const int64_t *__restrict__ owner_indptr;
  const int64_t *__restrict__ shadow_indptr;
  const float *__restrict__ partials;
  void *__restrict__ dst;
  const float *__restrict__ self_term;
  int64_t n_split_owners;
  int dim;
  int is_max, is_mean, epi, act;
};

template <typename T>
__global__ void __launch_bounds__(GATHER_THREADS) combine_kernel(CombineParams p) {
  const int lane = threadIdx.x & 31;
  const int64_t warps_total = (int64_t)gridDim.x * (GATHER_THREADS / 32);
  for (int64_t k = (int64_t)blockIdx.x * (GATHER_THREADS / 32) + (threadIdx.x >> 5); k < p.n_split_owners; k += warps_total) {
    const int64_t v = __ldg(p.split_owners + k);
    const int64_t r0 = __ldg(p.owner_indptr + v), r1 = __ldg(p.owner_indptr + v + 1);
    const int64_t p0 = r0 - v + k;
    const int64_t deg = __ldg(p.shadow_indptr + r1) - __ldg(p.shadow_indptr + r0);
    const float inv = (p.is_mean && deg > 0) ? 1.f / (float)deg : 1.f;
    for (int c = lane * 4; c < p.dim; c += 128) {
      float4 acc = __ldg(reinterpret_cast<const float4 *>(p.partials + p0 * p.dim + c));
      for (int64_t g = 1; g < r1 - r0; ++g) {
        float4 y = __ldg(reinterpret_cast<const float4 *>(p.partials + (p0 + g) * p.dim + c));
        if (p.is_max) {
          acc.x = fmaxf(acc.x, y.x); acc.y = fmaxf(acc.y, y.y); acc.z = fmaxf(acc.z, y.z); acc.w = fmaxf(acc.w, y.w);
        } else {
          acc.x += y.x; acc.y += y.y; acc.z += y.z; acc.w += y.w;
        }
      }
      float o[4] = {acc.x * inv, acc.y * inv, acc.z * inv, acc.w * inv};
      const int64_t off = v * p.dim + c;
      if (p.epi == IT_EPI_ADD_ACT) {
        float4 s = __ldg(reinterpret_cast<const float4 *>(p.self_term + off));
        o[0] = act_apply(o[0] + s.x, p.act); o[1] = act_apply(o[1] + s.y, p.act);
        o[2] = act_apply(o[2] + s.z, p.act); o[3] = act_apply(o[3] + s.w, p.act);
      }
      T *d = reinterpret_cast<T *>(p.dst) + off;
      if (sizeof(T) == 4) {
        *reinterpret_cast<float4 *>(d) = make_float4(o[0], o[1], o[2], o[3]);
      } else {
        __nv_bfloat162 h0 = __floats2bfloat162_rn(o[0], o[1]), h1 = __floats2bfloat162_rn(o[2], o[3]);
        *reinterpret_cast<uint2 *>(d) = make_uint2(*reinterpret_cast<uint32_t *>(&h0), *reinterpret_cast<uint32_t *>(&h1));
      }
    }
  }
}

// ----------------------------------------------------------------------------- dispatch
template <typename T, int LPR, bool IS_MAX, bool WEIGHTED>
it_status launch_buckets(const it_graph *g, GatherParams p, cudaStream_t st) {
  // longest rows first so that the tail of the launch sequence is made of short rows
  for (int b = g->n_buckets - 1; b >= 0; --b) {
    const int64_t lo = g->h_bucket_offsets[b], hi = g->h_bucket_offsets[b + 1];
    if (hi <= lo) continue;
    p.row_lo = lo; p.row_hi = hi;
    const int64_t bound = g->bucket_bounds[b];
    const int64_t rows = hi - lo;
    const int64_t max_blocks = (int64_t)g->num_sms * 8;
    // algorithmic bytes: per edge the index, the optional weight and one source row; per row its
    // two bounds, its id and destination, and one output row (plus the self row it is added to)
    const double row_bytes = (double)p.dim * sizeof(T);
    const double bytes = (double)g->h_bucket_edges[b] * (4.0 + (WEIGHTED ? 4.0 : 0.0) + row_bytes) +
                         (double)rows * (16.0 + 8.0 + row_bytes + (p.epi == IT_EPI_ADD_ACT ? 4.0 * p.dim : 0.0));
    if (bound > 256) {
      unsigned blocks = (unsigned)(rows < max_blocks ? rows : max_blocks);
      IT_LAUNCH(IT_K_GATHER_CTA, bytes, 0, st, gather_cta_kernel<T, LPR, IS_MAX, WEIGHTED><<<blocks, GATHER_THREADS, 0, st>>>(p));
    } else if (bound > 8 || LPR == 32) {
      int64_t want = (rows + (GATHER_THREADS / 32) - 1) / (GATHER_THREADS / 32);
      unsigned blocks = (unsigned)(want < max_blocks ? want : max_blocks);
      IT_LAUNCH(IT_K_GATHER_WARP, bytes, 0, st, gather_group_kernel<T, LPR, 32, IS_MAX, WEIGHTED><<<blocks, GATHER_THREADS, 0, st>>>(p));
    } else {
      int64_t want = (rows + (GATHER_THREADS / LPR) - 1) / (GATHER_THREADS / LPR);
      unsigned blocks = (unsigned)(want < max_blocks ? want : max_blocks);
      IT_LAUNCH(IT_K_GATHER_SUBWARP, bytes, 0, st, gather_group_kernel<T, LPR, LPR, IS_MAX, WEIGHTED><<<blocks, GATHER_THREADS, 0, st>>>(p));
    }
  }
  IT_CUDA_TRY(cudaGetLastError());
  return IT_OK;
}

template <typename T, int LPR>
it_status launch_ops(const it_gather_args &a, GatherParams p, cudaStream_t st) {
  const bool mx = a.op == IT_GATHER_MAX, w = a.use_edge_weights != 0;
  if (mx) return w ? launch_buckets<T, LPR, true, true>(a.g, p, st) : launch_buckets<T, LPR, true, false>(a.g, p, st);
  return w ? launch_buckets<T, LPR, false, true>(a.g, p, st) : launch_buckets<T, LPR, false, false>(a.g, p, st);
}

template <typename T>
it_status launch_lpr(const it_gather_args &a, GatherParams p, cudaStream_t st) {
  const int lpr = a.dim * (int)sizeof(T) / 16;
  switch (lpr) {
    case 1: return launch_ops<T, 1>(a, p, st);
    case 2: return launch_ops<T, 2>(a, p, st);
    case 4: return launch_ops<T, 4>(a, p, st);
    case 8: return launch_ops<T, 8>(a, p, st);
    case 16: return launch_ops<T, 16>(a, p, st);
    case 32: return launch_ops<T, 32>(a, p, st);
  }
  it_set_error("gather: row of %d x %d bytes is not 16, 32, 64, 128, 256 or 512 bytes", a.dim, (int)sizeof(T));
  return IT_ERR_UNSUPPORTED;
}

}  // namespace

it_status it_launch_gather(const it_gather_args &a, cudaStream_t st) {
  const it_graph *g = a.g;
  IT_REQUIRE(a.op == IT_GATHER_SUM || a.op == IT_GATHER_MEAN || a.op == IT_GATHER_MAX, IT_ERR_INVALID_ARG, "gather: bad op");
  IT_REQUIRE(!a.use_edge_weights || g->edge_weights, IT_ERR_INVALID_ARG, "layer uses edge weights but the graph has none");
  IT_REQUIRE(g->n_partial_rows == 0 || a.partials, IT_ERR_WORKSPACE, "gather: no partial buffer");
  if (g->n == 0) return IT_OK;
  GatherParams p;
  p.shadow_indptr = g->shadow_indptr; p.indices = g->indices; p.weights = g->edge_weights;
  p.bucket_rows = g->bucket_rows; p.row_dest = g->row_dest; p.src = a.src; p.partials = a.partials;
  p.dst = a.dst; p.self_term = a.self_term; p.row_lo = p.row_hi = 0; p.dim = a.dim;
  p.is_mean = a.op == IT_GATHER_MEAN; p.epi = a.epi; p.act = a.act;
  if (a.dtype == IT_F32) IT_TRY(launch_lpr<float>(a, p, st));
  else IT_TRY(launch_lpr<__nv_bfloat16>(a, p, st));
  if (g->n_split_owners > 0) {
    CombineParams c;
    c.split_owners = g->split_owners; c.owner_indptr = g->owner_indptr; c.shadow_indptr = g->shadow_indptr;
    c.partials = a.partials; c.dst = a.dst; c.self_term = a.self_term; c.n_split_owners = g->n_split_owners;
    c.dim = a.dim; c.is_max = a.op == IT_GATHER_MAX; c.is_mean = a.op == IT_GATHER_MEAN; c.epi = a.epi; c.act = a.act;
    int64_t want = (g->n_split_owners + 7) / 8;
    int64_t cap = (int64_t)g->num_sms * 8;
    unsigned blocks = (unsigned)(want < cap ? want : cap);
    const double cbytes = (double)g->n_partial_rows * a.dim * 4.0 +
                          (double)g->n_split_owners * a.dim * (a.dtype == IT_F32 ? 4.0 : 2.0);
    if (a.dtype == IT_F32) IT_LAUNCH(IT_K_COMBINE, cbytes, 0, st, combine_kernel<float><<<blocks, GATHER_THREADS, 0, st>>>(c));
    else IT_LAUNCH(IT_K_COMBINE, cbytes, 0, st, combine_kernel<__nv_bfloat16><<<blocks, GATHER_THREADS, 0, st>>>(c));
    IT_CUDA_TRY(cudaGetLastError());
  }
  return IT_OK;
}
