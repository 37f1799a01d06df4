// GAT reduce: per destination and head, e = LeakyReLU(s_src[u] + s_dst[v]), softmax over the
// in-edges, attention-weighted sum of the source rows z_u, then bias and activation.
// One pass over the edges with a running (max, sum, weighted accumulator) state per lane
// ("online" softmax); states of different edge slots / warps are merged in a fixed order.
// HBM-bound like the plain gather: one 16-byte row slice + one 4-byte score per lane per edge.
#include "common.cuh"

namespace {

constexpr int GAT_THREADS = 256;
constexpr int GAT_UNROLL = 4;

template <typename T> struct Vec16;
template <> struct Vec16<float> {
  static constexpr int VEC = 4;
  __device__ static __forceinline__ void load(const float *p, float (&v)[4]) {
    float4 x = __ldg(reinterpret_cast<const float4 *>(p));
    v[0] = x.x; v[1] = x.y; v[2] = x.z; v[3] = x.w;
  }
  __device__ static __forceinline__ void store(float *p, const float (&v)[4]) {
    *reinterpret_cast<float4 *>(p) = make_float4(v[0], v[1], v[2], v[3]);
  }
};
template <> struct Vec16<__nv_bfloat16> {
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

struct GatParams {
  const int64_t *__restrict__ shadow_indptr;
  const int32_t *__restrict__ indices;
  const int32_t *__restrict__ bucket_rows;
  const int32_t *__restrict__ row_dest;
  const void *__restrict__ z;
  const float *__restrict__ scores;  // [n, 2*heads]: source scores, then destination scores
  const float *__restrict__ bias;
  void *__restrict__ dst;
  int64_t row_lo, row_hi;
  int dim, heads, head_dim, act;
  float slope;
};

template <int VEC> struct SoftState {
  float m, l, acc[VEC];
  __device__ __forceinline__ void init() {
    m = -INFINITY; l = 0.f;
#pragma unroll
    for (int i = 0; i < VEC; ++i) acc[i] = 0.f;
  }
  // merge another state (m2, l2, acc2) into this one
  __device__ __forceinline__ void merge(float m2, float l2, const float (&a2)[VEC]) {
    const float mn = fmaxf(m, m2);
    const float f1 = (m == -INFINITY) ? 0.f : __expf(m - mn);
    const float f2 = (m2 == -INFINITY) ? 0.f : __expf(m2 - mn);
    l = l * f1 + l2 * f2;
#pragma unroll
    for (int i = 0; i < VEC; ++i) acc[i] = acc[i] * f1 + a2[i] * f2;
    m = mn;
  }
};

template <typename T, int LPR, int GROUP>
__device__ __forceinline__ void gat_edges(const GatParams &p, int64_t j0, int64_t j1, unsigned group_mask, int t,
                                          float s_dst, SoftState<Vec16<T>::VEC> &st) {
  constexpr int VEC = Vec16<T>::VEC;
  constexpr int SLOTS = GROUP / LPR;
  const int slot = t / LPR;
  const int col = (t % LPR) * VEC;
  const int head = col / p.head_dim;
  const int sstride = 2 * p.heads;
  const T *__restrict__ z = reinterpret_cast<const T *>(p.z);
  for (int64_t base = j0; base < j1; base += GROUP) {
    const int64_t mine = base + t;
    const int32_t my_idx = mine < j1 ? __ldg(p.indices + mine) : 0;
    const int cnt = (int)((j1 - base) < (int64_t)GROUP ? (j1 - base) : (int64_t)GROUP);
    for (int k0 = 0; k0 < cnt; k0 += SLOTS * GAT_UNROLL) {
      float v[GAT_UNROLL][VEC];
      float e[GAT_UNROLL];
      float mx = st.m;
#pragma unroll
      for (int u = 0; u < GAT_UNROLL; ++u) {
        const int ei = k0 + u * SLOTS + slot;
        const int32_t s = __shfl_sync(group_mask, my_idx, ei & (GROUP - 1), GROUP);
        e[u] = -INFINITY;
        if (ei < cnt) {
          Vec16<T>::load(z + (int64_t)s * p.dim + col, v[u]);
          const float x = __ldg(p.scores + (int64_t)s * sstride + head) + s_dst;
          e[u] = x > 0.f ? x : p.slope * x;
        }
      }
#pragma unroll
      for (int u = 0; u < GAT_UNROLL; ++u) mx = fmaxf(mx, e[u]);
      if (mx == -INFINITY) continue;  // this slot saw no edge yet
      const float scale = (st.m == -INFINITY) ? 0.f : __expf(st.m - mx);
      st.l *= scale;
#pragma unroll
      for (int i = 0; i < VEC; ++i) st.acc[i] *= scale;
      st.m = mx;
#pragma unroll
      for (int u = 0; u < GAT_UNROLL; ++u) {
        if (e[u] != -INFINITY) {
          const float pw = __expf(e[u] - mx);
          st.l += pw;
#pragma unroll
          for (int i = 0; i < VEC; ++i) st.acc[i] = fmaf(pw, v[u][i], st.acc[i]);
        }
      }
    }
  }
}

template <int LPR, int GROUP, int VEC>
__device__ __forceinline__ void fold_states(unsigned group_mask, SoftState<VEC> &st) {
#pragma unroll
  for (int o = GROUP / 2; o >= LPR; o >>= 1) {
    const float m2 = __shfl_xor_sync(group_mask, st.m, o, GROUP);
    const float l2 = __shfl_xor_sync(group_mask, st.l, o, GROUP);
    float a2[VEC];
#pragma unroll
    for (int i = 0; i < VEC; ++i) a2[i] = __shfl_xor_sync(group_mask, st.acc[i], o, GROUP);
    // only slot 0 is read at the end, and it is always the first operand: the order is fixed
    st.merge(m2, l2, a2);
  }
}

template <typename T>
__device__ __forceinline__ void gat_finish(const GatParams &p, int64_t v, int col, SoftState<Vec16<T>::VEC> &st) {
  constexpr int VEC = Vec16<T>::VEC;
  const float inv = st.l > 0.f ? 1.f / st.l : 0.f;
  float o[VEC];
#pragma unroll
  for (int i = 0; i < VEC; ++i) {
    float x = st.acc[i] * inv;
    if (p.bias) x += __ldg(p.bias + col + i);
    o[i] = act_apply(x, p.act);
  }
  Vec16<T>::store(reinterpret_cast<T *>(p.dst) + v * p.dim + col, o);
}

template <typename T, int LPR, int GROUP>
__global__ void __launch_bounds__(GAT_THREADS) gat_group_kernel(GatParams p) {
  constexpr int VEC = Vec16<T>::VEC;
  const int lane = threadIdx.x & 31;
  const int t = lane % GROUP;
  const unsigned group_mask = (GROUP == 32) ? 0xffffffffu : (((1u << (GROUP & 31)) - 1u) << (lane - t));
  const int64_t groups_total = (int64_t)gridDim.x * (GAT_THREADS / GROUP);
  const int64_t group_id = (int64_t)blockIdx.x * (GAT_THREADS / GROUP) + threadIdx.x / GROUP;
  const int col = (t % LPR) * VEC;
  const int head = col / p.head_dim;
  for (int64_t i = p.row_lo + group_id; i < p.row_hi; i += groups_total) {
    const int32_t r = __ldg(p.bucket_rows + i);
    const int64_t v = __ldg(p.row_dest + r);  // graph is unsplit: row == vertex
    const int64_t j0 = __ldg(p.shadow_indptr + r), j1 = __ldg(p.shadow_indptr + r + 1);
    const float s_dst = __ldg(p.scores + v * 2 * p.heads + p.heads + head);
    SoftState<VEC> st;
    st.init();
    gat_edges<T, LPR, GROUP>(p, j0, j1, group_mask, t, s_dst, st);
    fold_states<LPR, GROUP, VEC>(group_mask, st);
    if (t < LPR) gat_finish<T>(p, v, col, st);
  }
}

template <typename T, int LPR>
__global__ void __launch_bounds__(GAT_THREADS) gat_cta_kernel(GatParams p) {
  constexpr int VEC = Vec16<T>::VEC;
  constexpr int WARPS = GAT_THREADS / 32;
  __shared__ float red[WARPS][LPR][VEC + 2];
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int col = (lane % LPR) * VEC;
  const int head = col / p.head_dim;
  for (int64_t i = p.row_lo + blockIdx.x; i < p.row_hi; i += gridDim.x) {
    const int32_t r = __ldg(p.bucket_rows + i);
    const int64_t v = __ldg(p.row_dest + r);
    const int64_t j0 = __ldg(p.shadow_indptr + r), j1 = __ldg(p.shadow_indptr + r + 1);
    const float s_dst = __ldg(p.scores + v * 2 * p.heads + p.heads + head);
    int64_t chunk = (j1 - j0 + WARPS - 1) / WARPS;
    chunk = (chunk + 31) / 32 * 32;
    int64_t a = j0 + warp * chunk, b = a + chunk;
    if (a > j1) a = j1;
    if (b > j1) b = j1;
    SoftState<VEC> st;
    st.init();
    gat_edges<T, LPR, 32>(p, a, b, 0xffffffffu, lane, s_dst, st);
    fold_states<LPR, 32, VEC>(0xffffffffu, st);
    __syncthreads();
    if (lane < LPR) {
      red[warp][lane][0] = st.m; red[warp][lane][1] = st.l;
#pragma unroll
      for (int k = 0; k < VEC; ++k) red[warp][lane][2 + k] = st.acc[k];
    }
    __syncthreads();
    if (warp == 0 && lane < LPR) {
      for (int w = 1; w < WARPS; ++w) {
        float a2[VEC];
#pragma unroll
        for (int k = 0; k < VEC; ++k) a2[k] = red[w][lane][2 + k];
        st.merge(red[w][lane][0], red[w][lane][1], a2);
      }
      gat_finish<T>(p, v, col, st);
    }
  }
}

template <typename T, int LPR>
it_status launch_buckets(const it_graph *g, GatParams p, cudaStream_t st) {
  for (int b = g->n_buckets - 1; b >= 0; --b) {
    const int64_t lo = g->h_bucket_offsets[b], hi = g->h_bucket_offsets[b + 1];
    if (hi <= lo) continue;
    p.row_lo = lo; p.row_hi = hi;
    const int64_t bound = g->bucket_bounds[b], rows = hi - lo;
    const int64_t max_blocks = (int64_t)g->num_sms * 8;
    // algorithmic bytes: per edge the index, one source score per head and one source row; per
    // row its bounds, id, destination scores and one output row
    const double row_bytes = (double)p.dim * sizeof(T);
    const double bytes = (double)g->h_bucket_edges[b] * (4.0 + 4.0 * p.heads + row_bytes) +
                         (double)rows * (16.0 + 8.0 + 4.0 * p.heads + row_bytes);
    if (bound > 256) {
      unsigned blocks = (unsigned)(rows < max_blocks ? rows : max_blocks);
      IT_LAUNCH(IT_K_GAT_CTA, bytes, 0, st, gat_cta_kernel<T, LPR><<<blocks, GAT_THREADS, 0, st>>>(p));
    } else if (bound > 8 || LPR == 32) {
      int64_t want = (rows + (GAT_THREADS / 32) - 1) / (GAT_THREADS / 32);
      unsigned blocks = (unsigned)(want < max_blocks ? want : max_blocks);
      IT_LAUNCH(IT_K_GAT_WARP, bytes, 0, st, gat_group_kernel<T, LPR, 32><<<blocks, GAT_THREADS, 0, st>>>(p));
    } else {
      int64_t want = (rows + (GAT_THREADS / LPR) - 1) / (GAT_THREADS / LPR);
      unsigned blocks = (unsigned)(want < max_blocks ? want : max_blocks);
      IT_LAUNCH(IT_K_GAT_SUBWARP, bytes, 0, st, gat_group_kernel<T, LPR, LPR><<<blocks, GAT_THREADS, 0, st>>>(p));
    }
  }
  IT_CUDA_TRY(cudaGetLastError());
  return IT_OK;
}

template <typename T>
it_status launch_lpr(const it_gat_args &a, GatParams p, cudaStream_t st) {
  const int lpr = a.heads * a.head_dim * (int)sizeof(T) / 16;
  switch (lpr) {
    case 1: return launch_buckets<T, 1>(a.g, p, st);
    case 2: return launch_buckets<T, 2>(a.g, p, st);
    case 4: return launch_buckets<T, 4>(a.g, p, st);
    case 8: return launch_buckets<T, 8>(a.g, p, st);
    case 16: return launch_buckets<T, 16>(a.g, p, st);
    case 32: return launch_buckets<T, 32>(a.g, p, st);
  }
  it_set_error("gat: row of %d bytes is not 16, 32, 64, 128, 256 or 512 bytes", a.heads * a.head_dim * (int)sizeof(T));
  return IT_ERR_UNSUPPORTED;
}

}  // namespace

it_status it_launch_gat(const it_gat_args &a, cudaStream_t st) {
  const it_graph *g = a.g;
  IT_REQUIRE(g->n_split_owners == 0, IT_ERR_UNSUPPORTED,
             "GAT layers run on an unsplit graph (attention is reduced in apply_node, not by partial gather)");
  const int vec = a.dtype == IT_F32 ? 4 : 8;
  IT_REQUIRE(a.head_dim % vec == 0, IT_ERR_UNSUPPORTED, "gat: head_dim must be a multiple of %d", vec);
  if (g->n == 0) return IT_OK;
  GatParams p;
  p.shadow_indptr = g->shadow_indptr; p.indices = g->indices; p.bucket_rows = g->bucket_rows; p.row_dest = g->row_dest;
  p.z = a.z; p.scores = a.scores; p.bias = a.bias; p.dst = a.dst; p.row_lo = p.row_hi = 0;
  p.dim = a.heads * a.head_dim; p.heads = a.heads; p.head_dim = a.head_dim; p.act = a.act; p.slope = a.slope;
  return a.dtype == IT_F32 ? launch_lpr<float>(a, p, st) : launch_lpr<__nv_bfloat16>(a, p, st);
}
