// GAT reduce: per destination and head, e = LeakyReLU(s_src[u] + s_dst[v]), softmax over the
// in-edges, attention-weighted sum of the source rows z_u, then bias and activation.
// One pass over the edges with a running (max, sum, weighted accumulator) state per lane
// ("online" softmax).  Such states merge associatively — (m, l, acc) and (m', l', acc') give
// M = max(m, m'), l e^(m-M) + l' e^(m'-M), acc e^(m-M) + acc' e^(m'-M) — so the groups of a split
// hub are reduced independently into partial states and merged in group order, exactly like
// the partial sums of the plain gather.  The edge streaming lives in stream.cuh.
#include "stream.cuh"

namespace {

using namespace it_stream;

__host__ __device__ inline int gat_partial_stride(int dim, int heads) { return dim + ((2 * heads + 3) / 4) * 4; }

template <typename T, int SB>
struct GatPolicy {
  using Slice = RowSlice<T, SB>;
  static constexpr int VEC = Slice::VEC;
  static constexpr int NS = VEC + 2;   // accumulators, running max, running sum
  static constexpr bool WEIGHTED = false, HAS_EXTRA = true, NEEDS_OWNER = true;
  const float *__restrict__ scores;    // [n_src, 2*heads]: source scores of the vertex, then its destination scores
  const float *__restrict__ scores_dst;   // the same rows, counted from the first local destination
  const float *__restrict__ bias;
  void *__restrict__ dst;
  float *__restrict__ partials;        // [n_partial_rows, stride]: acc[dim], m[heads], l[heads]
  int dim, heads, head_dim, act;
  int src_stride;                      // floats from one row of `scores` to the next (2*heads; heads when the rows are per edge)
  float slope;
  // per-thread
  int col, head;
  float s_dst;

  __device__ __forceinline__ void setup(int t) { col = t * VEC; head = col / head_dim; s_dst = 0.f; }
  __device__ __forceinline__ void init(float (&st)[NS]) const {
#pragma unroll
    for (int k = 0; k < VEC; ++k) st[k] = 0.f;
    st[VEC] = -INFINITY;
    st[VEC + 1] = 0.f;
  }
  __device__ __forceinline__ float extra(uint32_t s) const { return __ldg(scores + (uint64_t)s * src_stride + head); }
  __device__ __forceinline__ const float *extra_ptr(uint32_t s) const { return scores + (uint64_t)s * src_stride + head; }
  __device__ __forceinline__ void edge(float (&st)[NS], const typename Slice::Raw &raw, float, float x) const {
    float e = x + s_dst;
    e = e > 0.f ? e : slope * e;
    // One exponential per edge: of the two factors exp(m - m_new) and exp(e - m_new) one is exp(0) = 1 and the other is
    // exp(-|e - m|).  (First edge: m = -inf, the old state is scaled by exp(-inf) = 0.)
    const float d = e - st[VEC];
    const float t = __expf(-fabsf(d));
    const bool up = d > 0.f;
    const float scale = up ? t : 1.f, pw = up ? 1.f : t;
    const float m_new = up ? e : st[VEC];
    float f[VEC];
    Slice::unpack(raw, f);
    if constexpr (VEC % 2 == 0) {
#pragma unroll
      for (int k = 0; k < VEC; k += 2) scale_fma_f32x2(st[k], st[k + 1], scale, pw, f[k], f[k + 1]);
    } else {
#pragma unroll
      for (int k = 0; k < VEC; ++k) st[k] = fmaf(pw, f[k], st[k] * scale);
    }
    st[VEC + 1] = fmaf(st[VEC + 1], scale, pw);
    st[VEC] = m_new;
  }
  __device__ __forceinline__ void merge(float (&st)[NS], const float (&o)[NS]) const {
    const float m_new = fmaxf(st[VEC], o[VEC]);
    const float f1 = st[VEC] == -INFINITY ? 0.f : __expf(st[VEC] - m_new);
    const float f2 = o[VEC] == -INFINITY ? 0.f : __expf(o[VEC] - m_new);
#pragma unroll
    for (int k = 0; k < VEC; ++k) st[k] = st[k] * f1 + o[k] * f2;
    st[VEC + 1] = st[VEC + 1] * f1 + o[VEC + 1] * f2;
    st[VEC] = m_new;
  }
  __device__ __forceinline__ void begin_row(int32_t, int32_t owner) {
    s_dst = __ldg(scores_dst + (int64_t)owner * (2 * heads) + heads + head);
  }
  __device__ __forceinline__ void end_row(float (&st)[NS], int32_t dest, int32_t, int64_t) const {
    if (dest < 0) {   // a group of a split vertex: its state goes to the partial buffer
      float *q = partials + (int64_t)(~dest) * gat_partial_stride(dim, heads);
      float a[VEC];
#pragma unroll
      for (int i = 0; i < VEC; ++i) a[i] = st[i];
      store_floats<VEC>(q + col, a);
      if (col % head_dim == 0) {
        q[dim + head] = st[VEC];
        q[dim + heads + head] = st[VEC + 1];
      }
      return;
    }
    const float inv = st[VEC + 1] > 0.f ? 1.f / st[VEC + 1] : 0.f;
    float o[VEC];
#pragma unroll
    for (int i = 0; i < VEC; ++i) o[i] = act_apply(st[i] * inv + (bias ? __ldg(bias + col + i) : 0.f), act);
    Slice::store(reinterpret_cast<T *>(dst) + (int64_t)dest * dim + col, o);
  }
};

// Merge the partial states of every split vertex in group order; one warp per vertex.
struct GatCombineParams {
  const int32_t *__restrict__ split_owners;
  const int64_t *__restrict__ owner_indptr;
  const float *__restrict__ partials;
  const float *__restrict__ bias;
  void *__restrict__ dst;
  int64_t n_split_owners;
  int dim, heads, head_dim, act;
};

template <typename T>
__global__ void __launch_bounds__(THREADS) gat_combine_kernel(GatCombineParams p) {
  const int lane = threadIdx.x & 31;
  const int stride = gat_partial_stride(p.dim, p.heads);
  const int64_t warps_total = (int64_t)gridDim.x * (THREADS / 32);
  for (int64_t k = (int64_t)blockIdx.x * (THREADS / 32) + (threadIdx.x >> 5); k < p.n_split_owners; k += warps_total) {
    const int64_t v = __ldg(p.split_owners + k);
    const int64_t r0 = __ldg(p.owner_indptr + v), r1 = __ldg(p.owner_indptr + v + 1);
    const float *P = p.partials + (r0 - v + k) * stride;   // first partial row of this vertex
    const int n = (int)(r1 - r0);
    for (int c = lane * 4; c < p.dim; c += 128) {
      const int head = c / p.head_dim;
      float M = -INFINITY;
      for (int g = 0; g < n; ++g) M = fmaxf(M, __ldg(P + (int64_t)g * stride + p.dim + head));
      float l = 0.f;
      float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
      for (int g = 0; g < n; ++g) {
        const float mg = __ldg(P + (int64_t)g * stride + p.dim + head);
        const float f = mg == -INFINITY ? 0.f : __expf(mg - M);
        l = fmaf(__ldg(P + (int64_t)g * stride + p.dim + p.heads + head), f, l);
        const float4 a = __ldg(reinterpret_cast<const float4 *>(P + (int64_t)g * stride + c));
        acc.x = fmaf(a.x, f, acc.x); acc.y = fmaf(a.y, f, acc.y); acc.z = fmaf(a.z, f, acc.z); acc.w = fmaf(a.w, f, acc.w);
      }
      const float inv = l > 0.f ? 1.f / l : 0.f;
      float o[4] = {acc.x * inv, acc.y * inv, acc.z * inv, acc.w * inv};
#pragma unroll
      for (int i = 0; i < 4; ++i) o[i] = act_apply(o[i] + (p.bias ? __ldg(p.bias + c + i) : 0.f), p.act);
      T *d = reinterpret_cast<T *>(p.dst) + v * p.dim + c;
      if (sizeof(T) == 4) {
        *reinterpret_cast<float4 *>(d) = make_float4(o[0], o[1], o[2], o[3]);
      } else {
        __nv_bfloat162 h0 = __floats2bfloat162_rn(o[0], o[1]), h1 = __floats2bfloat162_rn(o[2], o[3]);
        *reinterpret_cast<uint2 *>(d) = make_uint2(*reinterpret_cast<uint32_t *>(&h0), *reinterpret_cast<uint32_t *>(&h1));
      }
    }
  }
}

template <typename T, int SB, int LPR>
it_status launch_gat_lpr(const it_gat_args &a, StreamParams sp, int64_t bound_lo, int64_t bound_hi, cudaStream_t st) {
  GatPolicy<T, SB> pol;
  pol.scores = a.src_scores ? a.src_scores : a.scores; pol.src_stride = a.src_scores ? a.heads : 2 * a.heads;
  pol.scores_dst = a.scores_dst ? a.scores_dst : a.scores; pol.bias = a.bias; pol.dst = a.dst; pol.partials = a.partials;
  pol.dim = a.heads * a.head_dim; pol.heads = a.heads; pol.head_dim = a.head_dim; pol.act = a.act; pol.slope = a.slope;
  pol.col = 0; pol.head = 0; pol.s_dst = 0.f;
  const it_graph *g = a.g;
  // algorithmic bytes: per edge the index, one source score per head and one source row; per row
  // its metadata, owner, destination scores and one output row
  const double row_bytes = (double)pol.dim * sizeof(T);
  const int heads = a.heads;
  auto bytes_of = [=](int b, int64_t rows) {
    return (double)g->h_bucket_edges[b] * (4.0 + 4.0 * heads + row_bytes) + (double)rows * (20.0 + 4.0 * heads + row_bytes);
  };
  return launch_buckets<T, SB, LPR>(g, sp, pol, bytes_of, IT_K_GAT_CTA, IT_K_GAT_FLAT, IT_K_GAT_EMPTY, bound_lo, bound_hi, a.counters, st);
}

template <typename T>
it_status launch_gat(const it_gat_args &a, StreamParams sp, cudaStream_t st) {
  // 16-byte slices as long as one never straddles two heads
  const bool wide = (a.head_dim * (int)sizeof(T)) % 16 == 0;
  return dispatch_row_bytes(a.heads * a.head_dim * (int)sizeof(T), wide, [&]<int SB, int LPR>(int64_t lo, int64_t hi) {
    if ((a.head_dim * (int)sizeof(T)) % SB != 0) {
      it_set_error("gat: a %d-byte lane slice would straddle two heads (head_dim %d)", SB, a.head_dim);
      return IT_ERR_UNSUPPORTED;
    }
    return launch_gat_lpr<T, SB, LPR>(a, sp, lo, hi, st);
  });
}

}  // namespace

size_t it_gat_partial_bytes(const it_graph *g, int dim, int heads) {
  return (size_t)g->n_partial_rows * gat_partial_stride(dim, heads) * sizeof(float);
}

it_status it_launch_gat(const it_gat_args &a, cudaStream_t st) {
  const it_graph *g = a.g;
  IT_REQUIRE(g->n_partial_rows == 0 || a.partials, IT_ERR_WORKSPACE, "gat: no partial buffer");
  IT_REQUIRE(g->n_split_owners == 0 || a.head_dim % 4 == 0, IT_ERR_UNSUPPORTED, "gat on a split graph needs head_dim to be a multiple of 4");
  if (g->n == 0) return IT_OK;
  StreamParams sp;
  sp.meta = g->bucket_meta; sp.owner = g->bucket_owner; sp.indices = a.per_edge_rows ? nullptr : g->indices; sp.weights = nullptr;
  sp.src = a.z; sp.row_lo = sp.row_hi = 0; sp.dim = a.heads * a.head_dim; sp.batch_rows = 1; sp.counter = nullptr; sp.claim = 1;
  sp.src_pitch = (uint32_t)(sp.dim * it_dtype_size(a.dtype));
  if (a.dtype == IT_F32) IT_TRY(launch_gat<float>(a, sp, st));
  else IT_TRY(launch_gat<__nv_bfloat16>(a, sp, st));
  if (g->n_split_owners > 0) {
    GatCombineParams c;
    c.split_owners = g->split_owners; c.owner_indptr = g->owner_indptr; c.partials = a.partials; c.bias = a.bias;
    c.dst = a.dst; c.n_split_owners = g->n_split_owners; c.dim = a.heads * a.head_dim; c.heads = a.heads;
    c.head_dim = a.head_dim; c.act = a.act;
    int64_t want = (g->n_split_owners + 7) / 8;
    int64_t cap = (int64_t)g->num_sms * 8;
    unsigned blocks = (unsigned)(want < cap ? want : cap);
    const double cbytes = (double)it_gat_partial_bytes(g, c.dim, c.heads) +
                          (double)g->n_split_owners * c.dim * (a.dtype == IT_F32 ? 4.0 : 2.0);
    if (a.dtype == IT_F32) IT_LAUNCH(IT_K_COMBINE, cbytes, 0, st, gat_combine_kernel<float><<<blocks, THREADS, 0, st>>>(c));
    else IT_LAUNCH(IT_K_COMBINE, cbytes, 0, st, gat_combine_kernel<__nv_bfloat16><<<blocks, THREADS, 0, st>>>(c));
    IT_CUDA_TRY(cudaGetLastError());
  }
  return IT_OK;
}
