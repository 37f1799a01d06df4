// Gather (aggregate over the in-edges of one shadow row: sum / mean / max of w_e * h_src) and
// combine (fold the partial results of a split vertex).  The edge streaming itself lives in
// stream.cuh; this file supplies the per-lane state and what happens at the end of a row.
#include "stream.cuh"

namespace {

using namespace it_stream;
constexpr int GATHER_THREADS = THREADS;

// Per lane: VEC fp32 accumulators for its slice of the row.
enum { RED_SUM = 0, RED_MAX = 1, RED_MIN = 2 };   // sum also serves mean (the division happens once, at the end)

template <typename T, int SB, int RED, bool WEIGHTED_>
struct SagePolicy {
  using Slice = RowSlice<T, SB>;
  static constexpr int VEC = Slice::VEC;
  static constexpr int NS = VEC;
  static constexpr bool WEIGHTED = WEIGHTED_, HAS_EXTRA = false, NEEDS_OWNER = false;
  float *__restrict__ partials;
  void *__restrict__ dst;
  const void *__restrict__ self_term;
  const float *__restrict__ bias;
  int dim, dst_ld, self_ld, is_mean, epi, act;   // dim: width of this column chunk; *_ld: row lengths of dst / the self term
  int self_is_t;                                 // the self term is stored in T (else fp32)
  // per-thread
  int col;
  float self[VEC];

  __device__ __forceinline__ void setup(int t) { col = t * VEC; }
  __device__ __forceinline__ void init(float (&st)[NS]) const {
#pragma unroll
    for (int k = 0; k < NS; ++k) st[k] = RED == RED_MAX ? -INFINITY : (RED == RED_MIN ? INFINITY : 0.f);
  }
  __device__ __forceinline__ float extra(uint32_t) const { return 0.f; }
  __device__ __forceinline__ const float *extra_ptr(uint32_t) const { return nullptr; }
  __device__ __forceinline__ void edge(float (&st)[NS], const typename Slice::Raw &raw, float w, float) const {
    if constexpr (RED == RED_SUM && !WEIGHTED && sizeof(T) == 2 && IT_MIXED_ADD != 0) {
      // bf16 rows, plain sum: the mixed-precision add takes the bf16 operand as it is (same result as widening it first)
      uint32_t w[SB / 4];
      raw_words<SB>(raw, w);
#pragma unroll
      for (int i = 0; i < SB / 4; ++i) add_bf16x2_to_f32(st[2 * i], st[2 * i + 1], w[i]);
      return;
    }
    float f[VEC];
    Slice::unpack(raw, f);
    if constexpr (RED == RED_SUM && !WEIGHTED && VEC % 2 == 0) {   // two accumulators per instruction (measured: 1 % on the
#pragma unroll                                                      // 128-byte rows; with a weight the pair set-up eats the gain)
      for (int k = 0; k < VEC; k += 2) add_f32x2(st[k], st[k + 1], f[k], f[k + 1]);
    } else {
#pragma unroll
      for (int k = 0; k < VEC; ++k) {
        if (RED == RED_MAX) st[k] = fmaxf(st[k], WEIGHTED ? w * f[k] : f[k]);
        else if (RED == RED_MIN) st[k] = fminf(st[k], WEIGHTED ? w * f[k] : f[k]);
        else st[k] = WEIGHTED ? fmaf(w, f[k], st[k]) : st[k] + f[k];
      }
    }
  }
  __device__ __forceinline__ void merge(float (&st)[NS], const float (&o)[NS]) const {
#pragma unroll
    for (int k = 0; k < NS; ++k) st[k] = RED == RED_MAX ? fmaxf(st[k], o[k]) : (RED == RED_MIN ? fminf(st[k], o[k]) : st[k] + o[k]);
  }
  // the matching slice of the self term is fetched when the row starts, so that end_row does not wait for it
  __device__ __forceinline__ void begin_row(int32_t dest, int32_t) {
    if (epi == IT_EPI_ADD_ACT && dest >= 0) {
      if (sizeof(T) == 2 && self_is_t)
        Slice::unpack(Slice::load(reinterpret_cast<const char *>(self_term) + ((int64_t)dest * self_ld + col) * (int64_t)sizeof(T)), self);
      else
        load_floats_stream<VEC>(reinterpret_cast<const float *>(self_term) + (int64_t)dest * self_ld + col, self);
    }
  }
  __device__ __forceinline__ void end_row(float (&st)[NS], int32_t dest, int32_t, int64_t len) const {
    if (RED != RED_SUM && len == 0 && epi != IT_EPI_RAW_F32) {
#pragma unroll
      for (int i = 0; i < VEC; ++i) st[i] = 0.f;
    }
    if (dest < 0) {  // a group of a split vertex: raw partial, finished by the combine kernel
      store_floats<VEC>(partials + (int64_t)(~dest) * dim + col, st);
      return;
    }
    if (epi == IT_EPI_RAW_F32) {   // one part's share of a partial-gather: the reduce as it is (its identity for an empty row)
      store_floats<VEC>(reinterpret_cast<float *>(dst) + (int64_t)dest * dst_ld + col, st);
      return;
    }
    if (is_mean && len > 0) {
      const float inv = 1.f / (float)len;
#pragma unroll
      for (int i = 0; i < VEC; ++i) st[i] *= inv;
    }
    if (epi == IT_EPI_ADD_ACT) {
#pragma unroll
      for (int i = 0; i < VEC; ++i) st[i] = act_apply(st[i] + self[i], act);
    } else if (epi == IT_EPI_BIAS_ACT) {
#pragma unroll
      for (int i = 0; i < VEC; ++i) st[i] = act_apply(st[i] + (bias ? __ldg(bias + col + i) : 0.f), act);
    }
    Slice::store(reinterpret_cast<T *>(dst) + (int64_t)dest * dst_ld + col, st);
  }
};

// ----------------------------------------------------------------------------- combine
// One warp per split owner.  Its partial rows are rows [p0, p0 + n) of the partial buffer,
// folded in group order.
struct CombineParams {
  const int32_t *__restrict__ split_owners;
  const int64_t *__restrict__ owner_indptr;
  const int64_t *__restrict__ shadow_indptr;
  const float *__restrict__ partials;
  void *__restrict__ dst;
  const void *__restrict__ self_term;
  const float *__restrict__ bias;
  int64_t n_split_owners;
  int dim, dst_ld, self_ld, self_is_t;
  int red, is_mean, epi, act;   // red: RED_SUM / RED_MAX / RED_MIN
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
      auto fold = [&](const float4 &y) {
        if (p.red == RED_MAX) {
          acc.x = fmaxf(acc.x, y.x); acc.y = fmaxf(acc.y, y.y); acc.z = fmaxf(acc.z, y.z); acc.w = fmaxf(acc.w, y.w);
        } else if (p.red == RED_MIN) {
          acc.x = fminf(acc.x, y.x); acc.y = fminf(acc.y, y.y); acc.z = fminf(acc.z, y.z); acc.w = fminf(acc.w, y.w);
        } else {
          acc.x += y.x; acc.y += y.y; acc.z += y.z; acc.w += y.w;
        }
      };
      const int64_t n = r1 - r0;
      int64_t g = 1;
      for (; g + 8 <= n; g += 8) {   // eight partial rows in flight, folded in group order
        float4 y[8];
#pragma unroll
        for (int k = 0; k < 8; ++k) y[k] = __ldg(reinterpret_cast<const float4 *>(p.partials + (p0 + g + k) * p.dim + c));
#pragma unroll
        for (int k = 0; k < 8; ++k) fold(y[k]);
      }
      for (; g < n; ++g) fold(__ldg(reinterpret_cast<const float4 *>(p.partials + (p0 + g) * p.dim + c)));
      float o[4] = {acc.x * inv, acc.y * inv, acc.z * inv, acc.w * inv};
      const int64_t doff = v * p.dst_ld + c;
      if (p.epi == IT_EPI_RAW_F32) {
        *reinterpret_cast<float4 *>(reinterpret_cast<float *>(p.dst) + doff) = make_float4(o[0], o[1], o[2], o[3]);
        continue;
      }
      if (p.epi == IT_EPI_ADD_ACT) {
        float4 s;
        if (sizeof(T) == 2 && p.self_is_t) {
          const uint2 raw = __ldg(reinterpret_cast<const uint2 *>(reinterpret_cast<const T *>(p.self_term) + v * p.self_ld + c));
          s = make_float4(__uint_as_float(raw.x << 16), __uint_as_float(raw.x & 0xffff0000u), __uint_as_float(raw.y << 16),
                          __uint_as_float(raw.y & 0xffff0000u));
        } else {
          s = __ldg(reinterpret_cast<const float4 *>(reinterpret_cast<const float *>(p.self_term) + v * p.self_ld + c));
        }
        o[0] = act_apply(o[0] + s.x, p.act); o[1] = act_apply(o[1] + s.y, p.act);
        o[2] = act_apply(o[2] + s.z, p.act); o[3] = act_apply(o[3] + s.w, p.act);
      } else if (p.epi == IT_EPI_BIAS_ACT) {
#pragma unroll
        for (int i = 0; i < 4; ++i) o[i] = act_apply(o[i] + (p.bias ? __ldg(p.bias + c + i) : 0.f), p.act);
      }
      T *d = reinterpret_cast<T *>(p.dst) + doff;
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
template <typename T, int SB, int LPR, int RED, bool WEIGHTED>
it_status launch_policy(const it_gather_args &a, StreamParams sp, int64_t bound_lo, int64_t bound_hi, cudaStream_t st) {
  SagePolicy<T, SB, RED, WEIGHTED> pol;
  pol.partials = a.partials; pol.dst = a.dst; pol.self_term = a.self_term; pol.bias = a.bias; pol.dim = a.dim; pol.dst_ld = a.dst_ld > 0 ? a.dst_ld : a.dim; pol.self_ld = a.self_ld > 0 ? a.self_ld : a.dim;
  pol.is_mean = a.op == IT_GATHER_MEAN && a.epi != IT_EPI_RAW_F32; pol.epi = a.epi; pol.act = a.act; pol.col = 0;
  pol.self_is_t = a.self_dtype != IT_F32;
  const it_graph *g = a.g;
  // algorithmic bytes: per edge the index, the optional weight and one source row; per row its
  // metadata and one output row (plus the self row it is added to)
  const double row_bytes = (double)a.dim * sizeof(T);
  auto bytes_of = [=](int b, int64_t rows) {
    return (double)g->h_bucket_edges[b] * ((a.per_edge_rows ? 0.0 : 4.0) + (WEIGHTED ? 4.0 : 0.0) + row_bytes) +
           (double)rows * (16.0 + row_bytes + (a.epi == IT_EPI_ADD_ACT ? (a.self_dtype == IT_F32 ? 4.0 : (double)sizeof(T)) * a.dim : 0.0));
  };
  return launch_buckets<T, SB, LPR>(g, sp, pol, bytes_of, IT_K_GATHER_CTA, IT_K_GATHER_FLAT, IT_K_GATHER_EMPTY, bound_lo, bound_hi, a.counters, st);
}

template <typename T>
it_status launch_lpr(const it_gather_args &a, StreamParams sp, cudaStream_t st) {
  const bool w = a.use_edge_weights != 0;
  return dispatch_row_bytes(a.dim * (int)sizeof(T), true, [&]<int SB, int LPR>(int64_t lo, int64_t hi) {
    if (a.op == IT_GATHER_MAX) return w ? launch_policy<T, SB, LPR, RED_MAX, true>(a, sp, lo, hi, st) : launch_policy<T, SB, LPR, RED_MAX, false>(a, sp, lo, hi, st);
    if (a.op == IT_GATHER_MIN) return w ? launch_policy<T, SB, LPR, RED_MIN, true>(a, sp, lo, hi, st) : launch_policy<T, SB, LPR, RED_MIN, false>(a, sp, lo, hi, st);
    return w ? launch_policy<T, SB, LPR, RED_SUM, true>(a, sp, lo, hi, st) : launch_policy<T, SB, LPR, RED_SUM, false>(a, sp, lo, hi, st);
  });
}

}  // namespace

// One column chunk of the rows: `a.dim` is the chunk's width (a power of two between 16 and 512 bytes), the
// pointers already point at its first column, and the *_ld fields / src_ld carry the full row lengths.
static it_status launch_gather_chunk(const it_gather_args &a, cudaStream_t st) {
  const it_graph *g = a.g;
  StreamParams sp;
  sp.meta = g->bucket_meta; sp.owner = nullptr; sp.indices = a.per_edge_rows ? nullptr : g->indices; sp.weights = g->edge_weights;
  sp.src = a.src; sp.row_lo = sp.row_hi = 0; sp.dim = a.dim; sp.batch_rows = 1; sp.counter = nullptr; sp.claim = 1;
  sp.src_pitch = (uint32_t)((a.src_ld > 0 ? a.src_ld : a.dim) * it_dtype_size(a.dtype));
  if (a.dtype == IT_F32) IT_TRY(launch_lpr<float>(a, sp, st));
  else IT_TRY(launch_lpr<__nv_bfloat16>(a, sp, st));
  if (g->n_split_owners > 0) {
    CombineParams c;
    c.split_owners = g->split_owners; c.owner_indptr = g->owner_indptr; c.shadow_indptr = g->shadow_indptr;
    c.partials = a.partials; c.dst = a.dst; c.self_term = a.self_term; c.bias = a.bias; c.n_split_owners = g->n_split_owners;
    c.dim = a.dim; c.dst_ld = a.dst_ld > 0 ? a.dst_ld : a.dim; c.self_ld = a.self_ld > 0 ? a.self_ld : a.dim;
    c.red = a.op == IT_GATHER_MAX ? RED_MAX : (a.op == IT_GATHER_MIN ? RED_MIN : RED_SUM); c.is_mean = a.op == IT_GATHER_MEAN && a.epi != IT_EPI_RAW_F32; c.epi = a.epi; c.act = a.act; c.self_is_t = a.self_dtype != IT_F32;
    int64_t want = (g->n_split_owners + 7) / 8;
    int64_t cap = (int64_t)g->num_sms * 8;
    unsigned blocks = (unsigned)(want < cap ? want : cap);
    const double cbytes = (double)g->n_partial_rows * a.dim * 4.0 +
                          (double)g->n_split_owners * a.dim * (a.dtype == IT_F32 ? 4.0 : 2.0);
    if (a.dtype == IT_F32) IT_LAUNCH(IT_K_COMBINE, cbytes, 0, st, combine_kernel<float><<<blocks, GATHER_THREADS, 0, st>>>(c));
    else IT_LAUNCH(IT_K_COMBINE, cbytes, 0, st, combine_kernel<__nv_bfloat16><<<blocks, GATHER_THREADS, 0, st>>>(c));
  }
  return IT_OK;
}

// Rows of any multiple of 16 bytes: the kernels take rows of 16, 32, ..., 512 bytes, so a wider or odd row is cut
// into column chunks of those widths (largest first) and each chunk is gathered on its own, reading and writing
// its columns in place.  The aggregate is entry by entry, so the chunks are independent; each pass re-reads
// the edge indices (4 bytes against a chunk of up to 512 per edge).
it_status it_launch_gather(const it_gather_args &a, cudaStream_t st) {
  const it_graph *g = a.g;
  IT_REQUIRE(a.op == IT_GATHER_SUM || a.op == IT_GATHER_MEAN || a.op == IT_GATHER_MAX || a.op == IT_GATHER_MIN, IT_ERR_INVALID_ARG,
             "gather: bad op");
  IT_REQUIRE(!a.use_edge_weights || g->edge_weights, IT_ERR_INVALID_ARG, "layer uses edge weights but the graph has none");
  IT_REQUIRE(g->n_partial_rows == 0 || a.partials, IT_ERR_WORKSPACE, "gather: no partial buffer");
  const int es = it_dtype_size(a.dtype);
  IT_REQUIRE(a.dim > 0 && (a.dim * es) % 16 == 0, IT_ERR_INVALID_ARG, "gather: a row of %d bytes is not a multiple of 16", a.dim * es);
  if (g->n == 0) return IT_OK;
  const int full = a.dim;
  int c0 = 0;   // first column of the chunk
  while (c0 < full) {
    int bytes = 512;
    while (bytes > (full - c0) * es) bytes >>= 1;
    it_gather_args c = a;
    c.dim = bytes / es;
    c.src = (const char *)a.src + (size_t)c0 * es;
    c.src_ld = a.src_ld > 0 ? a.src_ld : full;
    c.dst = (char *)a.dst + (size_t)c0 * (a.epi == IT_EPI_RAW_F32 ? 4 : es);
    c.dst_ld = a.dst_ld > 0 ? a.dst_ld : full;
    c.self_term = a.self_term ? (const char *)a.self_term + (size_t)c0 * (a.self_dtype == IT_F32 ? 4 : es) : nullptr;
    c.self_ld = a.self_ld > 0 ? a.self_ld : full;
    c.bias = a.bias ? a.bias + c0 : nullptr;
    IT_TRY(launch_gather_chunk(c, st));
    c0 += c.dim;
  }
  return IT_OK;
}
