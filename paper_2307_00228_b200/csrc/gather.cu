// Gather (aggregate over the in-edges of one shadow row) and combine (fold the partial
// results of a split vertex).  HBM-bound: one 16-byte load per lane per edge, several edges in
// flight per lane, fp32 accumulation in a fixed order (results are bit-reproducible; no
// floating-point atomics anywhere).
//
// Work decomposition.  A feature row of `dim` elements is LPR = dim * sizeof(T) / 16 lanes wide.
//   * Rows of up to 2048 edges: a *group* of LPR lanes takes a batch of LPR rows of its bucket
//     (one coalesced 16-byte metadata load per row) and walks the batch's edges as one flat
//     stream: the lanes load LPR source ids at a time (the next chunk is prefetched while the
//     current one is consumed), every id is broadcast by shuffle, all lanes load their slice of
//     that source row, UNROLL rows in flight, and a row is written out when the stream crosses
//     its end.  Short rows therefore cost no dependent-load round trip of their own.
//   * Longer rows (up to the split threshold): one CTA per row, each warp a contiguous chunk,
//     warp results folded through shared memory in warp order.
//   * Empty rows: a streaming kernel that writes the epilogue of a zero aggregate.
#include "common.cuh"

namespace {

#ifndef IT_GATHER_UNROLL
#define IT_GATHER_UNROLL 8   // source rows in flight per lane
#endif
#ifndef IT_GATHER_MIN_BLOCKS
#define IT_GATHER_MIN_BLOCKS 2   // resident CTAs per SM the register budget is set for
#endif
#ifndef IT_GATHER_CTA_ABOVE
#define IT_GATHER_CTA_ABOVE 2048   // rows longer than this get a whole CTA; shorter ones a lane group
#endif
constexpr int GATHER_THREADS = 256;
constexpr int UNROLL = IT_GATHER_UNROLL;

// A 16-byte slice of a feature row stays packed in registers while it is in flight and is
// widened to fp32 only when it is accumulated.
template <typename T>
__device__ __forceinline__ uint4 load_slice(const T *p) { return __ldg(reinterpret_cast<const uint4 *>(p)); }

template <typename T> struct Row16;
template <> struct Row16<float> {
  static constexpr int VEC = 4;
  __device__ static __forceinline__ void unpack(const uint4 &x, float (&v)[4]) {
    v[0] = __uint_as_float(x.x); v[1] = __uint_as_float(x.y); v[2] = __uint_as_float(x.z); v[3] = __uint_as_float(x.w);
  }
  __device__ static __forceinline__ void store(float *p, const float (&v)[4]) {
    __stcs(reinterpret_cast<float4 *>(p), make_float4(v[0], v[1], v[2], v[3]));
  }
};
template <> struct Row16<__nv_bfloat16> {
  static constexpr int VEC = 8;
  __device__ static __forceinline__ void unpack(const uint4 &x, float (&v)[8]) {
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
    __stcs(reinterpret_cast<uint4 *>(p), make_uint4(w[0], w[1], w[2], w[3]));
  }
};

__device__ __forceinline__ float act_apply(float x, int act) {
  if (act == IT_ACT_RELU) return fmaxf(x, 0.f);
  if (act == IT_ACT_ELU) return x > 0.f ? x : expm1f(x);
  return x;
}

// streaming (read-once) loads: keep them from displacing feature rows in L2
__device__ __forceinline__ int32_t ld_stream(const int32_t *p) { return __ldcs(p); }
__device__ __forceinline__ float ld_stream(const float *p) { return __ldcs(p); }

struct GatherParams {
  const it_row_meta *__restrict__ meta;  // bucket order
  const int32_t *__restrict__ indices;
  const float *__restrict__ weights;
  const void *__restrict__ src;
  float *__restrict__ partials;
  void *__restrict__ dst;
  const float *__restrict__ self_term;
  int64_t row_lo, row_hi;  // range inside the bucket-ordered row list
  int dim;
  int is_mean, epi, act;
  int batch_rows;          // rows a lane group takes at a time in the flat kernel (<= LPR)
};

__device__ __forceinline__ it_row_meta load_meta(const it_row_meta *p) {
  const int4 raw = __ldcs(reinterpret_cast<const int4 *>(p));
  it_row_meta m;
  m.j0 = (int64_t)(((uint64_t)(uint32_t)raw.y << 32) | (uint32_t)raw.x);
  m.len = raw.z;
  m.dest = raw.w;
  return m;
}

// Write the aggregate of one shadow row (each of the LPR lanes holds its 16-byte slice).
// self[] is the matching slice of the self term (IT_EPI_ADD_ACT with dest >= 0 only).
template <typename T, bool IS_MAX>
__device__ __forceinline__ void finish_row(const GatherParams &p, int32_t dest, int64_t len, int col,
                                           float (&acc)[Row16<T>::VEC], const float (&self)[Row16<T>::VEC]) {
  constexpr int VEC = Row16<T>::VEC;
  if (IS_MAX && len == 0) {
#pragma unroll
    for (int i = 0; i < VEC; ++i) acc[i] = 0.f;
  }
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
  if (p.epi == IT_EPI_ADD_ACT) {
#pragma unroll
    for (int i = 0; i < VEC; ++i) acc[i] = act_apply(acc[i] + self[i], p.act);
  }
  Row16<T>::store(reinterpret_cast<T *>(p.dst) + (int64_t)dest * p.dim + col, acc);
}

template <int VEC>
__device__ __forceinline__ void load_self(const GatherParams &p, int32_t dest, int col, float (&self)[VEC]) {
  if (p.epi == IT_EPI_ADD_ACT && dest >= 0) {
#pragma unroll
    for (int i = 0; i < VEC; i += 4) {
      const float4 s = __ldcs(reinterpret_cast<const float4 *>(p.self_term + (int64_t)dest * p.dim + col + i));
      self[i] = s.x; self[i + 1] = s.y; self[i + 2] = s.z; self[i + 3] = s.w;
    }
  }
}

// ----------------------------------------------------------------------------- rows of <= 2048 edges
template <typename T, int LPR, bool IS_MAX, bool WEIGHTED>
__global__ void __launch_bounds__(GATHER_THREADS, IT_GATHER_MIN_BLOCKS) gather_flat_kernel(GatherParams p) {
  constexpr int VEC = Row16<T>::VEC;
  constexpr int G = LPR;
  constexpr int U = UNROLL < G ? UNROLL : G;
  const int lane = threadIdx.x & 31;
  const int t = lane % G;
  const unsigned gmask = (G == 32) ? 0xffffffffu : (((1u << (G & 31)) - 1u) << (lane - t));
  const int col = t * VEC;
  const T *__restrict__ src = reinterpret_cast<const T *>(p.src);
  const int64_t n_rows = p.row_hi - p.row_lo;
  const int BR = p.batch_rows;  // rows per batch, <= G: lanes t < BR hold their metadata
  const int64_t n_batches = (n_rows + BR - 1) / BR;
  const int64_t groups_total = (int64_t)gridDim.x * (GATHER_THREADS / G);

  for (int64_t b = (int64_t)blockIdx.x * (GATHER_THREADS / G) + threadIdx.x / G; b < n_batches; b += groups_total) {
    // ---- batch metadata: lane t owns row t of the batch
    const int64_t i = p.row_lo + b * BR + t;
    int64_t my_j0 = 0;
    int my_len = 0, my_dest = 0;
    if (t < BR && i < p.row_hi) {
      const it_row_meta m = load_meta(p.meta + i);
      my_j0 = m.j0; my_len = m.len; my_dest = m.dest;
    }
    const int64_t left = n_rows - b * BR;
    const int n_valid = left < BR ? (int)left : BR;
    int my_end = my_len;  // inclusive prefix sum of the row lengths
#pragma unroll
    for (int o = 1; o < G; o <<= 1) {
      const int y = __shfl_up_sync(gmask, my_end, o, G);
      if (t >= o) my_end += y;
    }
    const int total = __shfl_sync(gmask, my_end, G - 1, G);
    const int my_start = my_end - my_len;

    // ---- one chunk of the flat edge stream: lane t fetches edge (base + t) and learns whether
    // it is the last edge of its row; `ends` collects those flags for the whole chunk.
    // (Rows handled here have at least one edge: empty rows live in their own bucket.)
    auto load_chunk = [&](int base, int32_t &idx, float &w, unsigned &ends) {
      const int q = base + t;
      int lo = 0;
#pragma unroll
      for (int step = G / 2; step >= 1; step >>= 1) {
        const int e = __shfl_sync(gmask, my_end, lo + step - 1, G);
        if (e <= q) lo += step;
      }
      const int row_end = __shfl_sync(gmask, my_end, lo, G);
      const int64_t j = __shfl_sync(gmask, my_j0, lo, G) + (q - __shfl_sync(gmask, my_start, lo, G));
      idx = 0;
      w = 1.f;
      if (q < total) {
        idx = ld_stream(p.indices + j);
        if (WEIGHTED) w = ld_stream(p.weights + j);
      }
      ends = (__ballot_sync(gmask, q < total && q + 1 == row_end) >> (lane - t)) & (G == 32 ? 0xffffffffu : ((1u << (G & 31)) - 1u));
    };

    float acc[VEC], self[VEC];
#pragma unroll
    for (int k = 0; k < VEC; ++k) { acc[k] = IS_MAX ? -INFINITY : 0.f; self[k] = 0.f; }
    int cur = 0;  // row of the batch that acc belongs to
    if (n_valid > 0) load_self<VEC>(p, __shfl_sync(gmask, my_dest, 0, G), col, self);
    auto next_row = [&]() {
      finish_row<T, IS_MAX>(p, __shfl_sync(gmask, my_dest, cur, G), __shfl_sync(gmask, my_len, cur, G), col, acc, self);
      ++cur;
#pragma unroll
      for (int k = 0; k < VEC; ++k) acc[k] = IS_MAX ? -INFINITY : 0.f;
      const int32_t nd = __shfl_sync(gmask, my_dest, cur & (G - 1), G);
      if (cur < n_valid) load_self<VEC>(p, nd, col, self);
    };
    auto accumulate = [&](const uint4 &raw, float w) {
      float f[VEC];
      Row16<T>::unpack(raw, f);
#pragma unroll
      for (int k = 0; k < VEC; ++k) {
        if (IS_MAX) acc[k] = fmaxf(acc[k], WEIGHTED ? w * f[k] : f[k]);
        else acc[k] = WEIGHTED ? fmaf(w, f[k], acc[k]) : acc[k] + f[k];
      }
    };
    const char *my_src = reinterpret_cast<const char *>(src + col);
    const uint32_t row_bytes = (uint32_t)p.dim * (uint32_t)sizeof(T);

    int32_t idx_c, idx_n;
    float w_c, w_n;
    unsigned ends_c, ends_n;
    load_chunk(0, idx_c, w_c, ends_c);
    for (int base = 0; base < total; base += G) {
      load_chunk(base + G, idx_n, w_n, ends_n);  // in flight while this chunk is consumed
      const int cnt = (total - base) < G ? (total - base) : G;
      int k0 = 0;
      for (; k0 + U <= cnt; k0 += U) {  // full groups of U edges: no predicates
        uint4 v[U];
        float w[U];
#pragma unroll
        for (int u = 0; u < U; ++u) {
          const uint32_t s = (uint32_t)__shfl_sync(gmask, idx_c, k0 + u, G);
          w[u] = WEIGHTED ? __shfl_sync(gmask, w_c, k0 + u, G) : 1.f;
          v[u] = __ldg(reinterpret_cast<const uint4 *>(my_src + (uint64_t)s * row_bytes));
        }
#pragma unroll
        for (int u = 0; u < U; ++u) {
          accumulate(v[u], w[u]);
          if ((ends_c >> (k0 + u)) & 1u) next_row();  // group-uniform
        }
      }
      if (k0 < cnt) {  // tail of the chunk
        uint4 v[U];
        float w[U];
#pragma unroll
        for (int u = 0; u < U; ++u) {
          const int e = k0 + u;
          const uint32_t s = (uint32_t)__shfl_sync(gmask, idx_c, e & (G - 1), G);
          w[u] = WEIGHTED ? __shfl_sync(gmask, w_c, e & (G - 1), G) : 1.f;
          if (e < cnt) v[u] = __ldg(reinterpret_cast<const uint4 *>(my_src + (uint64_t)s * row_bytes));
        }
#pragma unroll
        for (int u = 0; u < U; ++u) {
          if (k0 + u < cnt) {
            accumulate(v[u], w[u]);
            if ((ends_c >> (k0 + u)) & 1u) next_row();
          }
        }
      }
      idx_c = idx_n; w_c = w_n; ends_c = ends_n;
    }
  }
}

// ----------------------------------------------------------------------------- long rows: one CTA each
// Aggregate edges [j0, j1) with the whole warp: SLOTS = 32 / LPR edges at once, index chunk of 32
// prefetched one step ahead.
template <typename T, int LPR, bool IS_MAX, bool WEIGHTED>
__device__ __forceinline__ void gather_edges_warp(const GatherParams &p, int64_t j0, int64_t j1, int lane,
                                                  float (&acc)[Row16<T>::VEC]) {
  constexpr int VEC = Row16<T>::VEC;
  constexpr int SLOTS = 32 / LPR;
  constexpr int U = UNROLL;
  const int slot = lane / LPR;
  const int col = (lane % LPR) * VEC;
  const T *__restrict__ src = reinterpret_cast<const T *>(p.src);
  auto load_chunk = [&](int64_t base, int32_t &idx, float &w) {
    idx = 0; w = 1.f;
    if (base + lane < j1) {
      idx = ld_stream(p.indices + base + lane);
      if (WEIGHTED) w = ld_stream(p.weights + base + lane);
    }
  };
  int32_t idx_c, idx_n;
  float w_c, w_n;
  load_chunk(j0, idx_c, w_c);
  for (int64_t base = j0; base < j1; base += 32) {
    load_chunk(base + 32, idx_n, w_n);
    const int cnt = (int)((j1 - base) < 32 ? (j1 - base) : 32);
    for (int k0 = 0; k0 < cnt; k0 += SLOTS * U) {
      uint4 v[U];
      float w[U];
      bool ok[U];
#pragma unroll
      for (int u = 0; u < U; ++u) {
        const int e = k0 + u * SLOTS + slot;
        const int32_t s = __shfl_sync(0xffffffffu, idx_c, e & 31);
        w[u] = WEIGHTED ? __shfl_sync(0xffffffffu, w_c, e & 31) : 1.f;
        ok[u] = e < cnt;
        if (ok[u]) v[u] = load_slice(src + (int64_t)s * p.dim + col);
      }
#pragma unroll
      for (int u = 0; u < U; ++u) {
        if (ok[u]) {
          float f[VEC];
          Row16<T>::unpack(v[u], f);
#pragma unroll
          for (int k = 0; k < VEC; ++k) {
            if (IS_MAX) acc[k] = fmaxf(acc[k], WEIGHTED ? w[u] * f[k] : f[k]);
            else acc[k] = WEIGHTED ? fmaf(w[u], f[k], acc[k]) : acc[k] + f[k];
          }
        }
      }
    }
    idx_c = idx_n; w_c = w_n;
  }
  // fold the SLOTS edge slots into slot 0 (fixed order)
#pragma unroll
  for (int o = 16; o >= LPR; o >>= 1) {
#pragma unroll
    for (int k = 0; k < VEC; ++k) {
      const float y = __shfl_xor_sync(0xffffffffu, acc[k], o);
      acc[k] = IS_MAX ? fmaxf(acc[k], y) : acc[k] + y;
    }
  }
}

template <typename T, int LPR, bool IS_MAX, bool WEIGHTED>
__global__ void __launch_bounds__(GATHER_THREADS, IT_GATHER_MIN_BLOCKS) gather_cta_kernel(GatherParams p) {
  constexpr int VEC = Row16<T>::VEC;
  constexpr int WARPS = GATHER_THREADS / 32;
  __shared__ float red[WARPS][LPR * VEC];
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  for (int64_t i = p.row_lo + blockIdx.x; i < p.row_hi; i += gridDim.x) {
    const it_row_meta m = load_meta(p.meta + i);
    const int64_t j0 = m.j0, j1 = m.j0 + m.len;
    const int64_t chunk = ((int64_t)m.len + WARPS - 1) / WARPS;
    int64_t a = j0 + warp * chunk, b = a + chunk;
    if (a > j1) a = j1;
    if (b > j1) b = j1;
    float acc[VEC], self[VEC];
#pragma unroll
    for (int k = 0; k < VEC; ++k) { acc[k] = IS_MAX ? -INFINITY : 0.f; self[k] = 0.f; }
    if (warp == 0 && lane < LPR) load_self<VEC>(p, m.dest, lane * VEC, self);
    gather_edges_warp<T, LPR, IS_MAX, WEIGHTED>(p, a, b, lane, acc);
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
          const float y = red[w][lane * VEC + k];
          acc[k] = IS_MAX ? fmaxf(acc[k], y) : acc[k] + y;
        }
      }
      finish_row<T, IS_MAX>(p, m.dest, m.len, lane * VEC, acc, self);
    }
  }
}

// ----------------------------------------------------------------------------- empty rows
template <typename T, int LPR>
__global__ void __launch_bounds__(GATHER_THREADS) gather_empty_kernel(GatherParams p) {
  constexpr int VEC = Row16<T>::VEC;
  const int t = threadIdx.x % LPR;
  const int64_t groups_total = (int64_t)gridDim.x * (GATHER_THREADS / LPR);
  for (int64_t i = p.row_lo + (int64_t)blockIdx.x * (GATHER_THREADS / LPR) + threadIdx.x / LPR; i < p.row_hi; i += groups_total) {
    const it_row_meta m = load_meta(p.meta + i);
    float acc[VEC], self[VEC];
#pragma unroll
    for (int k = 0; k < VEC; ++k) { acc[k] = 0.f; self[k] = 0.f; }
    load_self<VEC>(p, m.dest, t * VEC, self);
    finish_row<T, false>(p, m.dest, 0, t * VEC, acc, self);
  }
}

// ----------------------------------------------------------------------------- combine
// One warp per split owner.  Its partial rows are rows [p0, p0 + n) of the partial buffer,
// folded in group order.
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
    const int64_t max_blocks = (int64_t)g->num_sms * IT_GATHER_MIN_BLOCKS * 2;
    // algorithmic bytes: per edge the index, the optional weight and one source row; per row its
    // metadata and one output row (plus the self row it is added to)
    const double row_bytes = (double)p.dim * sizeof(T);
    const double bytes = (double)g->h_bucket_edges[b] * (4.0 + (WEIGHTED ? 4.0 : 0.0) + row_bytes) +
                         (double)rows * (16.0 + row_bytes + (p.epi == IT_EPI_ADD_ACT ? 4.0 * p.dim : 0.0));
    if (bound == 0) {
      int64_t want = (rows + (GATHER_THREADS / LPR) - 1) / (GATHER_THREADS / LPR);
      unsigned blocks = (unsigned)(want < max_blocks ? want : max_blocks);
      IT_LAUNCH(IT_K_GATHER_EMPTY, bytes, 0, st, gather_empty_kernel<T, LPR><<<blocks, GATHER_THREADS, 0, st>>>(p));
    } else if (bound > IT_GATHER_CTA_ABOVE) {
      unsigned blocks = (unsigned)(rows < max_blocks ? rows : max_blocks);
      IT_LAUNCH(IT_K_GATHER_CTA, bytes, 0, st, gather_cta_kernel<T, LPR, IS_MAX, WEIGHTED><<<blocks, GATHER_THREADS, 0, st>>>(p));
    } else {
      // about 256 edges per batch at most: 32 rows of <= 8 edges, 8 rows of <= 32, one longer row
      int br = bound <= 8 ? 32 : (bound <= 32 ? 8 : 1);
      if (br > LPR) br = LPR;
      p.batch_rows = br;
      const int64_t batches = (rows + br - 1) / br;
      int64_t want = (batches + (GATHER_THREADS / LPR) - 1) / (GATHER_THREADS / LPR);
      unsigned blocks = (unsigned)(want < max_blocks ? want : max_blocks);
      IT_LAUNCH(IT_K_GATHER_FLAT, bytes, 0, st, gather_flat_kernel<T, LPR, IS_MAX, WEIGHTED><<<blocks, GATHER_THREADS, 0, st>>>(p));
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
  p.meta = g->bucket_meta; p.indices = g->indices; p.weights = g->edge_weights;
  p.src = a.src; p.partials = a.partials;
  p.dst = a.dst; p.self_term = a.self_term; p.row_lo = p.row_hi = 0; p.dim = a.dim;
  p.is_mean = a.op == IT_GATHER_MEAN; p.epi = a.epi; p.act = a.act; p.batch_rows = 1;
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
  }
  return IT_OK;
}
