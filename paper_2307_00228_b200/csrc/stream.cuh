// Row-streaming machinery shared by the plain gather (sum / mean / max) and the GAT reduce.
//
// Both walk the in-edges of shadow rows and fold one slice of every source row per
// lane into a small per-lane state; they differ only in that state and its update (a Policy).
// HBM-bound: one 4- to 16-byte load per lane per edge, several edges in flight per lane, a fixed
// order of operations (results are bit-reproducible; no floating-point atomics anywhere).
//
// Work decomposition.  A feature row is cut into lane slices of SB bytes and is LPR = row bytes / SB
// lanes wide; rows are bucketed by length and each bucket gets the kernel that suits it.
//   * stream_rows_ring_kernel, stream_cta_ring_kernel (stream_ring.cuh; rows of 128 bytes and more):
//     a warp walks the edges of a batch of rows (or of its part of one very long row) as one flat
//     stream and stages the source rows through a per-warp ring in shared memory with cp.async.
//   * stream_short_rows_kernel (128-byte rows of at most a few dozen edges): one group of 8 lanes
//     per row, eight row loads back to back, no edge stream.
//   * stream_rows_kernel (rows narrower than 128 bytes): a *group* of LPR lanes takes a batch of rows
//     and walks the batch's edges as one flat stream with UNROLL rows in flight per lane in registers.
//   * stream_cta_kernel (the same rows, very long): one CTA per row, each warp a contiguous chunk,
//     SLOTS = 32 / LPR edges at once per warp; slot and warp states are merged in a fixed order.
//   * stream_empty_kernel: rows without edges.
//
// Policy interface (all __device__):
//   static constexpr int NS;                 // floats of per-lane state
//   static constexpr bool WEIGHTED, HAS_EXTRA, NEEDS_OWNER;
//   void init(float (&st)[NS]);
//   float extra(uint32_t src_row);           // per-edge scalar that is loaded with the row (HAS_EXTRA)
//   const float *extra_ptr(uint32_t src_row);   // its address, for the asynchronous copies of the ring kernels
//   void edge(float (&st)[NS], const Raw &raw, float w, float x);   // Raw = the packed slice
//   void merge(float (&st)[NS], const float (&other)[NS]);     // other comes later in edge order
//   void begin_row(int32_t dest, int32_t owner);               // prefetch what end_row needs
//   void end_row(float (&st)[NS], int32_t dest, int32_t owner, int64_t len);
#pragma once

#include <atomic>

#include "common.cuh"

#ifndef IT_GATHER_UNROLL
#define IT_GATHER_UNROLL 4   // source rows in flight per lane
#endif
#ifndef IT_GATHER_MIN_BLOCKS
#define IT_GATHER_MIN_BLOCKS 4   // resident CTAs per SM the register budget is set for
#endif
#ifndef IT_RING_MIN_BLOCKS
#define IT_RING_MIN_BLOCKS 4   // resident CTAs per SM of the shared-memory-ring kernel
#endif
#ifndef IT_RING_STAGE_ROWS
#define IT_RING_STAGE_ROWS 4   // 512-byte groups of rows per stage of the ring
#endif
#ifndef IT_RING_STAGES
#define IT_RING_STAGES 2
#endif
#ifndef IT_RING_DYNAMIC
#define IT_RING_DYNAMIC 1   // 1: the warps of the ring kernel claim their batches from a counter instead of walking a fixed stride
#endif
#ifndef IT_RING_CLAIMS_PER_WARP
#define IT_RING_CLAIMS_PER_WARP 16   // claims a warp of the ring kernel makes on average over a launch
#endif
#ifndef IT_SHORT_MIN_BLOCKS
#define IT_SHORT_MIN_BLOCKS 6   // resident CTAs per SM of the short-row kernel (eight 16-byte slices in flight per lane, staged in shared memory)
#endif
#ifndef IT_SHORT_EDGES
#define IT_SHORT_EDGES 8         // source rows a lane of the short-row kernel has in flight per round
#endif
#ifndef IT_SHORT_ASYNC
#define IT_SHORT_ASYNC 1         // 1: the short-row kernel stages its slices through shared memory with cp.async (0: in registers)
#endif
#ifndef IT_SHORT_256
#define IT_SHORT_256 1           // 1: 256-byte rows of at most IT_SHORT_BELOW edges take the lane-group kernel too (16 lanes per row)
#endif
#ifndef IT_SHORT_BELOW
#define IT_SHORT_BELOW 32       // 128-byte rows: buckets of rows up to this long take the short-row kernel
#endif
#ifndef IT_GATHER_CTA_ABOVE
#define IT_GATHER_CTA_ABOVE 1024   // rows longer than this get a whole CTA; shorter ones a lane group or a warp
#endif

namespace it_stream {

constexpr int THREADS = 256;
constexpr int UNROLL = IT_GATHER_UNROLL;

// One lane's slice of a feature row: SB = 4, 8 or 16 bytes, LPR = row bytes / SB lanes per row (see
// dispatch_row_bytes for the choice).  A slice stays packed while it is in flight and is widened to fp32
// only when it is consumed.
template <int SB> struct SliceRaw;
template <> struct SliceRaw<4> { using type = uint32_t; };
template <> struct SliceRaw<8> { using type = uint2; };
template <> struct SliceRaw<16> { using type = uint4; };

template <int SB>
__device__ __forceinline__ void raw_words(const typename SliceRaw<SB>::type &x, uint32_t (&w)[SB / 4]) {
  if constexpr (SB == 4) { w[0] = x; }
  else if constexpr (SB == 8) { w[0] = x.x; w[1] = x.y; }
  else { w[0] = x.x; w[1] = x.y; w[2] = x.z; w[3] = x.w; }
}
template <int SB>
__device__ __forceinline__ typename SliceRaw<SB>::type words_raw(const uint32_t (&w)[SB / 4]) {
  if constexpr (SB == 4) return w[0];
  else if constexpr (SB == 8) return make_uint2(w[0], w[1]);
  else return make_uint4(w[0], w[1], w[2], w[3]);
}

template <typename T, int SB> struct RowSlice {
  static constexpr int VEC = SB / (int)sizeof(T);
  using Raw = typename SliceRaw<SB>::type;
  __device__ static __forceinline__ Raw load(const char *p) { return __ldg(reinterpret_cast<const Raw *>(p)); }
  __device__ static __forceinline__ void unpack(const Raw &x, float (&v)[VEC]) {
    uint32_t w[SB / 4];
    raw_words<SB>(x, w);
    if constexpr (sizeof(T) == 4) {
#pragma unroll
      for (int i = 0; i < VEC; ++i) v[i] = __uint_as_float(w[i]);
    } else {
#pragma unroll
      for (int i = 0; i < SB / 4; ++i) {
        v[2 * i] = __uint_as_float(w[i] << 16);
        v[2 * i + 1] = __uint_as_float(w[i] & 0xffff0000u);
      }
    }
  }
  __device__ static __forceinline__ void store(T *p, const float (&v)[VEC]) {
    uint32_t w[SB / 4];
    if constexpr (sizeof(T) == 4) {
#pragma unroll
      for (int i = 0; i < VEC; ++i) w[i] = __float_as_uint(v[i]);
    } else {
#pragma unroll
      for (int i = 0; i < SB / 4; ++i) {
        __nv_bfloat162 h = __floats2bfloat162_rn(v[2 * i], v[2 * i + 1]);
        w[i] = *reinterpret_cast<uint32_t *>(&h);
      }
    }
    __stcs(reinterpret_cast<Raw *>(p), words_raw<SB>(w));
  }
};

// Two fp32 operations in one instruction (sm_100 has packed add / mul / fma on register pairs; each half is the IEEE
// operation of the scalar instruction, so results do not change).  The reduce of a row slice is the kernels' largest
// share of issued instructions; measured gain: 1 % on the 128-byte pooling rows, 3 % on the GAT rows.
#ifndef IT_PACKED_F32
#define IT_PACKED_F32 1
#endif
__device__ __forceinline__ uint64_t pack_f32x2(float lo, float hi) {
  uint64_t r;
  asm("mov.b64 %0, {%1, %2};" : "=l"(r) : "f"(lo), "f"(hi));
  return r;
}
__device__ __forceinline__ void unpack_f32x2(uint64_t v, float &lo, float &hi) {
  asm("mov.b64 {%0, %1}, %2;" : "=f"(lo), "=f"(hi) : "l"(v));
}
// a += b (pairwise)
__device__ __forceinline__ void add_f32x2(float &a0, float &a1, float b0, float b1) {
#if IT_PACKED_F32
  uint64_t d;
  asm("add.rn.f32x2 %0, %1, %2;" : "=l"(d) : "l"(pack_f32x2(a0, a1)), "l"(pack_f32x2(b0, b1)));
  unpack_f32x2(d, a0, a1);
#else
  a0 += b0; a1 += b1;
#endif
}
// a0 += low bf16 of w, a1 += high bf16 of w: mixed-precision adds (fp32 accumulator, bf16 addend; the addend is
// widened exactly, so each result equals the fp32 add of the widened value).
#ifndef IT_MIXED_ADD
#define IT_MIXED_ADD 1
#endif
__device__ __forceinline__ void add_bf16x2_to_f32(float &a0, float &a1, uint32_t w) {
  unsigned short lo, hi;
  asm("mov.b32 {%0, %1}, %2;" : "=h"(lo), "=h"(hi) : "r"(w));
  asm("add.rn.f32.bf16 %0, %1, %0;" : "+f"(a0) : "h"(lo));
  asm("add.rn.f32.bf16 %0, %1, %0;" : "+f"(a1) : "h"(hi));
}
// a = w * b + a * s (pairwise, scalars w and s): the running-softmax update
__device__ __forceinline__ void scale_fma_f32x2(float &a0, float &a1, float s, float w, float b0, float b1) {
#if IT_PACKED_F32
  uint64_t t, d;
  asm("mul.rn.f32x2 %0, %1, %2;" : "=l"(t) : "l"(pack_f32x2(a0, a1)), "l"(pack_f32x2(s, s)));
  asm("fma.rn.f32x2 %0, %1, %2, %3;" : "=l"(d) : "l"(pack_f32x2(w, w)), "l"(pack_f32x2(b0, b1)), "l"(t));
  unpack_f32x2(d, a0, a1);
#else
  a0 = fmaf(w, b0, a0 * s); a1 = fmaf(w, b1, a1 * s);
#endif
}

// VEC consecutive fp32 values (VEC = 1, 2, 4 or 8), vectorised
template <int VEC>
__device__ __forceinline__ void store_floats(float *p, const float (&v)[VEC]) {
  if constexpr (VEC == 1) { *p = v[0]; }
  else if constexpr (VEC == 2) { *reinterpret_cast<float2 *>(p) = make_float2(v[0], v[1]); }
  else {
#pragma unroll
    for (int i = 0; i < VEC; i += 4) *reinterpret_cast<float4 *>(p + i) = make_float4(v[i], v[i + 1], v[i + 2], v[i + 3]);
  }
}
template <int VEC>
__device__ __forceinline__ void load_floats_stream(const float *p, float (&v)[VEC]) {
  if constexpr (VEC == 1) { v[0] = __ldcs(p); }
  else if constexpr (VEC == 2) { const float2 x = __ldcs(reinterpret_cast<const float2 *>(p)); v[0] = x.x; v[1] = x.y; }
  else {
#pragma unroll
    for (int i = 0; i < VEC; i += 4) {
      const float4 x = __ldcs(reinterpret_cast<const float4 *>(p + i));
      v[i] = x.x; v[i + 1] = x.y; v[i + 2] = x.z; v[i + 3] = x.w;
    }
  }
}

__device__ __forceinline__ float act_apply(float x, int act) {
  if (act == IT_ACT_RELU) return fmaxf(x, 0.f);
  if (act == IT_ACT_ELU) return it_elu(x);
  return x;
}

// What every streaming kernel needs besides its policy.
struct StreamParams {
  const it_row_meta *__restrict__ meta;   // bucket order
  const int32_t *__restrict__ owner;      // bucket order: vertex a row belongs to (policies with NEEDS_OWNER)
  const int32_t *__restrict__ indices;    // source vertex of every edge; NULL: row j of src belongs to edge j itself (edge features)
  const float *__restrict__ weights;
  const void *__restrict__ src;           // [n, dim] rows that are gathered ([n_edges, dim] when indices is NULL)
  int64_t row_lo, row_hi;                 // range inside the bucket-ordered row list
  int dim;                                // elements of a row that are gathered (one column chunk of the source rows)
  uint32_t src_pitch;                     // bytes from one source row to the next (>= dim elements)
  int batch_rows;                         // rows a lane group takes at a time (<= LPR)
  int *counter;                           // ring kernel: zeroed device word from which the warps claim their batches after
                                          // their first ones (NULL: every warp walks a fixed stride of the batches)
  int claim;                              // batches per claim
};

__device__ __forceinline__ it_row_meta load_meta(const it_row_meta *p) {
  const int4 raw = __ldcs(reinterpret_cast<const int4 *>(p));
  it_row_meta m;
  m.j0 = (int64_t)(((uint64_t)(uint32_t)raw.y << 32) | (uint32_t)raw.x);
  m.len = raw.z;
  m.dest = raw.w;
  return m;
}

// ----------------------------------------------------------------------------- batches of rows per lane group
// Rows handled here have at least one edge: empty rows live in their own bucket.
template <typename T, int SB, int LPR, class Policy>
__global__ void __launch_bounds__(THREADS, IT_GATHER_MIN_BLOCKS) stream_rows_kernel(StreamParams p, Policy pol) {
  constexpr int G = LPR;
  // more rows in flight for narrower slices, as far as the register budget and the size of the unrolled
  // consume loop (which carries a copy of the end-of-row code per edge) allow
  constexpr int UW = Policy::HAS_EXTRA ? UNROLL : (UNROLL * (16 / SB) < 2 * UNROLL ? UNROLL * (16 / SB) : 2 * UNROLL);
  constexpr int U = UW < G ? UW : G;
  constexpr int NS = Policy::NS;
  const int lane = threadIdx.x & 31;
  const int t = lane % G;
  const unsigned gbits = (G == 32) ? 0xffffffffu : ((1u << (G & 31)) - 1u);
  const unsigned gmask = gbits << (lane - t);
  pol.setup(t);
  const int64_t n_rows = p.row_hi - p.row_lo;
  const int BR = p.batch_rows;  // rows per batch, <= G: lanes t < BR hold their metadata
  const int64_t n_batches = (n_rows + BR - 1) / BR;
  const int64_t groups_total = (int64_t)gridDim.x * (THREADS / G);
  const char *my_src = reinterpret_cast<const char *>(p.src) + (size_t)t * SB;
  using Slice = RowSlice<T, SB>;
  const uint32_t row_bytes = p.src_pitch;

  for (int64_t b = (int64_t)blockIdx.x * (THREADS / G) + threadIdx.x / G; b < n_batches; b += groups_total) {
    // ---- batch metadata: lane t owns row t of the batch
    const int64_t i = p.row_lo + b * BR + t;
    int64_t my_j0 = 0;
    int my_len = 0, my_dest = 0, my_owner = 0;
    if (t < BR && i < p.row_hi) {
      const it_row_meta m = load_meta(p.meta + i);
      my_j0 = m.j0; my_len = m.len; my_dest = m.dest;
      if (Policy::NEEDS_OWNER) my_owner = __ldcs(p.owner + i);
    }
    int my_end = my_len;  // inclusive prefix sum of the row lengths
#pragma unroll
    for (int o = 1; o < G; o <<= 1) {
      const int y = __shfl_up_sync(gmask, my_end, o, G);
      if (t >= o) my_end += y;
    }
    const int total = __shfl_sync(gmask, my_end, G - 1, G);
    const int my_start = my_end - my_len;

    // ---- one chunk of the flat edge stream: lane t fetches edge (base + t) and learns whether it
    // is the last edge of its row; `ends` collects those flags for the whole chunk.
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
        idx = p.indices ? __ldcs(p.indices + j) : (int32_t)j;
        if (Policy::WEIGHTED) w = __ldcs(p.weights + j);
      }
      ends = (__ballot_sync(gmask, q < total && q + 1 == row_end) >> (lane - t)) & gbits;
    };

    float st[NS];
    pol.init(st);
    int cur = 0;  // row of the batch that st belongs to
    pol.begin_row(__shfl_sync(gmask, my_dest, 0, G), __shfl_sync(gmask, my_owner, 0, G));
    auto next_row = [&]() {
      pol.end_row(st, __shfl_sync(gmask, my_dest, cur, G), __shfl_sync(gmask, my_owner, cur, G),
                  __shfl_sync(gmask, my_len, cur, G));
      ++cur;
      pol.init(st);
      const int32_t nd = __shfl_sync(gmask, my_dest, cur & (G - 1), G);
      const int32_t no = __shfl_sync(gmask, my_owner, cur & (G - 1), G);
      if (cur < BR && __shfl_sync(gmask, my_len, cur & (G - 1), G) > 0) pol.begin_row(nd, no);
    };

    int32_t idx_c, idx_n;
    float w_c, w_n;
    unsigned ends_c, ends_n;
    load_chunk(0, idx_c, w_c, ends_c);
    for (int base = 0; base < total; base += G) {
      load_chunk(base + G, idx_n, w_n, ends_n);  // in flight while this chunk is consumed
      const int cnt = (total - base) < G ? (total - base) : G;
      int k0 = 0;
      for (; k0 + U <= cnt; k0 += U) {  // full groups of U edges: no predicates
        typename Slice::Raw v[U];
        float w[U], x[U];
#pragma unroll
        for (int u = 0; u < U; ++u) {
          const uint32_t s = (uint32_t)__shfl_sync(gmask, idx_c, k0 + u, G);
          w[u] = Policy::WEIGHTED ? __shfl_sync(gmask, w_c, k0 + u, G) : 1.f;
          v[u] = Slice::load(my_src + (uint64_t)s * row_bytes);
          x[u] = Policy::HAS_EXTRA ? pol.extra(s) : 0.f;
        }
#pragma unroll
        for (int u = 0; u < U; ++u) {
          pol.edge(st, v[u], w[u], x[u]);
          if ((ends_c >> (k0 + u)) & 1u) next_row();  // group-uniform
        }
      }
      if (k0 < cnt) {  // tail of the chunk
        typename Slice::Raw v[U];
        float w[U], x[U];
#pragma unroll
        for (int u = 0; u < U; ++u) {
          const int e = k0 + u;
          const uint32_t s = (uint32_t)__shfl_sync(gmask, idx_c, e & (G - 1), G);
          w[u] = Policy::WEIGHTED ? __shfl_sync(gmask, w_c, e & (G - 1), G) : 1.f;
          x[u] = 0.f;
          if (e < cnt) {
            v[u] = Slice::load(my_src + (uint64_t)s * row_bytes);
            if (Policy::HAS_EXTRA) x[u] = pol.extra(s);
          }
        }
#pragma unroll
        for (int u = 0; u < U; ++u) {
          if (k0 + u < cnt) {
            pol.edge(st, v[u], w[u], x[u]);
            if ((ends_c >> (k0 + u)) & 1u) next_row();
          }
        }
      }
      idx_c = idx_n; w_c = w_n; ends_c = ends_n;
    }
  }
}

// ----------------------------------------------------------------------------- short rows: one lane group each, no edge stream
// For rows of at most a few dozen edges the bookkeeping of a flat edge stream costs more than the edges.
// Here a group of LPR lanes (16-byte slices, LPR >= 8) owns one row: lanes 0..7 of the group fetch eight
// source indices with one load, the group issues the eight row loads back to back and then reduces them;
// rows longer than eight edges take more rounds.  The slices are staged through shared memory (cp.async, 32 KB per
// CTA): the kernel is bound by the loads it keeps in flight, and without eight 16-byte slices in registers it fits
// six CTAs per SM instead of four (measured: 4.6 -> 5.6 TB/s on rows of at most 8 edges).  The groups of a warp run in lockstep (warp-wide loop
// bounds, predicated edges), so a warp never splits.
template <typename T, int LPR, class Policy>
__global__ void __launch_bounds__(THREADS, IT_SHORT_MIN_BLOCKS) stream_short_rows_kernel(StreamParams p, Policy pol) {
  constexpr int NS = Policy::NS;
  constexpr int E = IT_SHORT_EDGES;   // edges per round
  static_assert(LPR >= E, "lanes 0..7 of a group fetch the indices of a round");
  using Slice = RowSlice<T, 16>;
  const int lane = threadIdx.x & 31;
  const int t = lane % LPR, gbase = lane - t;
  pol.setup(t);
  const char *my_src = reinterpret_cast<const char *>(p.src) + (size_t)t * 16;
  const uint32_t ROWB = p.src_pitch;
  const int64_t rows_per_sweep = (int64_t)gridDim.x * (THREADS / LPR);
#if IT_SHORT_ASYNC
  __shared__ uint4 sbuf[E][THREADS];
  const uint32_t my_buf = (uint32_t)__cvta_generic_to_shared(&sbuf[0][threadIdx.x]);
#endif
  // warp-uniform loop: every group of the warp takes one row per iteration
  for (int64_t i0 = p.row_lo + (int64_t)blockIdx.x * (THREADS / LPR) + (threadIdx.x >> 5) * (32 / LPR); i0 < p.row_hi; i0 += rows_per_sweep) {
    const int64_t i = i0 + lane / LPR;
    const bool valid = i < p.row_hi;
    int64_t j0 = 0;
    int len = 0, dest = 0, owner = 0;
    if (valid) {
      const it_row_meta m = load_meta(p.meta + i);
      j0 = m.j0; len = m.len; dest = m.dest;
      if (Policy::NEEDS_OWNER) owner = __ldcs(p.owner + i);
    }
    const int maxlen = __reduce_max_sync(0xffffffffu, len);
    float st[NS];
    pol.init(st);
    if (valid) pol.begin_row(dest, owner);
    for (int k0 = 0; k0 < maxlen; k0 += E) {
      int32_t idx = 0;
      float w = 1.f;
      if (t < E && k0 + t < len) {
        idx = p.indices ? __ldcs(p.indices + j0 + k0 + t) : (int32_t)(j0 + k0 + t);
        if (Policy::WEIGHTED) w = __ldcs(p.weights + j0 + k0 + t);
      }
      float ww[E], xx[E];
#if IT_SHORT_ASYNC
      // the slices travel through shared memory (cp.async) instead of registers: each lane later reads back exactly
      // the bytes it copied, so waiting for its own copy group is all the synchronisation there is, and the
      // registers saved buy more resident warps
#pragma unroll
      for (int k = 0; k < E; ++k) {
        const uint32_t s = (uint32_t)__shfl_sync(0xffffffffu, idx, gbase + k);
        ww[k] = Policy::WEIGHTED ? __shfl_sync(0xffffffffu, w, gbase + k) : 1.f;
        xx[k] = 0.f;
        if (k0 + k < len) {
          asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(my_buf + (uint32_t)k * (THREADS * 16)), "l"(my_src + (uint64_t)s * ROWB) : "memory");
          if (Policy::HAS_EXTRA) xx[k] = pol.extra(s);
        }
      }
      asm volatile("cp.async.commit_group;" ::: "memory");
      asm volatile("cp.async.wait_group 0;" ::: "memory");
#pragma unroll
      for (int k = 0; k < E; ++k)
        if (k0 + k < len) {
          uint4 v;
          asm volatile("ld.shared.v4.b32 {%0, %1, %2, %3}, [%4];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "r"(my_buf + (uint32_t)k * (THREADS * 16)) : "memory");
          pol.edge(st, v, ww[k], xx[k]);
        }
#else
      typename Slice::Raw v[E];
#pragma unroll
      for (int k = 0; k < E; ++k) {
        const uint32_t s = (uint32_t)__shfl_sync(0xffffffffu, idx, gbase + k);
        ww[k] = Policy::WEIGHTED ? __shfl_sync(0xffffffffu, w, gbase + k) : 1.f;
        xx[k] = 0.f;
        if (k0 + k < len) {
          v[k] = Slice::load(my_src + (uint64_t)s * ROWB);
          if (Policy::HAS_EXTRA) xx[k] = pol.extra(s);
        }
      }
#pragma unroll
      for (int k = 0; k < E; ++k)
        if (k0 + k < len) pol.edge(st, v[k], ww[k], xx[k]);
#endif
    }
    if (valid) pol.end_row(st, dest, owner, len);
  }
}

// The same kernel with its three dependent loads (row record -> source indices -> source rows) overlapped across
// rounds: a round is one batch of up to E edges of one row per lane group.  While the source rows of the current
// round are in flight, the indices of the next round (of the same row if it is longer than E, else of the group's
// next row) and the record of the row after next are in flight too, so that only one memory round trip per round
// is exposed instead of three.  Costs a dozen registers per thread (four resident CTAs per SM instead of six).
// Measured against the plain loop above: 3 % to 6 % less time on the 128-byte rows of at most 32 edges, 2 % on
// the 256-byte fp32 rows, none on the GAT rows (that kernel is bound by its issue slots, not by exposed latency).
#ifndef IT_SHORT_PIPE
#define IT_SHORT_PIPE 1          // 1: short rows take the pipelined kernel
#endif
#ifndef IT_SHORT_PIPE_BLOCKS
#define IT_SHORT_PIPE_BLOCKS 4   // resident CTAs per SM the pipelined kernel's register budget is set for (measured: five spill and gain nothing)
#endif
#ifndef IT_RING_SINGLE_ROW
#define IT_RING_SINGLE_ROW 1     // the ring kernel walks a batch of one row as a stream without ends of rows
#endif
#ifndef IT_SHORT_PIPE_WAVES
#define IT_SHORT_PIPE_WAVES 1    // grid = SMs x resident CTAs x this: every CTA is resident from the start and walks its rows
#endif
template <typename T, int LPR, class Policy>
__global__ void __launch_bounds__(THREADS, IT_SHORT_PIPE_BLOCKS) stream_short_rows_pipe_kernel(StreamParams p, Policy pol) {
  constexpr int NS = Policy::NS;
  constexpr int E = IT_SHORT_EDGES;   // edges per round
  static_assert(LPR >= E, "lanes 0..7 of a group fetch the indices of a round");
  const int lane = threadIdx.x & 31;
  const int t = lane % LPR, gbase = lane - t;
  pol.setup(t);
  const char *my_src = reinterpret_cast<const char *>(p.src) + (size_t)t * 16;
  const uint32_t ROWB = p.src_pitch;
  const int64_t sweep = (int64_t)gridDim.x * (THREADS / LPR);
  __shared__ uint4 sbuf[E][THREADS];
  const uint32_t my_buf = (uint32_t)__cvta_generic_to_shared(&sbuf[0][threadIdx.x]);

  struct Row { int64_t j0; int len, dest, owner; };
  // the row this lane group takes in the sweep that starts at i0 (len 0: none; rows of these buckets have edges)
  auto load_row = [&](int64_t i0) {
    Row r{0, 0, 0, 0};
    const int64_t i = i0 + lane / LPR;
    if (i < p.row_hi) {
      const it_row_meta m = load_meta(p.meta + i);
      r.j0 = m.j0; r.len = m.len; r.dest = m.dest;
      if (Policy::NEEDS_OWNER) r.owner = __ldcs(p.owner + i);
    }
    return r;
  };
  // lanes 0..E-1 of the group: source index (and weight) of edge k + t of row r
  auto load_idx = [&](const Row &r, int k, int32_t &idx, float &w) {
    idx = 0; w = 1.f;
    if (t < E && k + t < r.len) {
      idx = p.indices ? __ldcs(p.indices + r.j0 + k + t) : (int32_t)(r.j0 + k + t);
      if (Policy::WEIGHTED) w = __ldcs(p.weights + r.j0 + k + t);
    }
  };

  int64_t i0 = p.row_lo + (int64_t)blockIdx.x * (THREADS / LPR) + (threadIdx.x >> 5) * (32 / LPR);   // warp-uniform
  Row cur = load_row(i0), nxt = load_row(i0 + sweep);
  int32_t idx_c; float w_c;
  load_idx(cur, 0, idx_c, w_c);
  for (; i0 < p.row_hi; i0 += sweep) {
    const Row nn = load_row(i0 + 2 * sweep);   // in flight for two rows
    const int maxlen = __reduce_max_sync(0xffffffffu, cur.len);
    float st[NS];
    pol.init(st);
    if (cur.len > 0) pol.begin_row(cur.dest, cur.owner);
    for (int k0 = 0; k0 < maxlen; k0 += E) {
      // the indices of the next round, in flight while this round's rows are
      int32_t idx_n; float w_n;
      if (k0 + E < maxlen) load_idx(cur, k0 + E, idx_n, w_n);
      else load_idx(nxt, 0, idx_n, w_n);
      float ww[E], xx[E];
#pragma unroll
      for (int k = 0; k < E; ++k) {
        const uint32_t s = (uint32_t)__shfl_sync(0xffffffffu, idx_c, gbase + k);
        ww[k] = Policy::WEIGHTED ? __shfl_sync(0xffffffffu, w_c, gbase + k) : 1.f;
        xx[k] = 0.f;
        if (k0 + k < cur.len) {
          asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(my_buf + (uint32_t)k * (THREADS * 16)), "l"(my_src + (uint64_t)s * ROWB) : "memory");
          if (Policy::HAS_EXTRA) xx[k] = pol.extra(s);
        }
      }
      asm volatile("cp.async.commit_group;" ::: "memory");
      asm volatile("cp.async.wait_group 0;" ::: "memory");
#pragma unroll
      for (int k = 0; k < E; ++k) {
        if (k0 + k < cur.len) {
          uint4 v;
          asm volatile("ld.shared.v4.b32 {%0, %1, %2, %3}, [%4];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "r"(my_buf + (uint32_t)k * (THREADS * 16)) : "memory");
          pol.edge(st, v, ww[k], xx[k]);
        }
      }
      idx_c = idx_n; w_c = w_n;
    }
    if (cur.len > 0) pol.end_row(st, cur.dest, cur.owner, cur.len);
    cur = nxt; nxt = nn;
  }
}

// Rows of at most E edges (one round each), two rows per lane group in flight: the copies of the group's next row are
// issued before the wait for the current row's, through two staging buffers in shared memory (64 KB per CTA, three
// resident CTAs per SM).  Rows this short carry few bytes each (three edges on average in a power-law graph), and
// with one row per lane group in flight the kernel does not keep enough bytes in flight to fill the memory system.
// Row records are loaded four rows ahead and source indices two rows ahead.  Policies without a per-edge scalar only.
#ifndef IT_SHORT_PIPE2
#define IT_SHORT_PIPE2 1
#endif
#ifndef IT_SHORT_PIPE2_AVG
#define IT_SHORT_PIPE2_AVG 4     // buckets whose rows hold at most this many edges on average take the kernel
#endif
#ifndef IT_SHORT_PIPE2_BLOCKS
#define IT_SHORT_PIPE2_BLOCKS 3
#endif
template <typename T, int LPR, class Policy>
__global__ void __launch_bounds__(THREADS, IT_SHORT_PIPE2_BLOCKS) stream_tiny_rows_kernel(StreamParams p, Policy pol) {
  constexpr int NS = Policy::NS;
  constexpr int E = IT_SHORT_EDGES;
  static_assert(LPR >= E && !Policy::HAS_EXTRA, "lanes 0..7 of a group fetch the indices of a row; no per-edge scalars");
  extern __shared__ uint4 tiny_buf[];   // [2][E][THREADS]
  const int lane = threadIdx.x & 31;
  const int t = lane % LPR, gbase = lane - t;
  pol.setup(t);
  const char *my_src = reinterpret_cast<const char *>(p.src) + (size_t)t * 16;
  const uint32_t ROWB = p.src_pitch;
  const int64_t sweep = (int64_t)gridDim.x * (THREADS / LPR);
  const uint32_t my_buf = (uint32_t)__cvta_generic_to_shared(&tiny_buf[threadIdx.x]);
  constexpr uint32_t SLOT = THREADS * 16, BUF = E * SLOT;

  struct Row { int64_t j0; int len, dest, owner; };
  auto load_row = [&](int64_t i0) {
    Row r{0, 0, 0, 0};
    const int64_t i = i0 + lane / LPR;
    if (i < p.row_hi) {
      const it_row_meta m = load_meta(p.meta + i);
      r.j0 = m.j0; r.len = m.len; r.dest = m.dest;
      if (Policy::NEEDS_OWNER) r.owner = __ldcs(p.owner + i);
    }
    return r;
  };
  auto load_idx = [&](const Row &r, int32_t &idx, float &w) {
    idx = 0; w = 1.f;
    if (t < E && t < r.len) {
      idx = p.indices ? __ldcs(p.indices + r.j0 + t) : (int32_t)(r.j0 + t);
      if (Policy::WEIGHTED) w = __ldcs(p.weights + r.j0 + t);
    }
  };
  auto issue = [&](const Row &r, int32_t idx, uint32_t buf) {
#pragma unroll
    for (int k = 0; k < E; ++k) {
      const uint32_t s = (uint32_t)__shfl_sync(0xffffffffu, idx, gbase + k);
      if (k < r.len)
        asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(buf + (uint32_t)k * SLOT), "l"(my_src + (uint64_t)s * ROWB) : "memory");
    }
    asm volatile("cp.async.commit_group;" ::: "memory");
  };

  int64_t i0 = p.row_lo + (int64_t)blockIdx.x * (THREADS / LPR) + (threadIdx.x >> 5) * (32 / LPR);   // warp-uniform
  Row r0 = load_row(i0), r1 = load_row(i0 + sweep), r2 = load_row(i0 + 2 * sweep), r3 = load_row(i0 + 3 * sweep);
  int32_t idx0, idx1; float w0, w1;
  load_idx(r0, idx0, w0);
  load_idx(r1, idx1, w1);
  uint32_t cur = my_buf, oth = my_buf + BUF;
  issue(r0, idx0, cur);
  for (; i0 < p.row_hi; i0 += sweep) {
    const Row r4 = load_row(i0 + 4 * sweep);
    int32_t idx2; float w2;
    load_idx(r2, idx2, w2);
    issue(r1, idx1, oth);                      // the next row's copies, in flight while this row is reduced
    float st[NS];
    pol.init(st);
    if (r0.len > 0) pol.begin_row(r0.dest, r0.owner);
    asm volatile("cp.async.wait_group 1;" ::: "memory");   // this row's copies have landed
#pragma unroll
    for (int k = 0; k < E; ++k) {
      const float ww = Policy::WEIGHTED ? __shfl_sync(0xffffffffu, w0, gbase + k) : 1.f;
      if (k < r0.len) {
        uint4 v;
        asm volatile("ld.shared.v4.b32 {%0, %1, %2, %3}, [%4];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "r"(cur + (uint32_t)k * SLOT) : "memory");
        pol.edge(st, v, ww, 0.f);
      }
    }
    if (r0.len > 0) pol.end_row(st, r0.dest, r0.owner, r0.len);
    r0 = r1; r1 = r2; r2 = r3; r3 = r4;
    idx0 = idx1; w0 = w1; idx1 = idx2; w1 = w2;
    const uint32_t sw = cur; cur = oth; oth = sw;
  }
  asm volatile("cp.async.wait_group 0;" ::: "memory");
}

// ----------------------------------------------------------------------------- very long rows: one CTA each
template <typename T, int SB, int LPR, class Policy>
__global__ void __launch_bounds__(THREADS, IT_GATHER_MIN_BLOCKS) stream_cta_kernel(StreamParams p, Policy pol) {
  constexpr int NS = Policy::NS;
  constexpr int WARPS = THREADS / 32;
  constexpr int SLOTS = 32 / LPR;
  constexpr int U = UNROLL * (16 / SB);   // the same bytes in flight per lane whatever the slice width
  __shared__ float red[WARPS][LPR][NS];
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int slot = lane / LPR, t = lane % LPR;
  pol.setup(t);
  const char *my_src = reinterpret_cast<const char *>(p.src) + (size_t)t * SB;
  using Slice = RowSlice<T, SB>;
  const uint32_t row_bytes = p.src_pitch;
  for (int64_t i = p.row_lo + blockIdx.x; i < p.row_hi; i += gridDim.x) {
    const it_row_meta m = load_meta(p.meta + i);
    const int32_t owner = Policy::NEEDS_OWNER ? __ldcs(p.owner + i) : 0;
    const int64_t j0 = m.j0, j1 = m.j0 + m.len;
    const int64_t chunk = ((int64_t)m.len + WARPS - 1) / WARPS;
    int64_t a = j0 + warp * chunk, b = a + chunk;
    if (a > j1) a = j1;
    if (b > j1) b = j1;
    float st[NS];
    pol.init(st);
    pol.begin_row(m.dest, owner);
    // edges [a, b) with the whole warp: SLOTS edges at once, index chunk of 32 prefetched one step ahead
    auto load_chunk = [&](int64_t base, int32_t &idx, float &w) {
      idx = 0; w = 1.f;
      if (base + lane < b) {
        idx = p.indices ? __ldcs(p.indices + base + lane) : (int32_t)(base + lane);
        if (Policy::WEIGHTED) w = __ldcs(p.weights + base + lane);
      }
    };
    int32_t idx_c, idx_n;
    float w_c, w_n;
    load_chunk(a, idx_c, w_c);
    for (int64_t base = a; base < b; base += 32) {
      load_chunk(base + 32, idx_n, w_n);
      const int cnt = (int)((b - base) < 32 ? (b - base) : 32);
      for (int k0 = 0; k0 < cnt; k0 += SLOTS * U) {
        typename Slice::Raw v[U];
        float w[U], x[U];
        bool ok[U];
#pragma unroll
        for (int u = 0; u < U; ++u) {
          const int e = k0 + u * SLOTS + slot;
          const uint32_t s = (uint32_t)__shfl_sync(0xffffffffu, idx_c, e & 31);
          w[u] = Policy::WEIGHTED ? __shfl_sync(0xffffffffu, w_c, e & 31) : 1.f;
          ok[u] = e < cnt;
          x[u] = 0.f;
          if (ok[u]) {
            v[u] = Slice::load(my_src + (uint64_t)s * row_bytes);
            if (Policy::HAS_EXTRA) x[u] = pol.extra(s);
          }
        }
#pragma unroll
        for (int u = 0; u < U; ++u)
          if (ok[u]) pol.edge(st, v[u], w[u], x[u]);
      }
      idx_c = idx_n; w_c = w_n;
    }
    // fold the SLOTS edge slots into slot 0, lower slot first
#pragma unroll
    for (int o = 16; o >= LPR; o >>= 1) {
      float other[NS];
#pragma unroll
      for (int k = 0; k < NS; ++k) other[k] = __shfl_xor_sync(0xffffffffu, st[k], o);
      pol.merge(st, other);   // only slot 0 is read at the end, and it is always the first operand
    }
    __syncthreads();  // red[] free again
    if (lane < LPR) {
#pragma unroll
      for (int k = 0; k < NS; ++k) red[warp][lane][k] = st[k];
    }
    __syncthreads();
    if (warp == 0 && lane < LPR) {
      for (int w = 1; w < WARPS; ++w) {
        float other[NS];
#pragma unroll
        for (int k = 0; k < NS; ++k) other[k] = red[w][lane][k];
        pol.merge(st, other);
      }
      pol.end_row(st, m.dest, owner, m.len);
    }
  }
}

// ----------------------------------------------------------------------------- empty rows
template <typename T, int SB, int LPR, class Policy>
__global__ void __launch_bounds__(THREADS) stream_empty_kernel(StreamParams p, Policy pol) {
  constexpr int NS = Policy::NS;
  const int t = threadIdx.x % LPR;
  pol.setup(t);
  const int64_t groups_total = (int64_t)gridDim.x * (THREADS / LPR);
  for (int64_t i = p.row_lo + (int64_t)blockIdx.x * (THREADS / LPR) + threadIdx.x / LPR; i < p.row_hi; i += groups_total) {
    const it_row_meta m = load_meta(p.meta + i);
    const int32_t owner = Policy::NEEDS_OWNER ? __ldcs(p.owner + i) : 0;
    float st[NS];
    pol.init(st);
    pol.begin_row(m.dest, owner);
    pol.end_row(st, m.dest, owner, 0);
  }
}

}  // namespace it_stream

#include "stream_ring.cuh"

namespace it_stream {

// The opt-in to more than 48 KB of dynamic shared memory is an attribute of the kernel ON ONE DEVICE: it is set once
// per device (the current one), remembered in a bit mask that any thread may update.
template <class Kernel>
it_status allow_dynamic_smem(Kernel kernel, int smem, std::atomic<uint64_t> &done) {
  int dev = -1;
  IT_CUDA_TRY(cudaGetDevice(&dev));
  const uint64_t bit = (dev >= 0 && dev < 64) ? (uint64_t)1 << dev : 0;   // ordinals beyond 63 are configured on every launch
  if (bit == 0 || !(done.load(std::memory_order_acquire) & bit)) {
    IT_CUDA_TRY(cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, smem));
    done.fetch_or(bit, std::memory_order_release);
  }
  return IT_OK;
}

// ----------------------------------------------------------------------------- bucket dispatch
// Longest rows first so that the tail of the launch sequence is made of short rows.
// bytes_of(bucket, rows) gives the algorithmic bytes of a launch; kid_* the instrumentation ids.
// Only the buckets whose bound lies in (bound_lo, bound_hi] are launched: callers may give long and short
// rows different slice widths.
// `counters`: IT_MAX_BUCKETS device words of scratch (or NULL): the ring kernel of bucket b hands out its batches from
// word b, which is zeroed here, in stream order, before the launches.
template <typename T, int SB, int LPR, class Policy, class BytesF>
it_status launch_buckets(const it_graph *g, StreamParams p, const Policy &pol, BytesF bytes_of, int kid_cta, int kid_rows,
                         int kid_empty, int64_t bound_lo, int64_t bound_hi, int *counters, cudaStream_t st) {
  constexpr bool RING = SB * LPR >= 128;   // rows of 128 bytes and more are staged through shared memory
#if !IT_RING_DYNAMIC
  counters = nullptr;
#endif
  if (RING && counters) IT_CUDA_TRY(cudaMemsetAsync(counters, 0, IT_MAX_BUCKETS * sizeof(int), st));
  p.counter = nullptr;
  for (int b = g->n_buckets - 1; b >= 0; --b) {
    const int64_t lo = g->h_bucket_offsets[b], hi = g->h_bucket_offsets[b + 1];
    if (hi <= lo || g->bucket_bounds[b] <= bound_lo || g->bucket_bounds[b] > bound_hi) continue;
    p.row_lo = lo; p.row_hi = hi;
    const int64_t bound = g->bucket_bounds[b];
    const int64_t rows = hi - lo;
    const int64_t max_blocks = (int64_t)g->num_sms * IT_GATHER_MIN_BLOCKS * 2;
    const double bytes = bytes_of(b, rows);
    if (bound == 0) {
      int64_t want = (rows + (THREADS / LPR) - 1) / (THREADS / LPR);
      unsigned blocks = (unsigned)(want < max_blocks ? want : max_blocks);
      IT_LAUNCH(kid_empty, bytes, 0, st, stream_empty_kernel<T, SB, LPR, Policy><<<blocks, THREADS, 0, st>>>(p, pol));
    } else if (bound > IT_GATHER_CTA_ABOVE) {
      if constexpr (RING) {
        constexpr int smem = (THREADS / 32) * ring_bytes_per_warp<SB, Policy::HAS_EXTRA>();
        static std::atomic<uint64_t> configured{0};   // per template instance: one bit per device ordinal
        IT_TRY(allow_dynamic_smem(stream_cta_ring_kernel<T, SB, LPR, Policy>, smem, configured));
        // one CTA per row as far as the grid allows: the hardware hands out rows as CTAs retire
        unsigned blocks = (unsigned)(rows < (1 << 20) ? rows : (1 << 20));
        IT_LAUNCH(kid_cta, bytes, 0, st, stream_cta_ring_kernel<T, SB, LPR, Policy><<<blocks, THREADS, smem, st>>>(p, pol));
      } else {
        unsigned blocks = (unsigned)(rows < max_blocks ? rows : max_blocks);
        IT_LAUNCH(kid_cta, bytes, 0, st, stream_cta_kernel<T, SB, LPR, Policy><<<blocks, THREADS, 0, st>>>(p, pol));
      }
    } else {
      // about 256 edges per batch at most: 32 rows of <= 8 edges, 8 rows of <= 32, one longer row (measured: walking
      // several longer rows as one stream, to pay the dependent loads at the start of a row once per batch, is slower)
      int br = bound <= 8 ? 32 : (bound <= 32 ? 8 : 1);
      if constexpr (SB == 16 && (LPR == 8 || (LPR == 16 && IT_SHORT_256 != 0))) {   // 128-byte rows (and 256-byte rows)
        if (bound <= IT_SHORT_BELOW) {   // one lane group per row
          const int64_t want = (rows + (THREADS / LPR) - 1) / (THREADS / LPR);
          if constexpr (IT_SHORT_PIPE2 != 0 && !Policy::HAS_EXTRA) {
            // one round per row, and rows so short (at most IT_SHORT_PIPE2_AVG edges on average) that one row per lane
            // group leaves the memory system short of bytes in flight: two rows per lane group in flight (measured:
            // 2.7 % less time on power-law rows of 2.9 edges on average, 7 % more on rows of 4.9)
            if (bound <= IT_SHORT_EDGES && g->h_bucket_edges[b] <= (int64_t)IT_SHORT_PIPE2_AVG * rows) {
              constexpr int smem = 2 * IT_SHORT_EDGES * THREADS * 16;
              static std::atomic<uint64_t> configured2{0};
              IT_TRY(allow_dynamic_smem(stream_tiny_rows_kernel<T, LPR, Policy>, smem, configured2));
              const int64_t tiny_max = (int64_t)g->num_sms * IT_SHORT_PIPE2_BLOCKS;
              unsigned blocks = (unsigned)(want < tiny_max ? want : tiny_max);
              IT_LAUNCH(kid_rows, bytes, 0, st, stream_tiny_rows_kernel<T, LPR, Policy><<<blocks, THREADS, smem, st>>>(p, pol));
              continue;
            }
          }
#if IT_SHORT_PIPE
          const int64_t short_max = (int64_t)g->num_sms * IT_SHORT_PIPE_BLOCKS * IT_SHORT_PIPE_WAVES;
          unsigned blocks = (unsigned)(want < short_max ? want : short_max);
          IT_LAUNCH(kid_rows, bytes, 0, st, stream_short_rows_pipe_kernel<T, LPR, Policy><<<blocks, THREADS, 0, st>>>(p, pol));
#else
          const int64_t short_max = (int64_t)g->num_sms * IT_SHORT_MIN_BLOCKS * 4;
          unsigned blocks = (unsigned)(want < short_max ? want : short_max);
          IT_LAUNCH(kid_rows, bytes, 0, st, stream_short_rows_kernel<T, LPR, Policy><<<blocks, THREADS, 0, st>>>(p, pol));
#endif
          continue;
        }
      }
      if constexpr (RING) {   // a whole warp per batch
        constexpr int smem = (THREADS / 32) * ring_bytes_per_warp<SB, Policy::HAS_EXTRA>();
        static std::atomic<uint64_t> configured{0}, configured1{0};   // per template instance: one bit per device ordinal
        const bool single = IT_RING_SINGLE_ROW && br == 1;
        if (single) IT_TRY(allow_dynamic_smem(stream_rows_ring_kernel<T, SB, LPR, Policy, true>, smem, configured1));
        else IT_TRY(allow_dynamic_smem(stream_rows_ring_kernel<T, SB, LPR, Policy, false>, smem, configured));
        p.batch_rows = br;
        const int64_t batches = (rows + br - 1) / br;
        // with a counter every CTA is resident from the start and its warps claim batches as they finish (rows of one
        // bucket differ in length by up to a factor of eight, and a fixed stride leaves warps idle at the end)
        p.counter = counters ? counters + b : nullptr;
        const int64_t ring_max = (int64_t)g->num_sms * IT_RING_MIN_BLOCKS * (counters ? 1 : 2);
        const int64_t want = (batches + (THREADS / 32) - 1) / (THREADS / 32);
        unsigned blocks = (unsigned)(want < ring_max ? want : ring_max);
        const int64_t per_warp = batches / ((int64_t)blocks * (THREADS / 32));
        p.claim = (int)(per_warp / IT_RING_CLAIMS_PER_WARP < 1 ? 1 : (per_warp / IT_RING_CLAIMS_PER_WARP > 4096 ? 4096 : per_warp / IT_RING_CLAIMS_PER_WARP));
        if (single) IT_LAUNCH(kid_rows, bytes, 0, st, stream_rows_ring_kernel<T, SB, LPR, Policy, true><<<blocks, THREADS, smem, st>>>(p, pol));
        else IT_LAUNCH(kid_rows, bytes, 0, st, stream_rows_ring_kernel<T, SB, LPR, Policy, false><<<blocks, THREADS, smem, st>>>(p, pol));
        p.counter = nullptr;
      } else {                                // a group of LPR lanes per batch
        if (br > LPR) br = LPR;
        p.batch_rows = br;
        const int64_t batches = (rows + br - 1) / br;
        int64_t want = (batches + (THREADS / LPR) - 1) / (THREADS / LPR);
        unsigned blocks = (unsigned)(want < max_blocks ? want : max_blocks);
        IT_LAUNCH(kid_rows, bytes, 0, st, stream_rows_kernel<T, SB, LPR, Policy><<<blocks, THREADS, 0, st>>>(p, pol));
      }
    }
  }
  IT_CUDA_TRY(cudaGetLastError());
  return IT_OK;
}

// Pick the slice width and group size for a row of `row_bytes` bytes and call
// f.template operator()<SB, LPR>(bound_lo, bound_hi) for the buckets that take them.  Unless `wide` is false,
// rows of 128 bytes use 16-byte slices throughout and rows of 256 bytes use them for their long rows, with
// one slice per lane for the short ones (measured: the cheaper end of row wins there).
#ifndef IT_WIDE_ABOVE
#define IT_WIDE_ABOVE 32   // buckets of rows longer than this use 16-byte slices
#endif
template <class F>
it_status dispatch_row_bytes(int row_bytes, bool wide, F f) {
  constexpr int64_t ALL = INT64_MAX;
  switch (row_bytes) {
    case 512: return f.template operator()<16, 32>(-1, ALL);
    case 256:
      if (!wide) return f.template operator()<8, 32>(-1, ALL);
      if (IT_SHORT_256) {   // every row with edges takes 16-byte slices (short rows: the lane-group kernel); <8, 32> keeps the empty rows
        IT_TRY((f.template operator()<16, 16>(0, ALL)));
        return f.template operator()<8, 32>(-1, 0);
      }
      IT_TRY((f.template operator()<16, 16>(IT_WIDE_ABOVE, ALL)));
      return f.template operator()<8, 32>(-1, IT_WIDE_ABOVE);
    case 128:
      if (!wide) return f.template operator()<4, 32>(-1, ALL);
      return f.template operator()<16, 8>(-1, ALL);
    case 64: return f.template operator()<4, 16>(-1, ALL);
    case 32: return f.template operator()<4, 8>(-1, ALL);
    case 16: return f.template operator()<4, 4>(-1, ALL);
  }
  it_set_error("feature row of %d bytes is not 16, 32, 64, 128, 256 or 512 bytes", row_bytes);
  return IT_ERR_UNSUPPORTED;
}

}  // namespace it_stream
