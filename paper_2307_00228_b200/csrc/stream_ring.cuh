// Row streaming through shared memory, for feature rows of 128, 256 and 512 bytes.
//
// A row is cut into lane slices of SB = 4, 8 or 16 bytes, so it takes LPR = row bytes / SB lanes and a warp
// moves SL = 32 / LPR rows ("edge slots") with every instruction: lane = slot * LPR + t fetches slice t of
// the source row of edge (g * SL + slot) of the flat edge stream.  Wide slices (SL > 1) cost the fewest
// instructions per edge and suit long rows; SL = 1 has the cheapest end of row and suits short ones.
// The rows are copied asynchronously (cp.async) into a small per-warp ring of stages in shared memory; while one stage is
// reduced the copies of the others are in flight.  Each lane later reads back exactly the bytes it copied,
// so cp.async.wait_group alone orders the copy and the read and no warp synchronisation is needed.
//
// Every slot keeps its own partial state of the current row; when a row ends the slots are folded with
// Policy::merge (lower slot first) and slot 0 runs the row's epilogue.  Edges of one group of SL that
// lie on either side of an end of row are applied in order: up to the end, fold, epilogue, then the rest.
//
// Included by stream.cuh (uses its StreamParams, RowSlice, load_meta).
#pragma once

namespace it_stream {

template <int SB>
__device__ __forceinline__ void cp_async_slice(uint32_t smem_dst, const void *gmem_src) {   // smem_dst: shared-window address
  if constexpr (SB == 16) asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(smem_dst), "l"(gmem_src) : "memory");
  else if constexpr (SB == 8) asm volatile("cp.async.ca.shared.global [%0], [%1], 8;" ::"r"(smem_dst), "l"(gmem_src) : "memory");
  else asm volatile("cp.async.ca.shared.global [%0], [%1], 4;" ::"r"(smem_dst), "l"(gmem_src) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int N>
__device__ __forceinline__ void cp_async_wait() { asm volatile("cp.async.wait_group %0;" ::"n"(N) : "memory"); }
template <int SB>
__device__ __forceinline__ typename SliceRaw<SB>::type lds_slice(uint32_t a) {
  if constexpr (SB == 16) {
    uint4 v;
    asm volatile("ld.shared.v4.b32 {%0, %1, %2, %3}, [%4];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "r"(a) : "memory");
    return v;
  } else if constexpr (SB == 8) {
    uint2 v;
    asm volatile("ld.shared.v2.b32 {%0, %1}, [%2];" : "=r"(v.x), "=r"(v.y) : "r"(a) : "memory");
    return v;
  } else {
    uint32_t v;
    asm volatile("ld.shared.b32 %0, [%1];" : "=r"(v) : "r"(a) : "memory");
    return v;
  }
}
__device__ __forceinline__ float lds_f32(uint32_t a) {
  float v;
  asm volatile("ld.shared.f32 %0, [%1];" : "=f"(v) : "r"(a) : "memory");
  return v;
}

// Geometry of the ring for rows of LPR slices of SB bytes.  A stage always holds IT_RING_STAGE_ROWS * 512 bytes of rows.
template <int SB, int LPR>
struct RingGeom {
  static constexpr int SL = 32 / LPR;                        // edge slots: rows a warp moves per instruction
  static constexpr int ROWB = LPR * SB;                      // bytes of a row that are gathered (the source rows may be wider)
  static constexpr int GB = 32 * SB;                         // bytes of a group: what one instruction moves
  static constexpr int R = IT_RING_STAGE_ROWS * (16 / SB);   // groups per stage
  static constexpr int GE = R * SL;                          // edges per stage
  static constexpr int S = IT_RING_STAGES;
  static constexpr int AHEAD = (S - 1) * GE;                 // the stage being filled is this many edges ahead of the one reduced
  static_assert(GE <= 16 && 32 % GE == 0 && AHEAD <= 32, "an index chunk of 32 edges is a whole number of stages and the fill reaches at most into the next chunk");
};
template <int SB, bool HAS_EXTRA> constexpr int ring_bytes_per_warp() {
  return IT_RING_STAGES * IT_RING_STAGE_ROWS * (512 + (HAS_EXTRA ? (16 / SB) * 128 : 0));
}

// What a warp needs to drive its ring: addresses, the fill of a stage and the reduction of one group.
template <typename T, int SB, int LPR, class Policy>
struct RingWarp {
  using G = RingGeom<SB, LPR>;
  using Raw = typename SliceRaw<SB>::type;
  uint32_t my_ring, my_xring;   // shared-window addresses of my slice / my per-edge scalar in group 0 of stage 0
  const char *my_src;           // my slice of source row 0
  uint32_t pitch;               // bytes from one source row to the next
  int slot;

  __device__ __forceinline__ void setup(uint32_t ring_base, const void *src, uint32_t src_pitch, int lane) {
    pitch = src_pitch;
    my_ring = ring_base + lane * SB;
    my_xring = ring_base + G::S * G::R * G::GB + lane * 4;
    my_src = reinterpret_cast<const char *>(src) + (size_t)(lane % LPR) * SB;
    slot = lane / LPR;
  }
  // copy the rows of edges [k0, k0 + n) of the chunk whose indices sit in idxreg (one per lane) into a stage
  __device__ __forceinline__ void fill(const Policy &pol, int stage, int32_t idxreg, int k0, int n) const {
    const uint32_t d = my_ring + stage * (G::R * G::GB);
    const uint32_t dx = my_xring + stage * (G::R * 128);
    if (n == G::GE) {
#pragma unroll
      for (int u = 0; u < G::R; ++u) {
        const uint32_t s = (uint32_t)__shfl_sync(0xffffffffu, idxreg, k0 + u * G::SL + slot);
        cp_async_slice<SB>(d + u * G::GB, my_src + (uint64_t)s * pitch);
        if (Policy::HAS_EXTRA) cp_async_slice<4>(dx + u * 128, pol.extra_ptr(s));
      }
    } else {
      for (int u = 0; u * G::SL < n; ++u) {
        const uint32_t s = (uint32_t)__shfl_sync(0xffffffffu, idxreg, k0 + u * G::SL + slot);
        if (u * G::SL + slot < n) {
          cp_async_slice<SB>(d + u * G::GB, my_src + (uint64_t)s * pitch);
          if (Policy::HAS_EXTRA) cp_async_slice<4>(dx + u * 128, pol.extra_ptr(s));
        }
      }
    }
  }
  // fold the slots' states into slot 0, lower slot first
  __device__ __forceinline__ void fold(const Policy &pol, float (&st)[Policy::NS]) const {
#pragma unroll
    for (int o = 16; o >= LPR; o >>= 1) {
      float other[Policy::NS];
#pragma unroll
      for (int k = 0; k < Policy::NS; ++k) other[k] = __shfl_xor_sync(0xffffffffu, st[k], o);
      pol.merge(st, other);   // only slot 0 is read afterwards, and there st is always the lower slot
    }
  }
};

// The walk over one flat edge stream of `total` (>= 1) edges: index chunks of 32 edges prefetched one ahead,
// stages filled AHEAD edges in front of the one being reduced.
//   load_chunk(base, idx, w, ends): lane q gets the source index / weight of edge base + q (0 / 1 past the end)
//                                   and the warp-uniform mask of the edges of the chunk that end a row;
//   finish_row():                   warp-uniform; folds the slots, runs the row's epilogue and starts the next row.
template <typename T, int SB, int LPR, class Policy, class LoadChunk, class FinishRow>
__device__ __forceinline__ void ring_stream(const RingWarp<T, SB, LPR, Policy> &rw, const Policy &pol, float (&st)[Policy::NS], int total,
                                            LoadChunk load_chunk, FinishRow finish_row) {
  using G = RingGeom<SB, LPR>;
  using Raw = typename SliceRaw<SB>::type;
  constexpr int SL = G::SL, GE = G::GE, R = G::R, S = G::S, AHEAD = G::AHEAD, GB = G::GB;
  const int slot = rw.slot;

  // reduce the edges [k0, k0 + n) of the current chunk out of the stage at (sr, sx)
  auto reduce = [&](int k0, int n, uint32_t sr, uint32_t sx, float w_c, unsigned ends_c) {
    const unsigned e = (ends_c >> k0) & ((1u << GE) - 1u);   // rows that end inside this stage (GE <= 16)
    if (n == GE && e == 0) {
#pragma unroll
      for (int u = 0; u < R; ++u) {
        const Raw raw = lds_slice<SB>(sr + u * GB);
        const float w = Policy::WEIGHTED ? __shfl_sync(0xffffffffu, w_c, k0 + u * SL + slot) : 1.f;
        const float x = Policy::HAS_EXTRA ? lds_f32(sx + u * 128) : 0.f;
        pol.edge(st, raw, w, x);
      }
    } else {
      for (int u = 0; u * SL < n; ++u) {
        const Raw raw = lds_slice<SB>(sr + u * GB);   // lanes past the end of the stream read stale bytes and drop them
        const float w = Policy::WEIGHTED ? __shfl_sync(0xffffffffu, w_c, k0 + u * SL + slot) : 1.f;
        const float x = Policy::HAS_EXTRA ? lds_f32(sx + u * 128) : 0.f;
        unsigned gm = (e >> (u * SL)) & ((1u << SL) - 1u);   // ends of rows among this group's SL edges
        const int valid = (n - u * SL) < SL ? (n - u * SL) : SL;
        int lo = 0;   // slots below lo have applied their edge
        while (gm) {
          const int pe = __ffs(gm) - 1;
          if (slot >= lo && slot <= pe) pol.edge(st, raw, w, x);
          finish_row();
          lo = pe + 1;
          gm &= gm - 1;
        }
        if (slot >= lo && slot < valid) pol.edge(st, raw, w, x);
      }
    }
  };

  int32_t idx_c, idx_n;
  float w_c, w_n;
  unsigned ends_c, ends_n;
  load_chunk(0, idx_c, w_c, ends_c);
#pragma unroll
  for (int q = 0; q < S - 1; ++q) {   // stages 0 .. S-2
    const int k = q * GE;
    if (k < total) rw.fill(pol, q, idx_c, k, (total - k) < GE ? (total - k) : GE);
    cp_async_commit();
  }
  int cs = 0;   // stage to reduce next; the one to fill next is S - 1 stages further on
  for (int base = 0; base < total; base += 32) {
    load_chunk(base + 32, idx_n, w_n, ends_n);  // in flight while this chunk is reduced
    const int cnt = (total - base) < 32 ? (total - base) : 32;
    for (int k0 = 0; k0 < cnt; k0 += GE) {
      const int f = k0 + AHEAD;
      const int fs = cs == 0 ? S - 1 : cs - 1;
      if (f < 32) {
        const int left = cnt - f;
        if (left > 0) rw.fill(pol, fs, idx_c, f, left < GE ? left : GE);
      } else {
        const int left = total - (base + f);
        if (left > 0) rw.fill(pol, fs, idx_n, f - 32, left < GE ? left : GE);
      }
      cp_async_commit();
      cp_async_wait<S - 1>();
      reduce(k0, (cnt - k0) < GE ? (cnt - k0) : GE, rw.my_ring + cs * (R * GB), rw.my_xring + cs * (R * 128), w_c, ends_c);
      cs = cs + 1 == S ? 0 : cs + 1;
    }
    idx_c = idx_n; w_c = w_n; ends_c = ends_n;
  }
  cp_async_wait<0>();   // only empty groups are left
}

// ----------------------------------------------------------------------------- batches of rows per warp
// Rows handled here have at least one edge: empty rows live in their own bucket.
// SINGLE: every batch is one row (p.batch_rows == 1): the stream is the row and its end is the end of the stream, so
// there is no bookkeeping of row ends and no metadata spread over the lanes (fewer instructions per row, fewer
// registers).
template <typename T, int SB, int LPR, class Policy, bool SINGLE>
__global__ void __launch_bounds__(THREADS, IT_RING_MIN_BLOCKS) stream_rows_ring_kernel(StreamParams p, Policy pol) {
  constexpr int NS = Policy::NS;
  extern __shared__ uint4 ring_raw[];
  const int lane = threadIdx.x & 31;
  RingWarp<T, SB, LPR, Policy> rw;
  rw.setup((uint32_t)__cvta_generic_to_shared(ring_raw) + (uint32_t)(threadIdx.x >> 5) * (uint32_t)ring_bytes_per_warp<SB, Policy::HAS_EXTRA>(),
           p.src, p.src_pitch, lane);
  const int slot = rw.slot;
  pol.setup(lane % LPR);
  const int64_t n_rows = p.row_hi - p.row_lo;
  const int BR = p.batch_rows;  // rows per batch, <= 32: lanes < BR hold their metadata
  const int64_t n_batches = (n_rows + BR - 1) / BR;
  const int64_t warps_total = (int64_t)gridDim.x * (THREADS / 32);

  // a warp's first batch is fixed; the following ones are claimed from the launch's counter (or, without one, follow at
  // a fixed stride).  Which warp takes a batch has no influence on the batch's result.
  // Batches are handed out in claims of p.claim consecutive batches (sized so that a warp makes about sixteen claims:
  // one atomic per batch would serialise on the counter when the rows are short).
  auto next_claim = [&](int64_t c) -> int64_t {
    if (p.counter == nullptr) return c + warps_total;
    int v = 0;
    if (lane == 0) v = atomicAdd(p.counter, 1);
    return warps_total + (int64_t)__shfl_sync(0xffffffffu, v, 0);
  };
  const int64_t CH = p.counter ? p.claim : 1;
  for (int64_t c = (int64_t)blockIdx.x * (THREADS / 32) + (threadIdx.x >> 5); c * CH < n_batches; c = next_claim(c))
  for (int64_t b = c * CH; b < (c + 1) * CH && b < n_batches; ++b) {
    if constexpr (SINGLE) {
      const it_row_meta m = load_meta(p.meta + p.row_lo + b);
      const int32_t owner = Policy::NEEDS_OWNER ? __ldcs(p.owner + p.row_lo + b) : 0;
      float st[NS];
      pol.init(st);
      pol.begin_row(m.dest, owner);
      const int64_t a = m.j0;
      const int total = m.len;
      auto load_chunk = [&](int base, int32_t &idx, float &w, unsigned &ends) {
        idx = 0; w = 1.f; ends = 0u;
        if (base + lane < total) {
          idx = p.indices ? __ldcs(p.indices + a + base + lane) : (int32_t)(a + base + lane);
          if (Policy::WEIGHTED) w = __ldcs(p.weights + a + base + lane);
        }
      };
      ring_stream<T, SB, LPR, Policy>(rw, pol, st, total, load_chunk, [] {});
      rw.fold(pol, st);
      if (slot == 0) pol.end_row(st, m.dest, owner, m.len);
    } else {
    // ---- batch metadata: lane i owns row i of the batch
    const int64_t i = p.row_lo + b * BR + lane;
    int64_t my_j0 = 0;
    int my_len = 0, my_dest = 0, my_owner = 0;
    if (lane < BR && i < p.row_hi) {
      const it_row_meta m = load_meta(p.meta + i);
      my_j0 = m.j0; my_len = m.len; my_dest = m.dest;
      if (Policy::NEEDS_OWNER) my_owner = __ldcs(p.owner + i);
    }
    int my_end = my_len;  // inclusive prefix sum of the row lengths
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      const int y = __shfl_up_sync(0xffffffffu, my_end, o);
      if (lane >= o) my_end += y;
    }
    const int total = __shfl_sync(0xffffffffu, my_end, 31);
    const int my_start = my_end - my_len;
    const int64_t j_first = __shfl_sync(0xffffffffu, my_j0, 0);

    // lane q fetches the index of edge (base + q) and learns whether it is the last edge of its row
    auto load_chunk = [&](int base, int32_t &idx, float &w, unsigned &ends) {
      const int q = base + lane;
      int row_end = total;
      int64_t j = j_first + q;
      if (BR > 1) {   // which row of the batch edge q belongs to
        int lo = 0;
#pragma unroll
        for (int step = 16; step >= 1; step >>= 1) {
          const int e = __shfl_sync(0xffffffffu, my_end, lo + step - 1);
          if (e <= q) lo += step;
        }
        row_end = __shfl_sync(0xffffffffu, my_end, lo);
        j = __shfl_sync(0xffffffffu, my_j0, lo) + (q - __shfl_sync(0xffffffffu, my_start, lo));
      }
      idx = 0;
      w = 1.f;
      if (q < total) {
        idx = p.indices ? __ldcs(p.indices + j) : (int32_t)j;
        if (Policy::WEIGHTED) w = __ldcs(p.weights + j);
      }
      ends = __ballot_sync(0xffffffffu, q < total && q + 1 == row_end);
    };

    float st[NS];
    pol.init(st);
    int cur = 0;  // row of the batch that st belongs to
    pol.begin_row(__shfl_sync(0xffffffffu, my_dest, 0), Policy::NEEDS_OWNER ? __shfl_sync(0xffffffffu, my_owner, 0) : 0);
    auto finish_row = [&]() {   // warp-uniform
      rw.fold(pol, st);
      const int32_t dest = __shfl_sync(0xffffffffu, my_dest, cur);
      const int32_t owner = Policy::NEEDS_OWNER ? __shfl_sync(0xffffffffu, my_owner, cur) : 0;
      const int32_t len = __shfl_sync(0xffffffffu, my_len, cur);
      if (slot == 0) pol.end_row(st, dest, owner, len);
      ++cur;
      pol.init(st);
      const int32_t nd = __shfl_sync(0xffffffffu, my_dest, cur & 31);
      const int32_t no = Policy::NEEDS_OWNER ? __shfl_sync(0xffffffffu, my_owner, cur & 31) : 0;
      if (cur < BR && __shfl_sync(0xffffffffu, my_len, cur & 31) > 0) pol.begin_row(nd, no);
    };
    ring_stream<T, SB, LPR, Policy>(rw, pol, st, total, load_chunk, finish_row);
    }
  }
}

// ----------------------------------------------------------------------------- very long rows: one CTA each
// Each warp streams its part of the row through its ring; there is no end of row inside a part.
template <typename T, int SB, int LPR, class Policy>
__global__ void __launch_bounds__(THREADS, IT_RING_MIN_BLOCKS) stream_cta_ring_kernel(StreamParams p, Policy pol) {
  constexpr int NS = Policy::NS;
  constexpr int WARPS = THREADS / 32;
  extern __shared__ uint4 ring_raw[];
  __shared__ float red[WARPS][LPR][NS];
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  RingWarp<T, SB, LPR, Policy> rw;
  rw.setup((uint32_t)__cvta_generic_to_shared(ring_raw) + (uint32_t)warp * (uint32_t)ring_bytes_per_warp<SB, Policy::HAS_EXTRA>(), p.src, p.src_pitch, lane);
  pol.setup(lane % LPR);

  for (int64_t i = p.row_lo + blockIdx.x; i < p.row_hi; i += gridDim.x) {
    const it_row_meta m = load_meta(p.meta + i);
    const int32_t owner = Policy::NEEDS_OWNER ? __ldcs(p.owner + i) : 0;
    // this warp's part of the row: edges [a, a + total)
    const int part = (m.len + WARPS - 1) / WARPS;
    const int first = warp * part < m.len ? warp * part : m.len;
    const int total = (m.len - first) < part ? (m.len - first) : part;
    const int64_t a = m.j0 + first;
    float st[NS];
    pol.init(st);
    pol.begin_row(m.dest, owner);
    auto load_chunk = [&](int base, int32_t &idx, float &w, unsigned &ends) {
      idx = 0; w = 1.f; ends = 0u;
      if (base + lane < total) {
        idx = p.indices ? __ldcs(p.indices + a + base + lane) : (int32_t)(a + base + lane);
        if (Policy::WEIGHTED) w = __ldcs(p.weights + a + base + lane);
      }
    };
    if (total > 0) ring_stream<T, SB, LPR, Policy>(rw, pol, st, total, load_chunk, [] {});
    rw.fold(pol, st);
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

}  // namespace it_stream
