// Graph ingest, validation, hub split into shadow rows, degree buckets.
// Integer-only work; every array produced here is a pure function of (indptr, threshold)
// and is built without atomics on data, so it is reproducible bit for bit.
#include <new>
#include <stdarg.h>
#include <string.h>

#include "common.cuh"

// ----------------------------------------------------------------------------- error text
static thread_local char g_err[512] = "";
void it_set_error(const char *fmt, ...) {
  va_list ap;
  va_start(ap, fmt);
  vsnprintf(g_err, sizeof(g_err), fmt, ap);
  va_end(ap);
}
extern "C" const char *it_last_error_message(void) { return g_err; }
extern "C" const char *it_status_string(it_status s) {
  switch (s) {
    case IT_OK: return "IT_OK";
    case IT_ERR_INVALID_ARG: return "IT_ERR_INVALID_ARG";
    case IT_ERR_BAD_GRAPH: return "IT_ERR_BAD_GRAPH";
    case IT_ERR_UNSUPPORTED: return "IT_ERR_UNSUPPORTED";
    case IT_ERR_WORKSPACE: return "IT_ERR_WORKSPACE";
    case IT_ERR_OOM: return "IT_ERR_OOM";
    case IT_ERR_CUDA: return "IT_ERR_CUDA";
    case IT_ERR_TIMEOUT: return "IT_ERR_TIMEOUT";
  }
  return "IT_ERR_?";
}

// ----------------------------------------------------------------------------- indptr access
struct IndptrView {
  const void *p;
  int is64;
  __device__ __forceinline__ int64_t operator[](int64_t i) const {
    return is64 ? reinterpret_cast<const int64_t *>(p)[i]
                : (int64_t) reinterpret_cast<const int32_t *>(p)[i];
  }
};

__device__ __forceinline__ int64_t groups_of(int64_t d, int64_t T) {
  return (T <= 0 || d <= T) ? 1 : (d + T - 1) / T;
}

// ----------------------------------------------------------------------------- validation
// bit 0: indptr[0] != 0, bit 1: indptr decreasing, bit 2: indptr[n] != e, bit 3: source out of range
__global__ void validate_indptr_kernel(IndptrView ip, int64_t n, int64_t e, int *flags) {
  int64_t i = blockIdx.x * (int64_t)blockDim.x + threadIdx.x;
  int bad = 0;
  if (i == 0) {
    if (ip[0] != 0) bad |= 1;
    if (ip[n] != e) bad |= 4;
  }
  if (i < n && ip[i + 1] < ip[i]) bad |= 2;
  if (bad) atomicOr(flags, bad);
}

__global__ void validate_indices_kernel(const int32_t *__restrict__ idx, int64_t e, int64_t n,
                                        int *flags) {
  int64_t stride = (int64_t)gridDim.x * blockDim.x;
  int bad = 0;
  for (int64_t i = blockIdx.x * (int64_t)blockDim.x + threadIdx.x; i < e; i += stride) {
    int32_t s = idx[i];
    if (s < 0 || (int64_t)s >= n) bad = 8;
  }
  if (bad) atomicOr(flags, bad);
}

// ----------------------------------------------------------------------------- scan-and-emit
// Exclusive prefix sum of value(i), i in [0, n), handed to emit(i, prefix) — three launches,
// no inter-block waiting.  Tile = SCAN_THREADS * SCAN_ITEMS consecutive items per block.
constexpr int SCAN_THREADS = 256;
constexpr int SCAN_ITEMS = 8;
constexpr int SCAN_TILE = SCAN_THREADS * SCAN_ITEMS;

__device__ __forceinline__ int64_t block_exclusive_scan(int64_t x, int64_t *total, int64_t *smem /*[33]*/) {
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, nwarps = blockDim.x >> 5;
  int64_t incl = x;
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    int64_t y = __shfl_up_sync(0xffffffffu, incl, o);
    if (lane >= o) incl += y;
  }
  __syncthreads();  // smem may still be read from a previous call
  if (lane == 31) smem[warp] = incl;
  __syncthreads();
  if (warp == 0) {
    int64_t w = lane < nwarps ? smem[lane] : 0;
    int64_t wi = w;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      int64_t y = __shfl_up_sync(0xffffffffu, wi, o);
      if (lane >= o) wi += y;
    }
    if (lane < nwarps) smem[lane] = wi - w;  // exclusive warp offsets
    if (lane == 31) smem[32] = wi;           // block total
  }
  __syncthreads();
  *total = smem[32];
  return smem[warp] + incl - x;
}

template <class ValueF>
__global__ void __launch_bounds__(SCAN_THREADS) scan_tile_sums_kernel(int64_t n, ValueF value, int64_t *tile_sums) {
  __shared__ int64_t smem[33];
  int64_t base = (int64_t)blockIdx.x * SCAN_TILE + (int64_t)threadIdx.x * SCAN_ITEMS;
  int64_t s = 0;
#pragma unroll
  for (int k = 0; k < SCAN_ITEMS; ++k)
    if (base + k < n) s += value(base + k);
  int64_t total;
  block_exclusive_scan(s, &total, smem);
  if (threadIdx.x == 0) tile_sums[blockIdx.x] = total;
}

// One block: exclusive scan of tile_sums in place; grand total to *total_out.
__global__ void __launch_bounds__(1024) scan_tile_offsets_kernel(int64_t n_tiles, int64_t *tile_sums, int64_t *total_out) {
  __shared__ int64_t smem[33];
  int64_t carry = 0;
  for (int64_t base = 0; base < n_tiles; base += blockDim.x) {
    int64_t i = base + threadIdx.x;
    int64_t x = i < n_tiles ? tile_sums[i] : 0;
    int64_t total;
    int64_t ex = block_exclusive_scan(x, &total, smem);
    if (i < n_tiles) tile_sums[i] = carry + ex;
    carry += total;
  }
  if (threadIdx.x == 0) *total_out = carry;
}

template <class ValueF, class EmitF>
__global__ void __launch_bounds__(SCAN_THREADS) scan_emit_kernel(int64_t n, ValueF value, EmitF emit, const int64_t *tile_offsets) {
  __shared__ int64_t smem[33];
  int64_t base = (int64_t)blockIdx.x * SCAN_TILE + (int64_t)threadIdx.x * SCAN_ITEMS;
  int64_t v[SCAN_ITEMS];
  int64_t s = 0;
#pragma unroll
  for (int k = 0; k < SCAN_ITEMS; ++k) {
    v[k] = (base + k < n) ? value(base + k) : 0;
    s += v[k];
  }
  int64_t total;
  int64_t prefix = tile_offsets[blockIdx.x] + block_exclusive_scan(s, &total, smem);
#pragma unroll
  for (int k = 0; k < SCAN_ITEMS; ++k) {
    if (base + k < n) emit(base + k, prefix);
    prefix += v[k];
  }
}

// tile_sums: device scratch of at least ceil(n / SCAN_TILE) + 1 int64; the last entry receives the total.
template <class ValueF, class EmitF>
static it_status scan_and_emit(int kid, int64_t n, ValueF value, EmitF emit, int64_t *tile_sums, int64_t *d_total, cudaStream_t st) {
  int64_t n_tiles = (n + SCAN_TILE - 1) / SCAN_TILE;
  if (n_tiles == 0) {
    IT_CUDA_TRY(cudaMemsetAsync(d_total, 0, sizeof(int64_t), st));
    return IT_OK;
  }
  IT_LAUNCH(kid, 0, 0, st, scan_tile_sums_kernel<<<(unsigned)n_tiles, SCAN_THREADS, 0, st>>>(n, value, tile_sums));
  IT_LAUNCH(kid, 0, 0, st, scan_tile_offsets_kernel<<<1, 1024, 0, st>>>(n_tiles, tile_sums, d_total));
  IT_LAUNCH(kid, 0, 0, st, scan_emit_kernel<<<(unsigned)n_tiles, SCAN_THREADS, 0, st>>>(n, value, emit, tile_sums));
  IT_CUDA_TRY(cudaGetLastError());
  return IT_OK;
}

// ----------------------------------------------------------------------------- split functors
struct RowsOfVertex {
  IndptrView ip; int64_t T;
  __device__ int64_t operator()(int64_t v) const { return groups_of(ip[v + 1] - ip[v], T); }
};
struct EmitOwnerIndptr {
  int64_t *owner_indptr; int64_t n;
  __device__ void operator()(int64_t v, int64_t prefix) const { owner_indptr[v] = prefix; }
};
struct IsSplit {
  IndptrView ip; int64_t T;
  __device__ int64_t operator()(int64_t v) const { return groups_of(ip[v + 1] - ip[v], T) > 1 ? 1 : 0; }
};
struct EmitSplitOwner {
  IndptrView ip; int64_t T; int32_t *split_owners;
  __device__ void operator()(int64_t v, int64_t k) const {
    if (groups_of(ip[v + 1] - ip[v], T) > 1) split_owners[k] = (int32_t)v;
  }
};
// count pass only (the list is not allocated yet)
struct EmitNothing {
  __device__ void operator()(int64_t, int64_t) const {}
};

// Rows of unsplit vertices: one thread per vertex.
__global__ void fill_unsplit_rows_kernel(IndptrView ip, int64_t n, int64_t T, const int64_t *__restrict__ owner_indptr,
                                         int64_t *shadow_indptr, int32_t *shadow_owner, int32_t *row_dest,
                                         int64_t n_rows, int64_t e) {
  int64_t v = blockIdx.x * (int64_t)blockDim.x + threadIdx.x;
  if (v == 0) shadow_indptr[n_rows] = e;
  if (v >= n) return;
  int64_t d = ip[v + 1] - ip[v];
  if (groups_of(d, T) > 1) return;
  int64_t r = owner_indptr[v];
  shadow_indptr[r] = ip[v];
  shadow_owner[r] = (int32_t)v;
  row_dest[r] = (int32_t)v;
}

// Rows of split vertices: one block per split owner, groups written by closed form
//   start(g) = indptr[v] + g * base + min(g, rem),  base = d / n, rem = d % n.
__global__ void fill_split_rows_kernel(IndptrView ip, int64_t T, const int32_t *__restrict__ split_owners,
                                       const int64_t *__restrict__ owner_indptr, int64_t *shadow_indptr,
                                       int32_t *shadow_owner, int32_t *row_dest) {
  int64_t k = blockIdx.x;
  int64_t v = split_owners[k];
  int64_t d = ip[v + 1] - ip[v];
  int64_t ng = groups_of(d, T);
  int64_t base = d / ng, rem = d % ng;
  int64_t r0 = owner_indptr[v];
  int64_t p0 = r0 - v + k;  // rows of earlier split owners = all earlier rows minus earlier unsplit vertices
  for (int64_t g = threadIdx.x; g < ng; g += blockDim.x) {
    shadow_indptr[r0 + g] = ip[v] + g * base + (g < rem ? g : rem);
    shadow_owner[r0 + g] = (int32_t)v;
    row_dest[r0 + g] = (int32_t)~(p0 + g);
  }
}

// ----------------------------------------------------------------------------- bucket functors
struct Bounds { int64_t b[IT_MAX_BUCKETS]; int nb; };
__device__ __forceinline__ int bucket_of(int64_t len, const Bounds &B) {
  int k = 0;
  while (k < B.nb - 1 && len > B.b[k]) ++k;
  return k;
}
struct InBucket {
  const int64_t *sp; Bounds B; int which;
  __device__ int64_t operator()(int64_t r) const { return bucket_of(sp[r + 1] - sp[r], B) == which ? 1 : 0; }
};
struct EmitBucketRow {
  const int64_t *sp; Bounds B; int which; int32_t *bucket_rows; const int64_t *bucket_offsets;
  __device__ void operator()(int64_t r, int64_t pos) const {
    if (bucket_of(sp[r + 1] - sp[r], B) == which) bucket_rows[bucket_offsets[which] + pos] = (int32_t)r;
  }
};
struct EdgesInBucket {
  const int64_t *sp; Bounds B; int which;
  __device__ int64_t operator()(int64_t r) const {
    const int64_t len = sp[r + 1] - sp[r];
    return bucket_of(len, B) == which ? len : 0;
  }
};
__global__ void fill_bucket_meta_kernel(int64_t n_rows, const int32_t *__restrict__ bucket_rows,
                                       const int64_t *__restrict__ sp, const int32_t *__restrict__ row_dest,
                                       const int32_t *__restrict__ shadow_owner, it_row_meta *__restrict__ meta,
                                       int32_t *__restrict__ bucket_owner) {
  int64_t i = blockIdx.x * (int64_t)blockDim.x + threadIdx.x;
  if (i >= n_rows) return;
  const int32_t r = bucket_rows[i];
  it_row_meta m;
  m.j0 = sp[r];
  m.len = (int32_t)(sp[r + 1] - sp[r]);
  m.dest = row_dest[r];
  meta[i] = m;
  bucket_owner[i] = shadow_owner[r];
}
__global__ void set_next_bucket_offset_kernel(int64_t *bucket_offsets, int which, const int64_t *count) {
  if (which == 0) bucket_offsets[0] = 0;
  bucket_offsets[which + 1] = bucket_offsets[which] + *count;
}

// ----------------------------------------------------------------------------- host side
static void free_derived(it_graph *g) {
  cudaFree(g->shadow_indptr); cudaFree(g->shadow_owner); cudaFree(g->owner_indptr);
  cudaFree(g->row_dest); cudaFree(g->split_owners); cudaFree(g->bucket_offsets); cudaFree(g->bucket_rows);
  cudaFree(g->bucket_meta); g->bucket_meta = nullptr;
  cudaFree(g->bucket_owner); g->bucket_owner = nullptr;
  g->shadow_indptr = nullptr; g->shadow_owner = nullptr; g->owner_indptr = nullptr; g->row_dest = nullptr;
  g->split_owners = nullptr; g->bucket_offsets = nullptr; g->bucket_rows = nullptr;
  g->n_rows = g->n_split_owners = g->n_partial_rows = 0;
  g->n_buckets = 0;
}

static it_status split_impl(it_graph *g, int64_t T, cudaStream_t st) {
  free_derived(g);
  g->threshold = T > 0 ? T : 0;
  const int64_t n = g->n;
  IndptrView ip{g->indptr, g->indptr_type == IT_I64};

  int64_t *d_scratch = nullptr;  // tile sums (+ totals at the end)
  int64_t max_items = n;         // rows are scanned later; R is not known yet, scratch is re-sized then
  int64_t n_tiles = (max_items + SCAN_TILE - 1) / SCAN_TILE;
  IT_CUDA_TRY(cudaMalloc(&d_scratch, (size_t)(n_tiles + 4) * sizeof(int64_t)));
  int64_t *d_total = d_scratch + n_tiles;  // [0] rows, [1] split owners
  it_status rc = IT_OK;
  int64_t h_tot[2] = {0, 0};
  auto fail = [&](it_status s) { cudaFree(d_scratch); free_derived(g); return s; };
#define SPLIT_TRY(expr) do { rc = (expr); if (rc != IT_OK) return fail(rc); } while (0)
#define SPLIT_CUDA(expr) do { cudaError_t _e = (expr); if (_e != cudaSuccess) { \
    it_set_error("%s failed: %s", #expr, cudaGetErrorString(_e)); \
    return fail(_e == cudaErrorMemoryAllocation ? IT_ERR_OOM : IT_ERR_CUDA); } } while (0)

  SPLIT_CUDA(cudaMalloc(&g->owner_indptr, (size_t)(n + 1) * sizeof(int64_t)));
  SPLIT_TRY(scan_and_emit(IT_K_SPLIT_SCAN, n, RowsOfVertex{ip, T}, EmitOwnerIndptr{g->owner_indptr, n}, d_scratch, d_total, st));
  SPLIT_CUDA(cudaMemcpyAsync(g->owner_indptr + n, d_total, sizeof(int64_t), cudaMemcpyDeviceToDevice, st));
  SPLIT_TRY(scan_and_emit(IT_K_SPLIT_SCAN, n, IsSplit{ip, T}, EmitNothing{}, d_scratch, d_total + 1, st));
  SPLIT_CUDA(cudaMemcpyAsync(h_tot, d_total, 2 * sizeof(int64_t), cudaMemcpyDeviceToHost, st));
  SPLIT_CUDA(cudaStreamSynchronize(st));
  const int64_t R = n > 0 ? h_tot[0] : 0;
  const int64_t S = n > 0 ? h_tot[1] : 0;
  if (R > (int64_t)INT32_MAX - 1) {
    it_set_error("split produces %lld shadow rows; row ids are 32-bit", (long long)R);
    return fail(IT_ERR_UNSUPPORTED);
  }
  g->n_rows = R;
  g->n_split_owners = S;
  g->n_partial_rows = R - (n - S);

  SPLIT_CUDA(cudaMalloc(&g->shadow_indptr, (size_t)(R + 1) * sizeof(int64_t)));
  SPLIT_CUDA(cudaMalloc(&g->shadow_owner, (size_t)(R > 0 ? R : 1) * sizeof(int32_t)));
  SPLIT_CUDA(cudaMalloc(&g->row_dest, (size_t)(R > 0 ? R : 1) * sizeof(int32_t)));
  SPLIT_CUDA(cudaMalloc(&g->split_owners, (size_t)(S > 0 ? S : 1) * sizeof(int32_t)));
  SPLIT_CUDA(cudaMalloc(&g->bucket_rows, (size_t)(R > 0 ? R : 1) * sizeof(int32_t)));
  SPLIT_CUDA(cudaMalloc(&g->bucket_meta, (size_t)(R > 0 ? R : 1) * sizeof(it_row_meta)));
  SPLIT_CUDA(cudaMalloc(&g->bucket_owner, (size_t)(R > 0 ? R : 1) * sizeof(int32_t)));
  SPLIT_CUDA(cudaMalloc(&g->bucket_offsets, (IT_MAX_BUCKETS + 1) * sizeof(int64_t)));
  if (S > 0)
    SPLIT_TRY(scan_and_emit(IT_K_SPLIT_SCAN, n, IsSplit{ip, T}, EmitSplitOwner{ip, T, g->split_owners}, d_scratch, d_total + 1, st));
  {
    unsigned blocks = (unsigned)((n + 255) / 256);
    if (blocks == 0) blocks = 1;
    IT_LAUNCH(IT_K_SPLIT_FILL, 0, 0, st,
              fill_unsplit_rows_kernel<<<blocks, 256, 0, st>>>(ip, n, T, g->owner_indptr, g->shadow_indptr,
                                                               g->shadow_owner, g->row_dest, R, g->e));
    if (S > 0)
      IT_LAUNCH(IT_K_SPLIT_FILL, 0, 0, st,
                fill_split_rows_kernel<<<(unsigned)S, 128, 0, st>>>(ip, T, g->split_owners, g->owner_indptr,
                                                                    g->shadow_indptr, g->shadow_owner, g->row_dest));
    SPLIT_CUDA(cudaGetLastError());
  }

  // degree buckets: {0, 8, 32, 256, 1024, everything longer}
  Bounds B;
  const int64_t fixed[5] = {0, 8, 32, 256, 1024};
  B.nb = 0;
  for (int i = 0; i < 5; ++i)
    if (T <= 0 || fixed[i] < T) B.b[B.nb++] = fixed[i];
  B.b[B.nb++] = T > 0 ? T : INT64_MAX;
  g->n_buckets = B.nb;
  for (int i = 0; i < IT_MAX_BUCKETS; ++i) g->bucket_bounds[i] = i < B.nb ? B.b[i] : 0;

  // the row scans need ceil(R / tile) sums; R >= n, so regrow the scratch
  cudaFree(d_scratch);
  d_scratch = nullptr;
  n_tiles = (R + SCAN_TILE - 1) / SCAN_TILE;
  SPLIT_CUDA(cudaMalloc(&d_scratch, (size_t)(n_tiles + 4 + IT_MAX_BUCKETS) * sizeof(int64_t)));
  d_total = d_scratch + n_tiles;
  int64_t *d_edges = d_total + 4;
  for (int b = 0; b < B.nb; ++b) {
    if (b == 0) {
      // offsets[0] must exist before the first emit reads it
      SPLIT_CUDA(cudaMemsetAsync(g->bucket_offsets, 0, sizeof(int64_t), st));
    }
    SPLIT_TRY(scan_and_emit(IT_K_BUCKET_SCAN, R, InBucket{g->shadow_indptr, B, b},
                            EmitBucketRow{g->shadow_indptr, B, b, g->bucket_rows, g->bucket_offsets}, d_scratch,
                            d_total, st));
    IT_LAUNCH(IT_K_BUCKET_SCAN, 0, 0, st, set_next_bucket_offset_kernel<<<1, 1, 0, st>>>(g->bucket_offsets, b, d_total));
    SPLIT_TRY(scan_and_emit(IT_K_BUCKET_SCAN, R, EdgesInBucket{g->shadow_indptr, B, b}, EmitNothing{}, d_scratch,
                            d_edges + b, st));
  }
  if (R > 0)
    IT_LAUNCH(IT_K_BUCKET_SCAN, 0, 0, st,
              fill_bucket_meta_kernel<<<(unsigned)((R + 255) / 256), 256, 0, st>>>(R, g->bucket_rows, g->shadow_indptr,
                                                                                    g->row_dest, g->shadow_owner, g->bucket_meta, g->bucket_owner));
  SPLIT_CUDA(cudaGetLastError());
  SPLIT_CUDA(cudaMemcpyAsync(g->h_bucket_edges, d_edges, B.nb * sizeof(int64_t), cudaMemcpyDeviceToHost, st));
  SPLIT_CUDA(cudaMemcpyAsync(g->h_bucket_offsets, g->bucket_offsets, (B.nb + 1) * sizeof(int64_t),
                             cudaMemcpyDeviceToHost, st));
  SPLIT_CUDA(cudaStreamSynchronize(st));
  cudaFree(d_scratch);
#undef SPLIT_TRY
#undef SPLIT_CUDA
  return IT_OK;
}

extern "C" it_status it_graph_set_edge_features(it_graph *g, const void *edge_feat, int32_t edge_dim, it_dtype dtype) {
  IT_REQUIRE(g != nullptr, IT_ERR_INVALID_ARG, "graph is NULL");
  if (edge_feat == nullptr || edge_dim == 0) {
    IT_REQUIRE(edge_feat == nullptr && edge_dim == 0, IT_ERR_INVALID_ARG, "edge features need both a pointer and a dimension");
    g->edge_feat = nullptr; g->edge_dim = 0;
    return IT_OK;
  }
  IT_REQUIRE(dtype == IT_F32 || dtype == IT_BF16, IT_ERR_INVALID_ARG, "bad edge feature dtype");
  const int64_t row = (int64_t)edge_dim * it_dtype_size(dtype);
  IT_REQUIRE(edge_dim > 0 && row % 16 == 0, IT_ERR_INVALID_ARG, "an edge-feature row must be a multiple of 16 bytes (got %lld)", (long long)row);
  IT_REQUIRE(((uintptr_t)edge_feat % 16) == 0, IT_ERR_INVALID_ARG, "edge features must be 16-byte aligned");
  g->edge_feat = edge_feat; g->edge_dim = edge_dim; g->edge_dtype = dtype;
  return IT_OK;
}

static it_status create_impl(int64_t n, int64_t n_src, int64_t e, const void *indptr, it_itype indptr_type,
                             const int32_t *indices, const float *edge_weights, void *stream, it_graph **out) {
  IT_REQUIRE(out != nullptr, IT_ERR_INVALID_ARG, "out is NULL");
  *out = nullptr;
  IT_REQUIRE(n >= 0 && n <= (int64_t)INT32_MAX - 1, IT_ERR_INVALID_ARG, "n_vertices %lld outside [0, 2^31-2]", (long long)n);
  IT_REQUIRE(n_src >= 0 && n_src <= (int64_t)INT32_MAX - 1, IT_ERR_INVALID_ARG, "n_sources %lld outside [0, 2^31-2]", (long long)n_src);
  IT_REQUIRE(e == 0 || n_src > 0, IT_ERR_INVALID_ARG, "edges need at least one source vertex");
  IT_REQUIRE(e >= 0, IT_ERR_INVALID_ARG, "n_edges is negative");
  IT_REQUIRE(indptr != nullptr, IT_ERR_INVALID_ARG, "indptr is NULL");
  IT_REQUIRE(indices != nullptr || e == 0, IT_ERR_INVALID_ARG, "indices is NULL");
  IT_REQUIRE(indptr_type == IT_I32 || indptr_type == IT_I64, IT_ERR_INVALID_ARG, "bad indptr_type");
  IT_REQUIRE(indptr_type == IT_I64 || e <= (int64_t)INT32_MAX, IT_ERR_INVALID_ARG, "int32 indptr cannot index %lld edges", (long long)e);
  cudaStream_t st = (cudaStream_t)stream;

  int *d_flags = nullptr;
  IT_CUDA_TRY(cudaMalloc(&d_flags, sizeof(int)));
  IndptrView ip{indptr, indptr_type == IT_I64};
  cudaError_t ce = cudaMemsetAsync(d_flags, 0, sizeof(int), st);
  int h_flags = 0;
  if (ce == cudaSuccess) {
    IT_LAUNCH(IT_K_VALIDATE, 0, 0, st, validate_indptr_kernel<<<(unsigned)((n + 1 + 255) / 256), 256, 0, st>>>(ip, n, e, d_flags));
    ce = cudaMemcpyAsync(&h_flags, d_flags, sizeof(int), cudaMemcpyDeviceToHost, st);
  }
  if (ce == cudaSuccess) ce = cudaStreamSynchronize(st);
  // the source ids are only scanned once the indptr is known to be sane
  if (ce == cudaSuccess && h_flags == 0 && e > 0) {
    int64_t want = (e + 255) / 256;
    unsigned blocks = (unsigned)(want < 148 * 16 ? want : 148 * 16);
    IT_LAUNCH(IT_K_VALIDATE, 0, 0, st, validate_indices_kernel<<<blocks, 256, 0, st>>>(indices, e, n_src, d_flags));
    ce = cudaMemcpyAsync(&h_flags, d_flags, sizeof(int), cudaMemcpyDeviceToHost, st);
    if (ce == cudaSuccess) ce = cudaStreamSynchronize(st);
  }
  cudaFree(d_flags);
  if (ce != cudaSuccess) {
    it_set_error("graph validation failed to run: %s", cudaGetErrorString(ce));
    return IT_ERR_CUDA;
  }
  if (h_flags != 0) {
    it_set_error("bad CSR:%s%s%s%s", (h_flags & 1) ? " indptr[0] != 0;" : "", (h_flags & 2) ? " indptr decreases;" : "",
                 (h_flags & 4) ? " indptr[n] != n_edges;" : "", (h_flags & 8) ? " a source id is outside [0, n_sources);" : "");
    return IT_ERR_BAD_GRAPH;
  }

  it_graph *g = new (std::nothrow) it_graph();
  IT_REQUIRE(g != nullptr, IT_ERR_OOM, "host allocation failed");
  g->n = n; g->n_src = n_src; g->e = e; g->indptr = indptr; g->indptr_type = indptr_type;
  g->indices = indices; g->edge_weights = edge_weights;
  cudaGetDevice(&g->device);
  int sms = 0;
  if (cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, g->device) == cudaSuccess && sms > 0) g->num_sms = sms;
  if (cudaMalloc(&g->d_status, sizeof(int)) != cudaSuccess || cudaMemsetAsync(g->d_status, 0, sizeof(int), st) != cudaSuccess) {
    it_set_error("allocating the status word failed");
    cudaFree(g->d_status);
    delete g;
    return IT_ERR_OOM;
  }
  it_status rc = split_impl(g, 0, st);
  if (rc != IT_OK) { cudaFree(g->d_status); delete g; return rc; }
  *out = g;
  return IT_OK;
}

extern "C" it_status it_graph_create(int64_t n, int64_t e, const void *indptr, it_itype indptr_type,
                                     const int32_t *indices, const float *edge_weights, void *stream,
                                     it_graph **out) {
  return create_impl(n, n, e, indptr, indptr_type, indices, edge_weights, stream, out);
}

extern "C" it_status it_graph_create_part(int64_t n, int64_t n_sources, int64_t e, const void *indptr, it_itype indptr_type,
                                          const int32_t *indices, const float *edge_weights, void *stream,
                                          it_graph **out) {
  return create_impl(n, n_sources, e, indptr, indptr_type, indices, edge_weights, stream, out);
}

extern "C" it_status it_split_hubs(it_graph *g, int64_t threshold, void *stream, int64_t *out_n_rows,
                                   int64_t *out_n_split_owners) {
  IT_REQUIRE(g != nullptr, IT_ERR_INVALID_ARG, "graph is NULL");
  IT_TRY(split_impl(g, threshold, (cudaStream_t)stream));
  if (out_n_rows) *out_n_rows = g->n_rows;
  if (out_n_split_owners) *out_n_split_owners = g->n_split_owners;
  return IT_OK;
}

extern "C" it_status it_graph_get_split(const it_graph *g, int64_t *n_rows, const int64_t **shadow_indptr,
                                        const int32_t **shadow_owner, const int64_t **owner_indptr,
                                        const int64_t **bucket_offsets, const int32_t **bucket_rows,
                                        int32_t *n_buckets, int64_t *bucket_bounds) {
  IT_REQUIRE(g != nullptr, IT_ERR_INVALID_ARG, "graph is NULL");
  if (n_rows) *n_rows = g->n_rows;
  if (shadow_indptr) *shadow_indptr = g->shadow_indptr;
  if (shadow_owner) *shadow_owner = g->shadow_owner;
  if (owner_indptr) *owner_indptr = g->owner_indptr;
  if (bucket_offsets) *bucket_offsets = g->bucket_offsets;
  if (bucket_rows) *bucket_rows = g->bucket_rows;
  if (n_buckets) *n_buckets = g->n_buckets;
  if (bucket_bounds) memcpy(bucket_bounds, g->bucket_bounds, sizeof(g->bucket_bounds));
  return IT_OK;
}

extern "C" it_status it_graph_check(it_graph *g, void *stream) {
  IT_REQUIRE(g != nullptr, IT_ERR_INVALID_ARG, "graph is NULL");
  cudaStream_t st = (cudaStream_t)stream;
  int h = 0;
  IT_CUDA_TRY(cudaMemcpyAsync(&h, g->d_status, sizeof(int), cudaMemcpyDeviceToHost, st));
  IT_CUDA_TRY(cudaStreamSynchronize(st));
  if (h != 0) {
    IT_CUDA_TRY(cudaMemsetAsync(g->d_status, 0, sizeof(int), st));
    it_set_error("a kernel gave up a bounded wait; its outputs are not valid");
    return IT_ERR_TIMEOUT;
  }
  return IT_OK;
}

extern "C" it_status it_graph_destroy(it_graph *g) {
  if (!g) return IT_OK;
  free_derived(g);
  cudaFree(g->d_status);
  delete g;
  return IT_OK;
}
