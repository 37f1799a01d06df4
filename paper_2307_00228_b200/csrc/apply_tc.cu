// Apply on the 5th-generation tensor cores: a persistent, warp-specialised GEMM
//   C[M, NB] = X1[M, K1] * B[0:K1, :] + X2[M, K2] * B[K1:, :]
// with tcgen05.mma (accumulators in TMEM), operands staged in shared memory by TMA
// (128-byte swizzle), the small weight matrix resident in shared memory for the life of the
// CTA, two TMEM accumulator buffers so that the epilogue of one 128-row tile overlaps the
// main loop of the next, and bias / activation / dtype routing / GAT scores in the epilogue.
//
// Two operand modes:
//   bf16 : kind::f16 with bf16 inputs, fp32 accumulation.
//   fp32 : three kind::tf32 products per step, A = A_hi + A_lo and B = B_hi + B_lo with
//          A_hi*B_hi + A_lo*B_hi + A_hi*B_lo (the dropped A_lo*B_lo term is ~2^-22 relative);
//          a single TF32 pass (10-bit mantissa) would miss the 1e-4 error bound.  Four dedicated
//          warps read each raw A tile from shared memory once, split it and write both parts to
//          TMEM (tcgen05.st), so that the MMAs take A from TMEM and read only the weights from
//          shared memory; B is split once by the prep kernel.
//
// Every wait on an mbarrier is bounded: when one gives up, the CTA raises a flag that all
// roles poll, drains, frees its TMEM and returns, and a status word in global memory is set.
#include <cuda.h>

#include "common.cuh"

// fp32 mode: A_hi = x with the low 13 mantissa bits cleared (what the tensor core keeps of a tf32 operand),
// A_lo = x - A_hi, exact in fp32.  (Were the hi part rounded instead while the lo part assumed truncation,
// half of the products would be off by 2^-11 relative, ten times the fp32 parity tolerance.)

namespace {

constexpr int TC_BM = 128;          // rows per tile (UMMA M)
constexpr int TC_KBLOCK_BYTES = 128;  // one swizzle row of K per k-block
constexpr int TC_EPI_WARPS = 16;      // four warps per TMEM lane quarter, each takes every fourth 16-column group
constexpr int TC_THREADS_BF16 = 64 + 32 * TC_EPI_WARPS;   // warp 0 TMA, warp 1 MMA + TMEM, warps 2-17 epilogue
#ifndef IT_TC_EPI_BACKOFF
#define IT_TC_EPI_BACKOFF 128   // ns the epilogue warps sleep between polls of the accumulator barrier
#endif
#ifndef IT_TC_TMA_BACKOFF
#define IT_TC_TMA_BACKOFF 64    // ns the TMA producer sleeps between polls of a stage's empty barrier
#endif
#ifndef IT_TC_EPI_GROUPS
#define IT_TC_EPI_GROUPS 2   // staged epilogue: groups of epilogue warps that take alternate tiles (1 or 2)
#endif
#ifndef IT_TC_TMA_STORE
#define IT_TC_TMA_STORE 1   // 0: always store the results straight from registers
#endif
#ifndef IT_TC_MAX_STAGES
#define IT_TC_MAX_STAGES 8   // operand stages in shared memory (as many as fit, up to this)
#endif
#ifndef IT_TC_SPLIT_GROUPS
#define IT_TC_SPLIT_GROUPS 1   // groups of four split warps; group g takes every k-block c with c % groups == g (measured: a second group gains nothing)
#endif
constexpr int TC_SPLIT_GROUPS = IT_TC_SPLIT_GROUPS;
constexpr int TC_THREADS_TF32 = TC_THREADS_BF16 + 128 * TC_SPLIT_GROUPS;   // ... plus the warps splitting A into hi / lo
#ifndef IT_TC_TSTAGES_MAX
#define IT_TC_TSTAGES_MAX 4
#endif
constexpr int TC_TSTAGES_MAX = IT_TC_TSTAGES_MAX;     // fp32 mode: split A tiles in flight in TMEM
constexpr int TC_TSTAGE_COLS = 64;    // TMEM columns of one split A k-block: 32 of hi, 32 of lo
constexpr uint32_t TC_SPIN_LIMIT = 1u << 22;

// ----------------------------------------------------------------------------- PTX wrappers
__device__ __forceinline__ uint32_t smem_u32(const void *p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint64_t *bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(bar)), "r"(count));
}
__device__ __forceinline__ void mbar_arrive(uint64_t *bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_u32(bar)) : "memory");
}
__device__ __forceinline__ void mbar_arrive_expect_tx(uint64_t *bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_u32(bar)), "r"(bytes) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint64_t *bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(ok)
      : "r"(smem_u32(bar)), "r"(parity)
      : "memory");
  return ok != 0;
}
// Bounded wait.  Returns false if the CTA is aborting (or this wait ran out and started the abort).
// `backoff_ns` > 0: sleep between polls, for roles whose waits are long and off the critical path (their polling
// would otherwise take issue slots from the warps that feed the tensor core).
// `limit`: the number of polls after which the wait gives up.
__device__ __forceinline__ bool mbar_wait(uint64_t *bar, uint32_t parity, volatile int *abort_flag, uint32_t limit, uint32_t backoff_ns = 0) {
  for (uint32_t it = 0; it < limit; ++it) {
    if (mbar_try_wait(bar, parity)) return true;
    if (backoff_ns) __nanosleep(backoff_ns);
    if ((it & 63u) == 63u && *abort_flag) return false;
  }
  *abort_flag = 1;
  return false;
}
__device__ __forceinline__ void tma_load_2d(void *dst, const CUtensorMap *map, int c0, int c1, uint64_t *bar) {
  asm volatile(
      "cp.async.bulk.tensor.2d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4}], [%2];"
      ::"r"(smem_u32(dst)), "l"(map), "r"(smem_u32(bar)), "r"(c0), "r"(c1)
      : "memory");
}
// TMA store of one 128-byte-swizzled panel [128 rows x 128 bytes] from shared memory; rows past the end of the
// tensor are clipped by the copy engine.
__device__ __forceinline__ void tma_store_2d(const CUtensorMap *map, const void *src, int c0, int c1) {
  asm volatile("cp.async.bulk.tensor.2d.global.shared::cta.tile.bulk_group [%0, {%2, %3}], [%1];"
               ::"l"(map), "r"(smem_u32(src)), "r"(c0), "r"(c1)
               : "memory");
}
__device__ __forceinline__ void tma_store_commit() { asm volatile("cp.async.bulk.commit_group;" ::: "memory"); }
__device__ __forceinline__ void tma_store_wait_read() { asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory"); }
__device__ __forceinline__ void tma_store_wait_all() { asm volatile("cp.async.bulk.wait_group 0;" ::: "memory"); }
// Named barriers of the epilogue warps (immediate operands): barrier 1 over all sixteen warps, or barriers 1 and 2
// over the eight warps of a group.  The reducing form also tells every thread whether any of them failed.
__device__ __forceinline__ void epi_bar_sync(int groups, int group) {
  if (groups == 1) asm volatile("bar.sync 1, %0;" ::"n"(32 * TC_EPI_WARPS) : "memory");
  else if (group == 0) asm volatile("bar.sync 1, %0;" ::"n"(16 * TC_EPI_WARPS) : "memory");
  else asm volatile("bar.sync 2, %0;" ::"n"(16 * TC_EPI_WARPS) : "memory");
}
#define IT_EPI_BAR_RED(ID, N)                                                        \
  asm volatile("{\n\t.reg .pred p, q;\n\tsetp.ne.u32 p, %1, 0;\n\t"                 \
               "bar.red.or.pred q, " #ID ", %2, p;\n\t"                              \
               "selp.u32 %0, 1, 0, q;\n\t}"                                          \
               : "=r"(r)                                                             \
               : "r"((uint32_t)flag), "n"(N)                                         \
               : "memory")
__device__ __forceinline__ bool epi_bar_any(int groups, int group, bool flag) {
  uint32_t r;
  if (groups == 1) IT_EPI_BAR_RED(1, 32 * TC_EPI_WARPS);
  else if (group == 0) IT_EPI_BAR_RED(1, 16 * TC_EPI_WARPS);
  else IT_EPI_BAR_RED(2, 16 * TC_EPI_WARPS);
  return r != 0;
}
__device__ __forceinline__ void st_shared_v4(uint32_t addr, uint32_t a, uint32_t b, uint32_t c, uint32_t d) {
  asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(addr), "r"(a), "r"(b), "r"(c), "r"(d) : "memory");
}
__device__ __forceinline__ void tmem_alloc(uint32_t *dst_smem, uint32_t ncols) {
  asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(dst_smem)), "r"(ncols));
}
__device__ __forceinline__ void tmem_relinquish() {
  asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::);
}
__device__ __forceinline__ void tmem_dealloc(uint32_t taddr, uint32_t ncols) {
  asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(taddr), "r"(ncols));
}
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_commit(uint64_t *bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(smem_u32(bar)) : "memory");
}
template <bool TF32>
__device__ __forceinline__ void tc_mma(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc, uint32_t accumulate) {
  if (TF32) {
    asm volatile(
        "{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::tf32 [%0], %1, %2, %3, {%5, %5, %5, %5}, p;\n\t}"
        ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate), "r"(0u)
        : "memory");
  } else {
    asm volatile(
        "{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, {%5, %5, %5, %5}, p;\n\t}"
        ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate), "r"(0u)
        : "memory");
  }
}
// The same product with the A operand in tensor memory (lane = row of the tile, one 32-bit column per tf32 element).
__device__ __forceinline__ void tc_mma_tf32_tmem_a(uint32_t d_tmem, uint32_t a_tmem, uint64_t b_desc, uint32_t idesc, uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::tf32 [%0], [%1], %2, %3, {%5, %5, %5, %5}, p;\n\t}"
      ::"r"(d_tmem), "r"(a_tmem), "l"(b_desc), "r"(idesc), "r"(accumulate), "r"(0u)
      : "memory");
}
// Lane i of the warp writes 16 consecutive 32-bit columns of TMEM lane (lane base of taddr) + i.
__device__ __forceinline__ void tmem_st16(uint32_t taddr, const uint32_t (&r)[16]) {
  asm volatile(
      "tcgen05.st.sync.aligned.32x32b.x16.b32 [%0], {%1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, %16};"
      ::"r"(taddr), "r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]), "r"(r[7]), "r"(r[8]),
        "r"(r[9]), "r"(r[10]), "r"(r[11]), "r"(r[12]), "r"(r[13]), "r"(r[14]), "r"(r[15])
      : "memory");
}
__device__ __forceinline__ void tmem_st_wait() { asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory"); }
__device__ __forceinline__ void tmem_ld16(uint32_t taddr, uint32_t (&r)[16]) {
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x16.b32 {%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15}, [%16];"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]),
        "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15])
      : "r"(taddr));
}
__device__ __forceinline__ void tmem_ld_wait() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }

// Shared-memory matrix descriptor of a K-major tile whose rows are 128-byte swizzle rows:
// start address, leading offset 16 B (unused for swizzled K-major), 1024 B between 8-row
// groups, descriptor version 1, layout SWIZZLE_128B.
__device__ __forceinline__ uint64_t make_desc(uint32_t smem_addr) {
  return (uint64_t)((smem_addr & 0x3FFFFu) >> 4) | ((uint64_t)1 << 16) | ((uint64_t)(1024 >> 4) << 32) | ((uint64_t)1 << 46) |
         ((uint64_t)2 << 61);
}

// ----------------------------------------------------------------------------- kernel
struct TcParams {
  int64_t M;
  int n_tiles_m, n_splits, nbc;   // row tiles, column splits, columns per CTA
  int kb1, kb2;                   // k-blocks that come from X1 / X2
  int NB;                         // total columns
  int stages;
  int tstages;                    // fp32 mode: split A k-blocks in flight in TMEM
  // epilogue routing (columns are global column ids)
  int n0; void *out0; int out0_bf16; const float *bias0; int act0;
  int n1; void *out1; int out1_bf16;
  float *scores; const float *att_src; const float *att_dst; int heads, head_dim;  // GAT: scores [M, 2*heads]
  int *status;                    // set to 1 if a bounded wait gave up
  int tma_store;                  // 1: the epilogue stages each output tile in shared memory and writes it with TMA stores
  int out_panels;                 // 16 KB panels of one staging tile (128 rows x 128 bytes each)
  int epi_groups;                 // staged epilogue: 1, or 2 groups of eight warps that take alternate tiles (one staging tile each)
  uint32_t spin_limit;            // polls after which a wait on a barrier gives up
  int no_loads;                   // test hook: the producer issues no copies, so every wait runs out
};

template <bool TF32>
__global__ void __launch_bounds__(TF32 ? TC_THREADS_TF32 : TC_THREADS_BF16, 1)
gemm_tc_kernel(const __grid_constant__ CUtensorMap map_x1, const __grid_constant__ CUtensorMap map_x2,
               const __grid_constant__ CUtensorMap map_b, const __grid_constant__ CUtensorMap map_o0,
               const __grid_constant__ CUtensorMap map_o1, const TcParams p) {
  extern __shared__ unsigned char smem_raw[];
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int KB = p.kb1 + p.kb2;
  const int b_tile_bytes = p.nbc * TC_KBLOCK_BYTES;              // one k-block of B (one part)
  const int b_bytes = (TF32 ? 2 : 1) * KB * b_tile_bytes;
  constexpr int a_tile_bytes = TC_BM * TC_KBLOCK_BYTES;          // 16 KB

  // shared memory: resident weights | operand stages (bf16 tiles the MMAs read, or raw fp32 tiles the split warps read) |
  // output staging panels | barriers
  unsigned char *base = reinterpret_cast<unsigned char *>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
  unsigned char *smem_b = base;
  unsigned char *smem_a = base + b_bytes;   // b_bytes is a multiple of 1024 (nbc is a multiple of 16)
  unsigned char *smem_out = smem_a + (size_t)p.stages * a_tile_bytes;   // output staging panels (TMA-store epilogue), 1024-byte aligned
  uint64_t *bars = reinterpret_cast<uint64_t *>(smem_out + (size_t)p.out_panels * p.epi_groups * a_tile_bytes);
  uint64_t *full = bars;                    // [stages]  TMA landed
  uint64_t *empty = bars + p.stages;        // [stages]  the stage's readers are done (bf16: its MMAs; fp32: the split warps)
  uint64_t *ready = bars + 2 * p.stages;    // [TC_TSTAGES_MAX]  (fp32 mode) hi / lo parts written to TMEM
  uint64_t *a_free = ready + TC_TSTAGES_MAX;   // [TC_TSTAGES_MAX]  (fp32 mode) MMAs that read a TMEM stage are done
  uint64_t *b_full = a_free + TC_TSTAGES_MAX;  // [1]
  uint64_t *acc_full = b_full + 1;          // [2]
  uint64_t *acc_empty = acc_full + 2;       // [2]
  uint32_t *tmem_slot = reinterpret_cast<uint32_t *>(acc_empty + 2);
  volatile int *abort_flag = reinterpret_cast<volatile int *>(tmem_slot + 1);
  // per-column constants of this CTA's columns, 16-byte aligned: bias (0 where none applies), GAT attention vectors
  float *bias_s = reinterpret_cast<float *>((reinterpret_cast<uintptr_t>(tmem_slot + 2) + 15) & ~(uintptr_t)15);   // [nbc]
  float *att_s = bias_s + p.nbc;   // [2][nbc]: source vector, destination vector (only with scores)

  // fp32 mode: columns [nbc, 2 nbc) of an accumulator hold A_hi * B_lo, added to the first half by the epilogue
  const uint32_t acc_cols = (uint32_t)p.nbc * (TF32 ? 2u : 1u);
  const uint32_t a_col0 = 2 * acc_cols;   // fp32 mode: the split A stages follow the two accumulators
  uint32_t tmem_cols = 32;
  while (tmem_cols < 2 * acc_cols + (TF32 ? (uint32_t)p.tstages * TC_TSTAGE_COLS : 0u)) tmem_cols <<= 1;

  if (threadIdx.x == 0) {
    for (int s = 0; s < p.stages; ++s) {
      mbar_init(&full[s], 1);
      mbar_init(&empty[s], TF32 ? 4 : 1);
    }
    for (int s = 0; s < TC_TSTAGES_MAX; ++s) {
      mbar_init(&ready[s], 4);
      mbar_init(&a_free[s], 1);
    }
    mbar_init(b_full, 1);
    for (int a = 0; a < 2; ++a) {
      mbar_init(&acc_full[a], 1);
      mbar_init(&acc_empty[a], p.tma_store ? TC_EPI_WARPS / p.epi_groups : TC_EPI_WARPS);
    }
    *abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 1) {
    tmem_alloc(tmem_slot, tmem_cols);
    tmem_relinquish();
  }
  for (int c = threadIdx.x; c < p.nbc; c += blockDim.x) {
    const int gc = (blockIdx.x % p.n_splits) * p.nbc + c;
    bias_s[c] = (p.bias0 && gc < p.n0) ? p.bias0[gc] : 0.f;
    if (p.scores) {
      att_s[c] = p.att_src[gc];
      att_s[p.nbc + c] = p.att_dst[gc];
    }
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;

  const int n_tiles = p.n_tiles_m * p.n_splits;
  const int my_split = blockIdx.x % p.n_splits;   // gridDim.x is a multiple of n_splits: constant per CTA
  const int col_base = my_split * p.nbc;

  if (warp == 0) {
    // ------------------------------------------------------------------ TMA producer
    if (lane == 0 && !p.no_loads) {
      // the weights of this CTA's columns, once
      mbar_arrive_expect_tx(b_full, (uint32_t)b_bytes);
      const int bk_elems = TF32 ? 32 : 64;
      // fp32 mode: the hi and the lo tile of a k-block sit next to each other, so that one descriptor covers
      // both as a single operand of 2 nbc columns
      constexpr int parts = TF32 ? 2 : 1;
      for (int part = 0; part < parts; ++part)
        for (int kb = 0; kb < KB; ++kb)
          tma_load_2d(smem_b + (size_t)(kb * parts + part) * b_tile_bytes, &map_b, kb * bk_elems, part * p.NB + col_base, b_full);
      uint32_t stage = 0, phase = 0;
      bool ok = true;
      for (int tile = blockIdx.x; tile < n_tiles && ok; tile += gridDim.x) {
        const int m0 = (tile / p.n_splits) * TC_BM;
        for (int kb = 0; kb < KB; ++kb) {
          ok = mbar_wait(&empty[stage], phase ^ 1u, abort_flag, p.spin_limit, IT_TC_TMA_BACKOFF);
          if (!ok) break;
          mbar_arrive_expect_tx(&full[stage], (uint32_t)a_tile_bytes);
          if (kb < p.kb1) tma_load_2d(smem_a + (size_t)stage * a_tile_bytes, &map_x1, kb * bk_elems, m0, &full[stage]);
          else tma_load_2d(smem_a + (size_t)stage * a_tile_bytes, &map_x2, (kb - p.kb1) * bk_elems, m0, &full[stage]);
          if (++stage == (uint32_t)p.stages) { stage = 0; phase ^= 1u; }
        }
      }
      if (!ok) {
        // aborting: give the copies that were issued time to land before the CTA may exit (bounded)
        for (int s = 0; s < p.stages; ++s)
          for (uint32_t it = 0; it < TC_SPIN_LIMIT; ++it)
            if (mbar_try_wait(&full[s], 0) || mbar_try_wait(&full[s], 1)) break;
      }
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------------ MMA issuer
    if (lane == 0) {
      // instruction descriptor: D = fp32, A/B = bf16 or tf32, both K-major, N = nbc, M = 128
      const uint32_t fmt = TF32 ? 2u : 1u;
      const uint32_t idesc = (1u << 4) | (fmt << 7) | (fmt << 10) | ((uint32_t)(p.nbc >> 3) << 17) | ((uint32_t)(TC_BM >> 4) << 24);
      const uint32_t idesc_wide = (1u << 4) | (fmt << 7) | (fmt << 10) | ((uint32_t)((2 * p.nbc) >> 3) << 17) | ((uint32_t)(TC_BM >> 4) << 24);
      bool ok = mbar_wait(b_full, 0, abort_flag, p.spin_limit);
      uint32_t stage = 0, phase = 0;
      uint32_t acc = 0, acc_phase = 0;
      uint32_t ts = 0, tphase = 0;   // fp32 mode: TMEM stage of the split A k-block
      for (int tile = blockIdx.x; tile < n_tiles && ok; tile += gridDim.x) {
        ok = mbar_wait(&acc_empty[acc], acc_phase ^ 1u, abort_flag, p.spin_limit);
        if (!ok) break;
        tc_fence_after();
        const uint32_t d_tmem = tmem_base + acc * acc_cols;
        for (int kb = 0; kb < KB; ++kb) {
          const uint32_t b_hi = smem_u32(smem_b + (size_t)kb * (TF32 ? 2 : 1) * b_tile_bytes);
          if (TF32) {
            ok = mbar_wait(&ready[ts], tphase, abort_flag, p.spin_limit);
            if (!ok) break;
            tc_fence_after();
            const uint32_t a_hi = tmem_base + a_col0 + ts * TC_TSTAGE_COLS, a_lo = a_hi + 32;
#pragma unroll
            for (int k = 0; k < 4; ++k) {   // four K steps of 8 tf32 elements: 8 TMEM columns of A, 32 bytes of a B row
              // A_hi * [B_hi | B_lo] in one instruction, then A_lo * B_hi onto the first half
              tc_mma_tf32_tmem_a(d_tmem, a_hi + k * 8, make_desc(b_hi + k * 32), idesc_wide, (kb | k) != 0);
              tc_mma_tf32_tmem_a(d_tmem, a_lo + k * 8, make_desc(b_hi + k * 32), idesc, 1u);
            }
            tc_commit(&a_free[ts]);   // TMEM stage reusable once these MMAs have read it
            if (++ts == (uint32_t)p.tstages) { ts = 0; tphase ^= 1u; }
          } else {
            ok = mbar_wait(&full[stage], phase, abort_flag, p.spin_limit);
            if (!ok) break;
            tc_fence_after();
            const uint32_t a_s = smem_u32(smem_a + (size_t)stage * a_tile_bytes);
#pragma unroll
            for (int k = 0; k < 4; ++k)   // four 32-byte K steps inside the 128-byte swizzle row
              tc_mma<TF32>(d_tmem, make_desc(a_s + k * 32), make_desc(b_hi + k * 32), idesc, (kb | k) != 0);
            tc_commit(&empty[stage]);   // stage reusable once these MMAs have read it
            if (++stage == (uint32_t)p.stages) { stage = 0; phase ^= 1u; }
          }
        }
        if (!ok) break;
        tc_commit(&acc_full[acc]);    // accumulator complete
        if (++acc == 2) { acc = 0; acc_phase ^= 1u; }
      }
    }
  } else if (warp < 2 + TC_EPI_WARPS) {
    // ------------------------------------------------------------------ epilogue
    // 16 warps: 4 TMEM lane quarters x 4 column sub-sets.  Sub-set `sub` of a quarter takes the 16-column
    // groups g with g % 4 == sub, or, when attention scores are accumulated, the heads h with h % 4 == sub
    // (so that one warp sees every column of a head).
    const int quarter = warp & 3;   // a warp may only touch TMEM lanes [32 * (warp % 4), +32)
    const int sub = (warp - 2) >> 2;
    const int row_in_tile = quarter * 32 + lane;
    const bool odd = lane & 1;
    uint32_t acc = 0, acc_phase = 0;
    bool ok = true;
    const int n01 = p.n0 + p.n1;
    const int gph = p.scores ? p.head_dim / 16 : 1;          // 16-column groups per ownership unit
    const int n_units = (p.nbc / 16) / gph;                   // units in this CTA's columns
    const int unit0 = p.scores ? col_base / p.head_dim : 0;   // global index of the first unit (head)
    if (p.tma_store) {
      // ---- staged epilogue: every warp converts its 16-column groups and drops them, 128-byte-swizzled, into the
      // panels of the staging tile; one thread then writes each panel with a TMA store (whole 128-byte lines, and
      // per lane only: TMEM load, bias, activation, pack, shared-memory store).  The output columns of this CTA
      // are a run of out0 columns [lo0, hi0) and a run of out1 columns; each run is a whole number of panels.
      const int s0 = p.out0_bf16 ? 2 : 4, s1 = p.out1_bf16 ? 2 : 4;
      const int lo0 = col_base < p.n0 ? col_base : p.n0;
      const int hi0 = (col_base + p.nbc) < p.n0 ? (col_base + p.nbc) : p.n0;
      const int lo1 = col_base > p.n0 ? col_base : p.n0;
      const int hi1 = (col_base + p.nbc) < n01 ? (col_base + p.nbc) : n01;
      const int pan0 = hi0 > lo0 ? ((hi0 - lo0) * s0) / 128 : 0;
      const int pan1 = hi1 > lo1 ? ((hi1 - lo1) * s1) / 128 : 0;
      // With two groups, group g takes the tiles that land in accumulator g, so that the epilogues of two tiles run
      // side by side (one tile's epilogue is a chain of latencies: barrier, TMEM loads, shared-memory stores, fence).
      const int G = p.epi_groups, wpg = TC_EPI_WARPS / G;   // groups, warps per group
      const int group = (warp - 2) / wpg;
      const int gsub = ((warp - 2) % wpg) >> 2, n_sub = wpg >> 2;   // this warp's column sub-set inside its group
      unsigned char *my_out = smem_out + (size_t)group * p.out_panels * a_tile_bytes;
      const uint32_t out_base = smem_u32(my_out) + (uint32_t)row_in_tile * 128u;
      const uint32_t swz = (uint32_t)(row_in_tile & 7);
      const bool issuer = (warp - 2) % wpg == 0 && lane == 0;
      int last_u = -1;   // the last unit this warp owns (ownership: (unit0 + u) % n_sub == gsub)
      for (int u = n_units - 1; u >= 0; --u)
        if ((unit0 + u) % n_sub == gsub) { last_u = u; break; }
      int it = 0;   // tiles of this CTA so far: tile `it` uses accumulator it % 2, for the (it / 2)-th time
      for (int tile = blockIdx.x; tile < n_tiles; tile += gridDim.x, ++it) {
        if (G == 2 && (it & 1) != group) continue;
        acc = (uint32_t)it & 1u;
        acc_phase = ((uint32_t)it >> 1) & 1u;
        const int m0 = (tile / p.n_splits) * TC_BM;
        const int64_t m = (int64_t)m0 + row_in_tile;
        ok = mbar_wait(&acc_full[acc], acc_phase, abort_flag, p.spin_limit, IT_TC_EPI_BACKOFF);
        if (issuer) tma_store_wait_read();   // the stores of this group's previous tile have read the staging tile
        // one decision for all warps of the group (they meet at named barriers below, so none may leave alone)
        __syncwarp();
        if (epi_bar_any(G, group, !ok)) { ok = false; break; }
        tc_fence_after();
        const uint32_t taddr = tmem_base + ((uint32_t)(quarter * 32) << 16) + acc * acc_cols;
        bool released = false;
        for (int u = 0; u < n_units; ++u) {
          if ((unit0 + u) % n_sub != gsub) continue;
          float sc_a = 0.f, sc_b = 0.f;   // attention scores of this head
          for (int j0 = 0; j0 < gph; ++j0) {
            const int c = (u * gph + j0) * 16;   // local column of the group
            const int gc = col_base + c;         // global column; a group never straddles an output segment
            uint32_t r[16];
            tmem_ld16(taddr + (uint32_t)c, r);
            if (TF32) {
              uint32_t r2[16];
              tmem_ld16(taddr + (uint32_t)(p.nbc + c), r2);
              tmem_ld_wait();
#pragma unroll
              for (int i = 0; i < 16; ++i) r[i] = __float_as_uint(__uint_as_float(r[i]) + __uint_as_float(r2[i]));
            } else {
              tmem_ld_wait();
            }
            if (u == last_u && j0 + 1 == gph) {   // everything this warp needs is in registers: hand the accumulator back
              tc_fence_before();
              __syncwarp();
              if (lane == 0) mbar_arrive(&acc_empty[acc]);
              released = true;
            }
            float v[16];
#pragma unroll
            for (int i = 0; i < 16; ++i) v[i] = __uint_as_float(r[i]);
            if (p.scores) {   // GAT: attention scores from the unrounded accumulators
              const float4 *as4 = reinterpret_cast<const float4 *>(att_s + c);
              const float4 *ad4 = reinterpret_cast<const float4 *>(att_s + p.nbc + c);
#pragma unroll
              for (int i = 0; i < 4; ++i) {
                const float4 a4 = as4[i], d4 = ad4[i];
                sc_a = fmaf(v[4 * i], a4.x, sc_a); sc_a = fmaf(v[4 * i + 1], a4.y, sc_a);
                sc_a = fmaf(v[4 * i + 2], a4.z, sc_a); sc_a = fmaf(v[4 * i + 3], a4.w, sc_a);
                sc_b = fmaf(v[4 * i], d4.x, sc_b); sc_b = fmaf(v[4 * i + 1], d4.y, sc_b);
                sc_b = fmaf(v[4 * i + 2], d4.z, sc_b); sc_b = fmaf(v[4 * i + 3], d4.w, sc_b);
              }
            }
            if (gc >= n01) continue;
            int bf16, boff;   // output type, byte offset of the group inside the staging row of this CTA
            if (gc < p.n0) {
              const float4 *bs = reinterpret_cast<const float4 *>(bias_s + c);
#pragma unroll
              for (int i = 0; i < 4; ++i) {
                const float4 b4 = bs[i];
                v[4 * i] += b4.x; v[4 * i + 1] += b4.y; v[4 * i + 2] += b4.z; v[4 * i + 3] += b4.w;
              }
              if (p.act0 == IT_ACT_RELU) {
#pragma unroll
                for (int i = 0; i < 16; ++i) v[i] = fmaxf(v[i], 0.f);
              } else if (p.act0 == IT_ACT_ELU) {
#pragma unroll
                for (int i = 0; i < 16; ++i) v[i] = it_elu(v[i]);
              }
              bf16 = p.out0_bf16; boff = (gc - lo0) * s0;
            } else {
              bf16 = p.out1_bf16; boff = pan0 * 128 + (gc - lo1) * s1;
            }
            // panel = boff / 128 (16 KB each), 16-byte chunk inside the row = (boff % 128) / 16, swizzled by the row
            const uint32_t pbase = out_base + (uint32_t)(boff >> 7) * (uint32_t)a_tile_bytes;
            const uint32_t ch = (uint32_t)(boff & 127) >> 4;
            if (bf16) {
              uint32_t w[8];
#pragma unroll
              for (int i = 0; i < 8; ++i) {
                __nv_bfloat162 h2 = __floats2bfloat162_rn(v[2 * i], v[2 * i + 1]);
                w[i] = *reinterpret_cast<uint32_t *>(&h2);
              }
              st_shared_v4(pbase + (((ch + 0) ^ swz) << 4), w[0], w[1], w[2], w[3]);
              st_shared_v4(pbase + (((ch + 1) ^ swz) << 4), w[4], w[5], w[6], w[7]);
            } else {
#pragma unroll
              for (int q = 0; q < 4; ++q)
                st_shared_v4(pbase + (((ch + q) ^ swz) << 4), __float_as_uint(v[4 * q]), __float_as_uint(v[4 * q + 1]),
                             __float_as_uint(v[4 * q + 2]), __float_as_uint(v[4 * q + 3]));
            }
          }
          if (p.scores && m < p.M) {
            const int h = unit0 + u;
            p.scores[m * 2 * p.heads + h] = sc_a;
            p.scores[m * 2 * p.heads + p.heads + h] = sc_b;
          }
        }
        if (!released) {   // a warp that owns no columns of this CTA still has to sign off
          tc_fence_before();
          __syncwarp();
          if (lane == 0) mbar_arrive(&acc_empty[acc]);
        }
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");   // generic writes -> visible to the TMA store's reads
        epi_bar_sync(G, group);
        if (issuer) {
          for (int k = 0; k < pan0; ++k)
            tma_store_2d(&map_o0, my_out + (size_t)k * a_tile_bytes, lo0 + k * (128 / s0), m0);
          for (int k = 0; k < pan1; ++k)
            tma_store_2d(&map_o1, my_out + (size_t)(pan0 + k) * a_tile_bytes, (lo1 - p.n0) + k * (128 / s1), m0);
          tma_store_commit();
        }
      }
      if (issuer) tma_store_wait_all();   // the staging tile must outlive the last stores
    } else
    for (int tile = blockIdx.x; tile < n_tiles && ok; tile += gridDim.x) {
      const int64_t m = (int64_t)(tile / p.n_splits) * TC_BM + row_in_tile;
      const int64_t m_even = m - (odd ? 1 : 0), m_odd = m_even + 1;   // the two rows a lane pair writes together
      ok = mbar_wait(&acc_full[acc], acc_phase, abort_flag, p.spin_limit, IT_TC_EPI_BACKOFF);
      ok = __all_sync(0xffffffffu, ok);
      if (!ok) break;
      tc_fence_after();
      const uint32_t taddr = tmem_base + ((uint32_t)(quarter * 32) << 16) + acc * acc_cols;
      bool released = false;
      auto release = [&]() {   // everything this warp needs is in registers: hand the accumulator back
        tc_fence_before();
        __syncwarp();
        if (lane == 0) mbar_arrive(&acc_empty[acc]);
        released = true;
      };
      // the last unit this warp owns (ownership: (unit0 + u) % 4 == sub)
      int last_u = -1;
      for (int u = n_units - 1; u >= 0; --u)
        if (((unit0 + u) & 3) == sub) { last_u = u; break; }
      for (int u = 0; u < n_units; ++u) {
        if (((unit0 + u) & 3) != sub) continue;
        float sc_a = 0.f, sc_b = 0.f;   // attention scores of this head
        constexpr int GSTEP = TF32 ? 1 : 2;
        for (int j0 = 0; j0 < gph; j0 += GSTEP) {
          // two loads of 16 columns in flight from TMEM, one wait: two groups, or (fp32 mode) one group and its
          // A_hi * B_lo correction
          uint32_t r[2][16];
          const int c_first = (u * gph + j0) * 16;          // local column of the first group
          const int n_g = TF32 ? 1 : ((gph - j0) >= 2 ? 2 : 1);
          tmem_ld16(taddr + (uint32_t)c_first, r[0]);
          if (TF32) tmem_ld16(taddr + (uint32_t)(p.nbc + c_first), r[1]);
          else if (n_g == 2) tmem_ld16(taddr + (uint32_t)c_first + 16, r[1]);
          tmem_ld_wait();
          if (u == last_u && j0 + GSTEP >= gph) release();
          if (TF32) {
#pragma unroll
            for (int i = 0; i < 16; ++i) r[0][i] = __float_as_uint(__uint_as_float(r[0][i]) + __uint_as_float(r[1][i]));
          }
#pragma unroll
          for (int k = 0; k < 2; ++k) {
            if (k >= n_g) break;
            const int c = c_first + 16 * k;   // local column of r[k][0]
            const int gc = col_base + c;      // global column; a group never straddles an output segment
            float v[16];
#pragma unroll
            for (int i = 0; i < 16; ++i) v[i] = __uint_as_float(r[k][i]);
            if (p.scores) {   // GAT: attention scores from the unrounded accumulators
              const float4 *as4 = reinterpret_cast<const float4 *>(att_s + c);
              const float4 *ad4 = reinterpret_cast<const float4 *>(att_s + p.nbc + c);
#pragma unroll
              for (int i = 0; i < 4; ++i) {
                const float4 a4 = as4[i], d4 = ad4[i];
                sc_a = fmaf(v[4 * i], a4.x, sc_a); sc_a = fmaf(v[4 * i + 1], a4.y, sc_a);
                sc_a = fmaf(v[4 * i + 2], a4.z, sc_a); sc_a = fmaf(v[4 * i + 3], a4.w, sc_a);
                sc_b = fmaf(v[4 * i], d4.x, sc_b); sc_b = fmaf(v[4 * i + 1], d4.y, sc_b);
                sc_b = fmaf(v[4 * i + 2], d4.z, sc_b); sc_b = fmaf(v[4 * i + 3], d4.w, sc_b);
              }
            }
            if (gc >= n01) continue;
            void *dst; int bf16; int ld; int lc;
            if (gc < p.n0) {
              const float4 *bs = reinterpret_cast<const float4 *>(bias_s + c);
#pragma unroll
              for (int i = 0; i < 4; ++i) {
                const float4 b4 = bs[i];
                v[4 * i] += b4.x; v[4 * i + 1] += b4.y; v[4 * i + 2] += b4.z; v[4 * i + 3] += b4.w;
              }
              if (p.act0 == IT_ACT_RELU) {
#pragma unroll
                for (int i = 0; i < 16; ++i) v[i] = fmaxf(v[i], 0.f);
              } else if (p.act0 == IT_ACT_ELU) {
#pragma unroll
                for (int i = 0; i < 16; ++i) v[i] = it_elu(v[i]);
              }
              dst = p.out0; bf16 = p.out0_bf16; ld = p.n0; lc = gc;
            } else {
              dst = p.out1; bf16 = p.out1_bf16; ld = p.n1; lc = gc - p.n0;
            }
            // A lane pair (rows m_even, m_odd) swaps halves so that every store instruction writes whole
            // 32-byte sectors: the even lane takes the low 16 bytes of each 32-byte piece, the odd lane the high.
            if (bf16) {
              uint32_t w[8];
#pragma unroll
              for (int i = 0; i < 8; ++i) {
                __nv_bfloat162 h2 = __floats2bfloat162_rn(v[2 * i], v[2 * i + 1]);
                w[i] = *reinterpret_cast<uint32_t *>(&h2);
              }
              uint32_t got[4];
#pragma unroll
              for (int i = 0; i < 4; ++i) got[i] = __shfl_xor_sync(0xffffffffu, odd ? w[i] : w[4 + i], 1);
              // even lane: row_even bytes 0-15 (own w0-3), row_odd bytes 0-15 (partner's w0-3)
              // odd lane : row_even bytes 16-31 (partner's w4-7), row_odd bytes 16-31 (own w4-7)
              __nv_bfloat16 *o = reinterpret_cast<__nv_bfloat16 *>(dst) + lc + (odd ? 8 : 0);
              const uint4 first = odd ? make_uint4(got[0], got[1], got[2], got[3]) : make_uint4(w[0], w[1], w[2], w[3]);
              const uint4 second = odd ? make_uint4(w[4], w[5], w[6], w[7]) : make_uint4(got[0], got[1], got[2], got[3]);
              if (m_even < p.M) *reinterpret_cast<uint4 *>(o + m_even * ld) = first;
              if (m_odd < p.M) *reinterpret_cast<uint4 *>(o + m_odd * ld) = second;
            } else {
              float got[8];
#pragma unroll
              for (int i = 0; i < 4; ++i) {
                got[i] = __shfl_xor_sync(0xffffffffu, odd ? v[i] : v[4 + i], 1);           // columns 0-3 <-> 4-7
                got[4 + i] = __shfl_xor_sync(0xffffffffu, odd ? v[8 + i] : v[12 + i], 1);  // columns 8-11 <-> 12-15
              }
              // even lane: row_even cols 0-3, 8-11 (own); row_odd cols 0-3, 8-11 (partner's)
              // odd lane : row_even cols 4-7, 12-15 (partner's); row_odd cols 4-7, 12-15 (own)
              float *o = reinterpret_cast<float *>(dst) + lc + (odd ? 4 : 0);
              float4 e0, e1, o0, o1;
              if (!odd) {
                e0 = make_float4(v[0], v[1], v[2], v[3]); e1 = make_float4(v[8], v[9], v[10], v[11]);
                o0 = make_float4(got[0], got[1], got[2], got[3]); o1 = make_float4(got[4], got[5], got[6], got[7]);
              } else {
                e0 = make_float4(got[0], got[1], got[2], got[3]); e1 = make_float4(got[4], got[5], got[6], got[7]);
                o0 = make_float4(v[4], v[5], v[6], v[7]); o1 = make_float4(v[12], v[13], v[14], v[15]);
              }
              if (m_even < p.M) {
                *reinterpret_cast<float4 *>(o + m_even * ld) = e0;
                *reinterpret_cast<float4 *>(o + m_even * ld + 8) = e1;
              }
              if (m_odd < p.M) {
                *reinterpret_cast<float4 *>(o + m_odd * ld) = o0;
                *reinterpret_cast<float4 *>(o + m_odd * ld + 8) = o1;
              }
            }
          }
        }
        if (p.scores && m < p.M) {
          const int h = unit0 + u;
          p.scores[m * 2 * p.heads + h] = sc_a;
          p.scores[m * 2 * p.heads + p.heads + h] = sc_b;
        }
      }
      if (!released) release();   // a warp that owns no columns of this CTA still has to sign off
      if (++acc == 2) { acc = 0; acc_phase ^= 1u; }
    }
  } else {
    // ------------------------------------------------------------------ fp32 mode: split A into hi + lo, into TMEM
    // Thread = one row of the tile (TMEM lane quarter = warp index % 4).  The row's 128 bytes of the k-block are
    // eight 16-byte chunks, chunk c stored at position c ^ (row % 8) by the 128-byte swizzle of the TMA copy.
    if (TF32) {
      const int row = (warp & 3) * 32 + lane;
      const uint32_t t_lane = tmem_base + ((uint32_t)((warp & 3) * 32) << 16) + a_col0;
      const uint32_t group = (uint32_t)(warp - (TC_THREADS_BF16 >> 5)) >> 2;
      uint32_t stage = 0, phase = 0;
      uint32_t ts = 0, tphase = 0;
      uint32_t c = 0;   // k-blocks since the start of the CTA
      bool ok = true;
      for (int tile = blockIdx.x; tile < n_tiles && ok; tile += gridDim.x) {
        for (int kb = 0; kb < KB; ++kb, ++c) {
          if (c % TC_SPLIT_GROUPS != group) {   // another group's k-block: only keep the ring positions in step
            if (++stage == (uint32_t)p.stages) { stage = 0; phase ^= 1u; }
            if (++ts == (uint32_t)p.tstages) { ts = 0; tphase ^= 1u; }
            continue;
          }
          ok = mbar_wait(&full[stage], phase, abort_flag, p.spin_limit);
          ok = __all_sync(0xffffffffu, ok);
          if (!ok) break;
          const unsigned char *row_base = smem_a + (size_t)stage * a_tile_bytes + (size_t)row * TC_KBLOCK_BYTES;
          float4 x[8];
#pragma unroll
          for (int c = 0; c < 8; ++c) x[c] = *reinterpret_cast<const float4 *>(row_base + ((c ^ (row & 7)) << 4));
          ok = mbar_wait(&a_free[ts], tphase ^ 1u, abort_flag, p.spin_limit);
          ok = __all_sync(0xffffffffu, ok);
          if (!ok) break;
          tc_fence_after();
          const uint32_t t_hi = t_lane + ts * TC_TSTAGE_COLS, t_lo = t_hi + 32;
#pragma unroll
          for (int half = 0; half < 2; ++half) {
            uint32_t h[16], l[16];
#pragma unroll
            for (int c = 0; c < 4; ++c) {
              const float4 v = x[half * 4 + c];
              const float e[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
              for (int i = 0; i < 4; ++i) {
                const uint32_t hb = __float_as_uint(e[i]) & 0xffffe000u;
                h[c * 4 + i] = hb;
                l[c * 4 + i] = __float_as_uint(e[i] - __uint_as_float(hb));
              }
            }
            tmem_st16(t_hi + half * 16, h);
            tmem_st16(t_lo + half * 16, l);
          }
          // the MMA issuer is waiting for this: tell it first
          tmem_st_wait();
          tc_fence_before();
          __syncwarp();
          if (lane == 0) mbar_arrive(&ready[ts]);
          // Every value read from the stage has been used, so the reads are complete; the proxy fence orders these
          // generic-proxy reads before the asynchronous-proxy write of the TMA copy that refills the stage.
          asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
          __syncwarp();
          if (lane == 0) mbar_arrive(&empty[stage]);
          if (++stage == (uint32_t)p.stages) { stage = 0; phase ^= 1u; }
          if (++ts == (uint32_t)p.tstages) { ts = 0; tphase ^= 1u; }
        }
      }
    }
  }

  // ------------------------------------------------------------------ teardown
  tc_fence_before();
  __syncthreads();
  if (threadIdx.x == 0 && *abort_flag && p.status) atomicExch(p.status, 1);
  if (warp == 1) {
    tc_fence_after();
    tmem_dealloc(tmem_base, tmem_cols);
  }
}

// ----------------------------------------------------------------------------- two products back to back (bf16)
// The update of one layer followed by the transform of the next, for a layer whose output feeds only that transform:
//   H[M, N1]  = act1([X1 | X2] * B1 + bias1), rounded to bf16 exactly as it would be stored,
//   C[M, N2]  = H * B2,  columns [0, n0) + bias0 -> out0, columns [n0, n0 + n1) -> out1.
// H never leaves the SM: the epilogue warps drain the first accumulator into shared memory in the 128-byte-swizzled
// K-major layout a TMA copy would have produced, and the second product reads it from there.  Same roles as the
// single product: warp 0 copies operand tiles, warp 1 issues the MMAs, two groups of eight epilogue warps take
// alternate tiles.  The MMA issuer runs one tile ahead with the first product (the second product of tile i is
// issued after the first product of tile i + 1), so the tensor core and the copies do not wait for an epilogue.
// A group's shared-memory tile holds H and then, once the second product has read it, the staged output.
struct Tc2Params {
  int64_t M;
  int n_tiles;
  int kb1, kb2;          // k-blocks of the first product that come from X1 / X2
  int N1;                // columns of H (a multiple of 64): N1 / 64 k-blocks of the second product
  int N2;                // columns of the second product (n0 + n1)
  int n0, n1;            // multiples of 64 (whole 128-byte panels of bf16)
  const float *bias1; int act1;
  const float *bias0;
  int stages;
  int buf_panels;        // 16 KB panels of one group's tile: max(N1, N2) / 64
  int *status;
  uint32_t spin_limit;
  int no_loads;          // test hook: the producer issues no copies, so every wait runs out
};

constexpr int TC2_GROUP_WARPS = TC_EPI_WARPS / 2;
#ifndef IT_TC2_BACKOFF
#define IT_TC2_BACKOFF 32   // ns between polls of the second accumulator's barrier
#endif

// One epilogue group drains `ncols` accumulator columns of its TMEM lane quarter into the panels of its tile:
// column c of row r lands at byte 2 c of the row, panel (2 c) / 128, 16-byte chunk ((2 c) % 128) / 16 xor (r % 8).
// `cst` holds one fp32 constant per column (added), `act_cols` columns from the left get the activation.
__device__ __forceinline__ void tc2_drain(uint32_t taddr, int ncols, int gsub, const float *cst, int act, int act_cols,
                                          uint32_t out_row, uint32_t swz, uint64_t *release_bar, int lane) {
  const int n_groups = ncols >> 4;   // 16-column groups; this warp takes those with index % 2 == gsub, two per TMEM wait
  // bias, activation, bf16, swizzled store of one 16-column group held in r
  auto finish = [&](int c, const uint32_t (&r)[16]) {
    float v[16];
    const float4 *c4 = reinterpret_cast<const float4 *>(cst + c);
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      const float4 b4 = c4[i];
      v[4 * i] = __uint_as_float(r[4 * i]) + b4.x; v[4 * i + 1] = __uint_as_float(r[4 * i + 1]) + b4.y;
      v[4 * i + 2] = __uint_as_float(r[4 * i + 2]) + b4.z; v[4 * i + 3] = __uint_as_float(r[4 * i + 3]) + b4.w;
    }
    if (c < act_cols) {
      if (act == IT_ACT_RELU) {
#pragma unroll
        for (int i = 0; i < 16; ++i) v[i] = fmaxf(v[i], 0.f);
      } else if (act == IT_ACT_ELU) {
#pragma unroll
        for (int i = 0; i < 16; ++i) v[i] = it_elu(v[i]);
      }
    }
    uint32_t w[8];
#pragma unroll
    for (int i = 0; i < 8; ++i) {
      __nv_bfloat162 h2 = __floats2bfloat162_rn(v[2 * i], v[2 * i + 1]);
      w[i] = *reinterpret_cast<uint32_t *>(&h2);
    }
    const uint32_t boff = (uint32_t)c * 2u;
    const uint32_t pbase = out_row + (boff >> 7) * (uint32_t)(TC_BM * TC_KBLOCK_BYTES);
    const uint32_t ch = (boff & 127u) >> 4;
    st_shared_v4(pbase + (((ch + 0) ^ swz) << 4), w[0], w[1], w[2], w[3]);
    st_shared_v4(pbase + (((ch + 1) ^ swz) << 4), w[4], w[5], w[6], w[7]);
  };
  bool released = false;
  for (int gidx = gsub; gidx < n_groups; gidx += 4) {
    const bool two = gidx + 2 < n_groups;
    uint32_t r0[16], r1[16];
    tmem_ld16(taddr + (uint32_t)(gidx << 4), r0);
    if (two) tmem_ld16(taddr + (uint32_t)((gidx + 2) << 4), r1);
    tmem_ld_wait();
    if (gidx + 4 >= n_groups) {   // everything this warp needs is in registers: hand the accumulator back
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(release_bar);
      released = true;
    }
    finish(gidx << 4, r0);
    if (two) finish((gidx + 2) << 4, r1);
  }
  if (!released) {   // a warp that owns no columns still has to sign off
    tc_fence_before();
    __syncwarp();
    if (lane == 0) mbar_arrive(release_bar);
  }
}

__global__ void __launch_bounds__(TC_THREADS_BF16, 1)
gemm2_tc_kernel(const __grid_constant__ CUtensorMap map_x1, const __grid_constant__ CUtensorMap map_x2,
                const __grid_constant__ CUtensorMap map_b1, const __grid_constant__ CUtensorMap map_b2,
                const __grid_constant__ CUtensorMap map_o0, const __grid_constant__ CUtensorMap map_o1, const Tc2Params p) {
  extern __shared__ unsigned char smem_raw[];
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int KB1 = p.kb1 + p.kb2;
  const int KB2 = p.N1 >> 6;
  constexpr int a_tile_bytes = TC_BM * TC_KBLOCK_BYTES;          // 16 KB
  const int b1_tile_bytes = p.N1 * TC_KBLOCK_BYTES, b2_tile_bytes = p.N2 * TC_KBLOCK_BYTES;
  const int b1_bytes = KB1 * b1_tile_bytes, b2_bytes = KB2 * b2_tile_bytes;

  // shared memory: weights of both products | operand stages | one tile per epilogue group | barriers | constants
  unsigned char *base = reinterpret_cast<unsigned char *>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
  unsigned char *smem_b1 = base;
  unsigned char *smem_b2 = smem_b1 + b1_bytes;
  unsigned char *smem_a = smem_b2 + b2_bytes;
  unsigned char *smem_buf = smem_a + (size_t)p.stages * a_tile_bytes;
  uint64_t *bars = reinterpret_cast<uint64_t *>(smem_buf + (size_t)2 * p.buf_panels * a_tile_bytes);
  uint64_t *full = bars;                    // [stages]  TMA landed
  uint64_t *empty = bars + p.stages;        // [stages]  the MMAs that read the stage are done
  uint64_t *b_full = bars + 2 * p.stages;   // [1]
  uint64_t *acc1_full = b_full + 1;         // [2]  first product of a tile complete
  uint64_t *acc1_empty = acc1_full + 2;     // [2]  its accumulator drained
  uint64_t *h_full = acc1_empty + 2;        // [2]  H tile of the group written to shared memory
  uint64_t *acc2_full = h_full + 2;         // [2]  second product complete (and H read)
  uint64_t *acc2_empty = acc2_full + 2;     // [2]
  uint32_t *tmem_slot = reinterpret_cast<uint32_t *>(acc2_empty + 2);
  volatile int *abort_flag = reinterpret_cast<volatile int *>(tmem_slot + 1);
  float *cst1 = reinterpret_cast<float *>((reinterpret_cast<uintptr_t>(tmem_slot + 2) + 15) & ~(uintptr_t)15);   // [N1] bias of H
  float *cst2 = cst1 + p.N1;                                                                                     // [N2] bias0 | 0

  uint32_t tmem_cols = 32;
  while (tmem_cols < (uint32_t)(2 * (p.N1 + p.N2))) tmem_cols <<= 1;

  if (threadIdx.x == 0) {
    for (int s = 0; s < p.stages; ++s) {
      mbar_init(&full[s], 1);
      mbar_init(&empty[s], 1);
    }
    mbar_init(b_full, 1);
    for (int a = 0; a < 2; ++a) {
      mbar_init(&acc1_full[a], 1);
      mbar_init(&acc1_empty[a], TC2_GROUP_WARPS);
      mbar_init(&h_full[a], TC2_GROUP_WARPS);
      mbar_init(&acc2_full[a], 1);
      mbar_init(&acc2_empty[a], TC2_GROUP_WARPS);
    }
    *abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 1) {
    tmem_alloc(tmem_slot, tmem_cols);
    tmem_relinquish();
  }
  for (int c = threadIdx.x; c < p.N1; c += blockDim.x) cst1[c] = p.bias1 ? p.bias1[c] : 0.f;
  for (int c = threadIdx.x; c < p.N2; c += blockDim.x) cst2[c] = (p.bias0 && c < p.n0) ? p.bias0[c] : 0.f;
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;
  const uint32_t acc2_col0 = 2u * (uint32_t)p.N1;

  if (warp == 0) {
    // ------------------------------------------------------------------ TMA producer
    if (lane == 0 && !p.no_loads) {
      mbar_arrive_expect_tx(b_full, (uint32_t)(b1_bytes + b2_bytes));
      for (int kb = 0; kb < KB1; ++kb) tma_load_2d(smem_b1 + (size_t)kb * b1_tile_bytes, &map_b1, kb * 64, 0, b_full);
      for (int kb = 0; kb < KB2; ++kb) tma_load_2d(smem_b2 + (size_t)kb * b2_tile_bytes, &map_b2, kb * 64, 0, b_full);
      uint32_t stage = 0, phase = 0;
      bool ok = true;
      for (int tile = blockIdx.x; tile < p.n_tiles && ok; tile += gridDim.x) {
        const int m0 = tile * TC_BM;
        for (int kb = 0; kb < KB1; ++kb) {
          ok = mbar_wait(&empty[stage], phase ^ 1u, abort_flag, p.spin_limit, IT_TC_TMA_BACKOFF);
          if (!ok) break;
          mbar_arrive_expect_tx(&full[stage], (uint32_t)a_tile_bytes);
          if (kb < p.kb1) tma_load_2d(smem_a + (size_t)stage * a_tile_bytes, &map_x1, kb * 64, m0, &full[stage]);
          else tma_load_2d(smem_a + (size_t)stage * a_tile_bytes, &map_x2, (kb - p.kb1) * 64, m0, &full[stage]);
          if (++stage == (uint32_t)p.stages) { stage = 0; phase ^= 1u; }
        }
      }
      if (!ok) {
        // aborting: give the copies that were issued time to land before the CTA may exit (bounded)
        for (int s = 0; s < p.stages; ++s)
          for (uint32_t it = 0; it < TC_SPIN_LIMIT; ++it)
            if (mbar_try_wait(&full[s], 0) || mbar_try_wait(&full[s], 1)) break;
      }
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------------ MMA issuer
    if (lane == 0) {
      const uint32_t idesc1 = (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(p.N1 >> 3) << 17) | ((uint32_t)(TC_BM >> 4) << 24);
      const uint32_t idesc2 = (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(p.N2 >> 3) << 17) | ((uint32_t)(TC_BM >> 4) << 24);
      bool ok = mbar_wait(b_full, 0, abort_flag, p.spin_limit);
      uint32_t stage = 0, phase = 0;
      // second product of this CTA's tile number j (accumulator and group j % 2, used for the (j / 2)-th time)
      auto second = [&](int j) -> bool {
        const uint32_t a = (uint32_t)j & 1u, ph = ((uint32_t)j >> 1) & 1u;
        if (!mbar_wait(&acc2_empty[a], ph ^ 1u, abort_flag, p.spin_limit)) return false;
        if (!mbar_wait(&h_full[a], ph, abort_flag, p.spin_limit)) return false;
        tc_fence_after();
        const uint32_t d_tmem = tmem_base + acc2_col0 + a * (uint32_t)p.N2;
        const uint32_t h_s = smem_u32(smem_buf + (size_t)a * p.buf_panels * a_tile_bytes);
        for (int kb = 0; kb < KB2; ++kb) {
          const uint32_t a_s = h_s + (uint32_t)kb * (uint32_t)a_tile_bytes;
          const uint32_t b_s = smem_u32(smem_b2 + (size_t)kb * b2_tile_bytes);
#pragma unroll
          for (int k = 0; k < 4; ++k)
            tc_mma<false>(d_tmem, make_desc(a_s + k * 32), make_desc(b_s + k * 32), idesc2, (kb | k) != 0);
        }
        tc_commit(&acc2_full[a]);   // complete: the accumulator may be drained and the H tile overwritten
        return true;
      };
      int it = 0;
      for (int tile = blockIdx.x; tile < p.n_tiles && ok; tile += gridDim.x, ++it) {
        const uint32_t a = (uint32_t)it & 1u, ph = ((uint32_t)it >> 1) & 1u;
        ok = mbar_wait(&acc1_empty[a], ph ^ 1u, abort_flag, p.spin_limit);
        if (!ok) break;
        tc_fence_after();
        const uint32_t d_tmem = tmem_base + a * (uint32_t)p.N1;
        for (int kb = 0; kb < KB1; ++kb) {
          ok = mbar_wait(&full[stage], phase, abort_flag, p.spin_limit);
          if (!ok) break;
          tc_fence_after();
          const uint32_t a_s = smem_u32(smem_a + (size_t)stage * a_tile_bytes);
          const uint32_t b_s = smem_u32(smem_b1 + (size_t)kb * b1_tile_bytes);
#pragma unroll
          for (int k = 0; k < 4; ++k)
            tc_mma<false>(d_tmem, make_desc(a_s + k * 32), make_desc(b_s + k * 32), idesc1, (kb | k) != 0);
          tc_commit(&empty[stage]);
          if (++stage == (uint32_t)p.stages) { stage = 0; phase ^= 1u; }
        }
        if (!ok) break;
        tc_commit(&acc1_full[a]);
        if (it > 0) ok = second(it - 1);
      }
      if (ok && it > 0) second(it - 1);
    }
  } else {
    // ------------------------------------------------------------------ epilogue: group g takes the tiles it % 2 == g
    const int quarter = warp & 3;   // a warp may only touch TMEM lanes [32 * (warp % 4), +32)
    const int group = (warp - 2) / TC2_GROUP_WARPS;
    const int gsub = ((warp - 2) % TC2_GROUP_WARPS) >> 2;   // which of the two warps of this quarter in the group
    const int row_in_tile = quarter * 32 + lane;
    unsigned char *my_buf = smem_buf + (size_t)group * p.buf_panels * a_tile_bytes;
    const uint32_t out_row = smem_u32(my_buf) + (uint32_t)row_in_tile * 128u;
    const uint32_t swz = (uint32_t)(row_in_tile & 7);
    const bool issuer = (warp - 2) % TC2_GROUP_WARPS == 0 && lane == 0;
    const uint32_t lane_base = (uint32_t)(quarter * 32) << 16;
    const int pan0 = p.n0 >> 6, pan1 = p.n1 >> 6;
    int it = 0;
    for (int tile = blockIdx.x; tile < p.n_tiles; tile += gridDim.x, ++it) {
      if ((it & 1) != group) continue;
      const uint32_t ph = ((uint32_t)it >> 1) & 1u;
      const int m0 = tile * TC_BM;
      // ---- first accumulator -> H tile (bias, activation, bf16, swizzled)
      bool ok = mbar_wait(&acc1_full[group], ph, abort_flag, p.spin_limit, IT_TC_EPI_BACKOFF);
      if (issuer) tma_store_wait_read();   // the stores of this group's previous tile have read the tile
      __syncwarp();
      if (epi_bar_any(2, group, !ok)) break;   // one decision for all warps of the group
      tc_fence_after();
      tc2_drain(tmem_base + lane_base + (uint32_t)group * (uint32_t)p.N1, p.N1, gsub, cst1, p.act1, p.N1, out_row, swz,
                &acc1_empty[group], lane);
      asm volatile("fence.proxy.async.shared::cta;" ::: "memory");   // generic writes -> visible to the tensor core's reads
      __syncwarp();
      if (lane == 0) mbar_arrive(&h_full[group]);
      // ---- second accumulator -> staged output (the H tile has been read), then TMA stores
      // (a short wait: the second product follows the H tile at once; a warp whose wait ran out skips the drain and the
      // group decides together at the barrier below, which the stores need anyway)
      ok = mbar_wait(&acc2_full[group], ph, abort_flag, p.spin_limit, IT_TC2_BACKOFF);
      ok = __all_sync(0xffffffffu, ok);
      if (ok) {
        tc_fence_after();
        tc2_drain(tmem_base + lane_base + acc2_col0 + (uint32_t)group * (uint32_t)p.N2, p.N2, gsub, cst2, IT_ACT_NONE, 0, out_row,
                  swz, &acc2_empty[group], lane);
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");   // generic writes -> visible to the TMA store's reads
      }
      if (epi_bar_any(2, group, !ok)) break;
      if (issuer) {
        for (int k = 0; k < pan0; ++k) tma_store_2d(&map_o0, my_buf + (size_t)k * a_tile_bytes, k * 64, m0);
        for (int k = 0; k < pan1; ++k) tma_store_2d(&map_o1, my_buf + (size_t)(pan0 + k) * a_tile_bytes, k * 64, m0);
        tma_store_commit();
      }
    }
    if (issuer) tma_store_wait_all();   // the tile must outlive the last stores
  }

  // ------------------------------------------------------------------ teardown
  tc_fence_before();
  __syncthreads();
  if (threadIdx.x == 0 && *abort_flag && p.status) atomicExch(p.status, 1);
  if (warp == 1) {
    tc_fence_after();
    tmem_dealloc(tmem_base, tmem_cols);
  }
}

// ----------------------------------------------------------------------------- weight prep (K-major, split)
struct PrepTcParams {
  int kind, in_dim, out_dim, w_is_bf16, NB;
  int K1, K1p, K2, K2p;   // rows of W behind X1 / X2, and the same rounded up to whole k-blocks (the padding is zero)
  const void *W;
  void *B;   // bf16 [NB, K1p + K2p]  or  fp32 [2, NB, K1p + K2p] (hi, lo)
};

__global__ void prep_weights_tc_kernel(PrepTcParams p) {
  const int Kp = p.K1p + p.K2p;
  const int64_t total = (int64_t)p.NB * Kp;
  for (int64_t i = blockIdx.x * (int64_t)blockDim.x + threadIdx.x; i < total; i += (int64_t)gridDim.x * blockDim.x) {
    const int n = (int)(i / Kp), kp = (int)(i % Kp);
    // padded position -> row of the unpadded product (or none)
    const bool second = kp >= p.K1p;
    const int kin = second ? kp - p.K1p : kp;
    const bool real = kin < (second ? p.K2 : p.K1);
    const int k = second ? p.K1 + kin : kin;
    int64_t src;   // element of W that is B[k, n]
    if (p.kind == IT_PREP_SAGE_REORDER) src = n < p.out_dim ? (int64_t)k * p.out_dim + n : (int64_t)(p.in_dim + k) * p.out_dim + (n - p.out_dim);
    else src = (int64_t)k * p.out_dim + n;
    if (p.w_is_bf16) {
      reinterpret_cast<__nv_bfloat16 *>(p.B)[i] = real ? reinterpret_cast<const __nv_bfloat16 *>(p.W)[src] : __float2bfloat16_rn(0.f);
    } else {
      const float w = real ? reinterpret_cast<const float *>(p.W)[src] : 0.f;
      // hi = w rounded to tf32 (nearest even on the 13 dropped bits), lo = the exact remainder
      uint32_t u = __float_as_uint(w);
      u += 0xfffu + ((u >> 13) & 1u);
      u &= 0xffffe000u;
      const float hi = __uint_as_float(u);
      reinterpret_cast<float *>(p.B)[i] = hi;
      reinterpret_cast<float *>(p.B)[total + i] = w - hi;
    }
  }
}

// ----------------------------------------------------------------------------- host side
typedef CUresult (*EncodeTiledFn)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *, const cuuint64_t *,
                                  const cuuint32_t *, const cuuint32_t *, CUtensorMapInterleave, CUtensorMapSwizzle,
                                  CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn get_encode() {
  static EncodeTiledFn fn = nullptr;
  if (!fn) {
    void *p = nullptr;
    cudaDriverEntryPointQueryResult qres;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &qres) == cudaSuccess && qres == cudaDriverEntryPointSuccess)
      fn = reinterpret_cast<EncodeTiledFn>(p);
  }
  return fn;
}

// 2-D row-major matrix [rows, cols] of `elem` bytes; box = 128 bytes of a row x box_rows rows, 128-byte swizzle.
it_status make_map(CUtensorMap *map, const void *ptr, int elem, int64_t rows, int64_t cols, int box_rows) {
  EncodeTiledFn enc = get_encode();
  IT_REQUIRE(enc != nullptr, IT_ERR_CUDA, "cuTensorMapEncodeTiled is not available from the driver");
  const cuuint64_t dims[2] = {(cuuint64_t)cols, (cuuint64_t)rows};
  const cuuint64_t strides[1] = {(cuuint64_t)cols * (cuuint64_t)elem};
  const cuuint32_t box[2] = {(cuuint32_t)(TC_KBLOCK_BYTES / elem), (cuuint32_t)box_rows};
  const cuuint32_t estr[2] = {1, 1};
  const CUtensorMapDataType dt = elem == 2 ? CU_TENSOR_MAP_DATA_TYPE_BFLOAT16 : CU_TENSOR_MAP_DATA_TYPE_FLOAT32;
  CUresult r = enc(map, dt, 2, const_cast<void *>(ptr), dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
                   CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  IT_REQUIRE(r == CUDA_SUCCESS, IT_ERR_CUDA, "cuTensorMapEncodeTiled failed with code %d", (int)r);
  return IT_OK;
}

constexpr int kSmemBudget = 227 * 1024;
constexpr int kSmemAux = 1024 /*alignment slack*/ + 288 /*barriers, TMEM slot, abort flag, alignment*/;

}  // namespace

size_t it_tc_weights_bytes(const it_layer_desc *L, int NB, int K) {
  return (size_t)NB * (K + 128) * (L->feat_dtype == IT_BF16 ? 2 : 8);   // room for the padding of both operands' K
}

// Column split of the tensor-core path: the largest columns-per-CTA count (a multiple of 16 that divides NB, at
// most 256) whose resident weights leave room for three operand stages (which already give the time of eight)
// and one 32 KB staging tile of the epilogue.
constexpr size_t kWeightBudget = kSmemBudget - kSmemAux - 1024 /*per-column constants*/ - 3 * TC_BM * TC_KBLOCK_BYTES - 32 * 1024;
static bool tc_split(bool tf32, int NB, int KB, int *n_splits, int *nbc) {
  for (int s = 1; s <= 16; ++s) {
    if (NB % s != 0) continue;
    const int c = NB / s;
    // fp32 mode issues MMAs of 2 c columns and keeps 4 c TMEM columns of accumulators next to the split A stages
    if (c % 16 != 0 || c > (tf32 ? 64 : 256)) continue;
    if ((size_t)(tf32 ? 2 : 1) * KB * c * TC_KBLOCK_BYTES > kWeightBudget) continue;
    *n_splits = s; *nbc = c;
    return true;
  }
  return false;
}

bool it_tc_supported(const it_gemm_args &a, int heads, int head_dim, bool want_scores) {
  const bool tf32 = a.x_dtype == IT_F32;
  const int elem = tf32 ? 4 : 2;
  const int bk = TC_KBLOCK_BYTES / elem;
  if (a.M <= 0 || a.M > (int64_t)INT32_MAX) return false;
  const int K2 = a.X2 ? a.K2 : 0;
  // operand rows must be TMA-addressable (a multiple of 16 bytes); a K that is not a whole number of k-blocks is
  // padded: the TMA copy fills what lies beyond a row with zeros and the prepared weights carry zero rows there
  if (a.K1 <= 0 || (a.K1 * elem) % 16 != 0 || (K2 * elem) % 16 != 0) return false;
  const int NB = a.n0 + a.n1;   // score columns are not materialised on this path
  if (NB <= 0 || NB % 16 != 0 || a.n0 % 16 != 0) return false;
  int n_splits, nbc;
  if (!tc_split(tf32, NB, (a.K1 + bk - 1) / bk + (K2 + bk - 1) / bk, &n_splits, &nbc)) return false;
  if (want_scores && (heads > 8 || head_dim % 16 != 0 || nbc % head_dim != 0)) return false;
  return true;
}

it_status it_launch_prep_weights_tc(it_prep_kind kind, const it_layer_desc *L, int NB, int K1, int K2, void *B, cudaStream_t st) {
  PrepTcParams p;
  const int bk = TC_KBLOCK_BYTES / (L->weight_dtype == IT_BF16 ? 2 : 4);
  p.kind = kind; p.in_dim = L->in_dim; p.out_dim = L->out_dim; p.w_is_bf16 = L->weight_dtype == IT_BF16;
  p.NB = NB; p.K1 = K1; p.K2 = K2; p.K1p = (K1 + bk - 1) / bk * bk; p.K2p = (K2 + bk - 1) / bk * bk; p.W = L->W; p.B = B;
  IT_LAUNCH(IT_K_PREP, 0, 0, st, prep_weights_tc_kernel<<<64, 256, 0, st>>>(p));
  IT_CUDA_TRY(cudaGetLastError());
  return IT_OK;
}

// B: weights prepared by it_launch_prep_weights_tc.  a.B / a.NB / a.out2 of the generic args are ignored:
// the tensor-core path computes n0 + n1 columns and, for GAT, the scores in its epilogue.
it_status it_launch_gemm_tc(const it_gemm_args &a, const void *B, const float *att_src, const float *att_dst, int heads,
                            int head_dim, float *scores, int num_sms, int *status, cudaStream_t st) {
  if (a.M == 0) return IT_OK;
  const bool tf32 = a.x_dtype == IT_F32;
  const int elem = tf32 ? 4 : 2;
  const int bk = TC_KBLOCK_BYTES / elem;
  const int NB = a.n0 + a.n1;
  const int K2 = a.X2 ? a.K2 : 0;
  const int K = a.K1 + K2;
  const int kb1 = (a.K1 + bk - 1) / bk, kb2 = (K2 + bk - 1) / bk;
  const int KB = kb1 + kb2;
  int n_splits = 1, nbc = NB;
  IT_REQUIRE(tc_split(tf32, NB, KB, &n_splits, &nbc), IT_ERR_UNSUPPORTED, "tensor-core apply: cannot tile %d columns with K = %d", NB, K);
  const int b_bytes = (tf32 ? 2 : 1) * KB * nbc * TC_KBLOCK_BYTES;
  const int stage_bytes = TC_BM * TC_KBLOCK_BYTES;             // one operand tile (fp32 mode: the raw tile)
  const int const_bytes = nbc * 4 * (scores ? 3 : 1);          // bias (+ attention vectors) of this CTA's columns
  // Staged epilogue (TMA stores): possible when, for every column split, the out0 columns and the out1 columns of
  // the CTA are whole 128-byte panels that start on a panel boundary, and three operand stages still fit beside
  // the staging tile (three stages already give the time of eight).
  const int s0 = a.dt0 == IT_BF16 ? 2 : 4, s1 = a.dt1 == IT_BF16 ? 2 : 4;
  int out_panels = 0;
  bool staged = IT_TC_TMA_STORE != 0;
  for (int sp = 0; sp < n_splits && staged; ++sp) {
    const int cb = sp * nbc, ce = cb + nbc;
    const int lo0 = cb < a.n0 ? cb : a.n0, hi0 = ce < a.n0 ? ce : a.n0;
    const int lo1 = cb > a.n0 ? cb : a.n0, hi1 = ce < NB ? ce : NB;
    const int b0 = hi0 > lo0 ? (hi0 - lo0) * s0 : 0, b1 = hi1 > lo1 ? (hi1 - lo1) * s1 : 0;
    if (b0 % 128 != 0 || b1 % 128 != 0 || (b0 > 0 && (lo0 * s0) % 128 != 0) || (b1 > 0 && ((lo1 - a.n0) * s1) % 128 != 0)) staged = false;
    if (b0 / 128 + b1 / 128 > out_panels) out_panels = b0 / 128 + b1 / 128;
  }
  // two groups of epilogue warps (alternate tiles, a staging tile each) when the second staging tile still fits
  int epi_groups = IT_TC_EPI_GROUPS;
  if (staged && epi_groups == 2 && (kSmemBudget - kSmemAux - const_bytes - b_bytes - 2 * out_panels * stage_bytes) / stage_bytes < 3) {
    epi_groups = 1;
    if (!tf32) staged = false;   // measured: one group beats the direct stores in fp32 mode only (its tiles take long enough)
  }
  if (staged && (kSmemBudget - kSmemAux - const_bytes - b_bytes - epi_groups * out_panels * stage_bytes) / stage_bytes < 3) staged = false;
  if (!staged) { out_panels = 0; epi_groups = 1; }
  int stages = (kSmemBudget - kSmemAux - const_bytes - b_bytes - epi_groups * out_panels * stage_bytes) / stage_bytes;
  if (stages > IT_TC_MAX_STAGES) stages = IT_TC_MAX_STAGES;
  IT_REQUIRE(stages >= 2, IT_ERR_UNSUPPORTED, "tensor-core apply: no room for two operand stages");
  const int smem = b_bytes + (stages + epi_groups * out_panels) * stage_bytes + kSmemAux + const_bytes;
  // fp32 mode: TMEM holds two accumulators of 2 nbc columns; what is left of its 512 columns stages the split A
  int tstages = tf32 ? (512 - 4 * nbc) / TC_TSTAGE_COLS : 0;
  if (tstages > TC_TSTAGES_MAX) tstages = TC_TSTAGES_MAX;
  IT_REQUIRE(!tf32 || tstages >= 2, IT_ERR_UNSUPPORTED, "tensor-core apply: no room in TMEM for two split A stages");

  CUtensorMap m1, m2, mb;
  IT_TRY(make_map(&m1, a.X1, elem, a.M, a.K1, TC_BM));
  if (a.X2) IT_TRY(make_map(&m2, a.X2, elem, a.M, K2, TC_BM));
  else m2 = m1;
  IT_TRY(make_map(&mb, B, elem, (int64_t)(tf32 ? 2 : 1) * NB, (int64_t)KB * bk, nbc));
  CUtensorMap mo0 = m1, mo1 = m1;   // placeholders unless the epilogue is staged
  if (staged && a.n0 > 0) IT_TRY(make_map(&mo0, a.out0, s0, a.M, a.n0, TC_BM));
  if (staged && a.n1 > 0) IT_TRY(make_map(&mo1, a.out1, s1, a.M, a.n1, TC_BM));

  TcParams p;
  p.M = a.M; p.n_tiles_m = (int)((a.M + TC_BM - 1) / TC_BM); p.n_splits = n_splits; p.nbc = nbc;
  p.kb1 = kb1; p.kb2 = kb2; p.NB = NB; p.stages = stages; p.tstages = tstages;
  p.n0 = a.n0; p.out0 = a.out0; p.out0_bf16 = a.dt0 == IT_BF16; p.bias0 = a.bias0; p.act0 = a.act0;
  p.n1 = a.n1; p.out1 = a.out1; p.out1_bf16 = a.dt1 == IT_BF16;
  p.scores = scores; p.att_src = att_src; p.att_dst = att_dst; p.heads = heads; p.head_dim = head_dim > 0 ? head_dim : 1;
  p.status = status;
  p.tma_store = staged ? 1 : 0; p.out_panels = out_panels; p.epi_groups = epi_groups;
  p.spin_limit = a.spin_limit ? a.spin_limit : TC_SPIN_LIMIT; p.no_loads = a.no_loads;

  const int64_t n_tiles = (int64_t)p.n_tiles_m * n_splits;
  int64_t grid = (int64_t)(num_sms / n_splits) * n_splits;
  if (grid > n_tiles) grid = n_tiles;   // n_tiles is a multiple of n_splits
  const double xs = elem;
  const double bytes = (double)a.M * (K * xs + a.n0 * (a.dt0 == IT_F32 ? 4.0 : 2.0) + a.n1 * (a.dt1 == IT_F32 ? 4.0 : 2.0) +
                                     (scores ? 8.0 * heads : 0.0)) + (double)K * NB * xs;
  const double flops = 2.0 * (double)a.M * K * NB;
  if (tf32) {
    IT_CUDA_TRY(cudaFuncSetAttribute(gemm_tc_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem));
    IT_LAUNCH(IT_K_GEMM_TC, bytes, flops, st, gemm_tc_kernel<true><<<(unsigned)grid, TC_THREADS_TF32, smem, st>>>(m1, m2, mb, mo0, mo1, p));
  } else {
    IT_CUDA_TRY(cudaFuncSetAttribute(gemm_tc_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem));
    IT_LAUNCH(IT_K_GEMM_TC, bytes, flops, st, gemm_tc_kernel<false><<<(unsigned)grid, TC_THREADS_BF16, smem, st>>>(m1, m2, mb, mo0, mo1, p));
  }
  IT_CUDA_TRY(cudaGetLastError());
  return IT_OK;
}

// ----------------------------------------------------------------------------- two products back to back: host side
namespace {
struct Tc2Shape { int kb1, kb2, buf_panels, stages, smem; };

bool tc2_shape(const it_gemm2_args &a, Tc2Shape *out) {
  if (a.M <= 0 || a.M > (int64_t)INT32_MAX) return false;
  const int K2 = a.X2 ? a.K2 : 0;
  if (a.K1 <= 0 || (a.K1 * 2) % 16 != 0 || (K2 * 2) % 16 != 0) return false;
  const int N2 = a.n0 + a.n1;
  if (a.N1 <= 0 || a.N1 % 64 != 0 || a.N1 > 256) return false;           // H is a whole number of k-blocks of the second product
  if (a.n0 % 64 != 0 || a.n1 % 64 != 0 || N2 <= 0 || N2 > 256) return false;   // outputs are whole 128-byte panels
  if (2 * (a.N1 + N2) > 512) return false;                               // two accumulators per product in TMEM
  Tc2Shape s;
  s.kb1 = (a.K1 + 63) / 64; s.kb2 = (K2 + 63) / 64;
  s.buf_panels = (a.N1 > N2 ? a.N1 : N2) / 64;
  const int stage_bytes = TC_BM * TC_KBLOCK_BYTES;
  const int fixed = (s.kb1 + s.kb2) * a.N1 * TC_KBLOCK_BYTES + (a.N1 / 64) * N2 * TC_KBLOCK_BYTES + 2 * s.buf_panels * stage_bytes +
                    kSmemAux + (a.N1 + N2) * 4;
  s.stages = (kSmemBudget - fixed) / stage_bytes;
  if (s.stages < 3) return false;
  if (s.stages > IT_TC_MAX_STAGES) s.stages = IT_TC_MAX_STAGES;
  s.smem = fixed + s.stages * stage_bytes;
  *out = s;
  return true;
}
}  // namespace

bool it_tc2_supported(const it_gemm2_args &a) {
  Tc2Shape s;
  return tc2_shape(a, &s);
}

// B1, B2: bf16 weights prepared by it_launch_prep_weights_tc ([N1, padded K1 + padded K2] and [n0 + n1, N1]).
it_status it_launch_gemm2_tc(const it_gemm2_args &a, const void *B1, const void *B2, int num_sms, int *status, cudaStream_t st) {
  if (a.M == 0) return IT_OK;
  Tc2Shape s;
  IT_REQUIRE(tc2_shape(a, &s), IT_ERR_UNSUPPORTED, "fused tensor-core apply: shape not supported");
  const int K2 = a.X2 ? a.K2 : 0, N2 = a.n0 + a.n1;
  CUtensorMap m1, m2, mb1, mb2;
  IT_TRY(make_map(&m1, a.X1, 2, a.M, a.K1, TC_BM));
  if (a.X2) IT_TRY(make_map(&m2, a.X2, 2, a.M, K2, TC_BM));
  else m2 = m1;
  IT_TRY(make_map(&mb1, B1, 2, a.N1, (int64_t)(s.kb1 + s.kb2) * 64, a.N1));
  IT_TRY(make_map(&mb2, B2, 2, N2, a.N1, N2));
  CUtensorMap mo0 = m1, mo1 = m1;   // placeholders where a segment is empty
  if (a.n0 > 0) IT_TRY(make_map(&mo0, a.out0, 2, a.M, a.n0, TC_BM));
  if (a.n1 > 0) IT_TRY(make_map(&mo1, a.out1, 2, a.M, a.n1, TC_BM));

  Tc2Params p;
  p.M = a.M; p.n_tiles = (int)((a.M + TC_BM - 1) / TC_BM);
  p.kb1 = s.kb1; p.kb2 = s.kb2; p.N1 = a.N1; p.N2 = N2; p.n0 = a.n0; p.n1 = a.n1;
  p.bias1 = a.bias1; p.act1 = a.act1; p.bias0 = a.bias0;
  p.stages = s.stages; p.buf_panels = s.buf_panels; p.status = status;
  p.spin_limit = a.spin_limit ? a.spin_limit : TC_SPIN_LIMIT; p.no_loads = a.no_loads;

  int64_t grid = num_sms;
  if (grid > p.n_tiles) grid = p.n_tiles;
  const int K = a.K1 + K2;
  const double bytes = (double)a.M * 2.0 * (K + N2) + 2.0 * ((double)K * a.N1 + (double)a.N1 * N2);
  const double flops = 2.0 * (double)a.M * ((double)K * a.N1 + (double)a.N1 * N2);
  IT_CUDA_TRY(cudaFuncSetAttribute(gemm2_tc_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, s.smem));
  IT_LAUNCH(IT_K_GEMM2_TC, bytes, flops, st, gemm2_tc_kernel<<<(unsigned)grid, TC_THREADS_BF16, s.smem, st>>>(m1, m2, mb1, mb2, mo0, mo1, p));
  IT_CUDA_TRY(cudaGetLastError());
  return IT_OK;
}

// Test hook for the bounded waits: a 128 x 64 product (bf16, or fp32 with its operand-splitting warps) whose producer issues no copies, with waits that give up
// after a few thousand polls.  Every role runs out of patience, the CTA drains, frees its TMEM and returns, and the
// status word of the graph is set, which the next it_graph_check reports as IT_ERR_TIMEOUT.
extern "C" it_status it_debug_expire_wait(it_graph *g, it_dtype dtype, const void *x, void *out, void *workspace, size_t workspace_bytes,
                                           void *stream) {
  IT_REQUIRE(g != nullptr && x != nullptr && out != nullptr && workspace != nullptr, IT_ERR_INVALID_ARG, "NULL argument");
  IT_REQUIRE(workspace_bytes >= 64 * 1024 && ((uintptr_t)workspace % 256) == 0, IT_ERR_WORKSPACE, "needs 64 KB of aligned workspace");
  it_gemm_args a{};
  IT_REQUIRE(dtype == IT_F32 || dtype == IT_BF16, IT_ERR_INVALID_ARG, "bad dtype");
  a.M = 128; a.x_dtype = dtype; a.X1 = x; a.K1 = 64; a.X2 = nullptr; a.K2 = 0; a.B = nullptr; a.NB = 64;
  a.n0 = 64; a.out0 = out; a.dt0 = dtype; a.bias0 = nullptr; a.act0 = IT_ACT_NONE;
  a.n1 = 0; a.out1 = nullptr; a.dt1 = dtype; a.out2 = nullptr;
  a.spin_limit = 4096; a.no_loads = 1;
  return it_launch_gemm_tc(a, workspace, nullptr, nullptr, 1, 64, nullptr, g->num_sms, g->d_status, (cudaStream_t)stream);
}

// The same hook for the kernel that runs two products back to back (bf16: 128 x 64 times 64 x 64 times 64 x 64).
extern "C" it_status it_debug_expire_wait_fused(it_graph *g, const void *x, void *out, void *workspace, size_t workspace_bytes,
                                                 void *stream) {
  IT_REQUIRE(g != nullptr && x != nullptr && out != nullptr && workspace != nullptr, IT_ERR_INVALID_ARG, "NULL argument");
  IT_REQUIRE(workspace_bytes >= 64 * 1024 && ((uintptr_t)workspace % 256) == 0, IT_ERR_WORKSPACE, "needs 64 KB of aligned workspace");
  it_gemm2_args a{};
  a.M = 128; a.X1 = x; a.K1 = 64; a.X2 = nullptr; a.K2 = 0; a.N1 = 64; a.bias1 = nullptr; a.act1 = IT_ACT_NONE;
  a.n0 = 0; a.out0 = nullptr; a.bias0 = nullptr; a.n1 = 64; a.out1 = out;
  a.spin_limit = 4096; a.no_loads = 1;
  return it_launch_gemm2_tc(a, workspace, (const char *)workspace + 32 * 1024, g->num_sms, g->d_status, (cudaStream_t)stream);
}
