// Optional per-kernel instrumentation: CUDA events around every kernel this library launches,
// on the stream the kernel is launched on, plus the algorithmic bytes / flops of each launch.
// Off by default (then a launch only bumps a counter).
#include <mutex>
#include <string.h>
#include <vector>

#include "common.cuh"

namespace {
struct Slot { int kid; cudaEvent_t a, b; double bytes, flops; };
std::mutex g_mu;
bool g_on = false;
std::vector<Slot> g_slots;       // slots in use since it_profile_begin
std::vector<Slot> g_pool;        // recycled event pairs
int64_t g_launches = 0;
const char *const kNames[IT_K_COUNT] = {"validate", "split_scan", "split_fill", "bucket_scan", "prep_weights",
                                        "gather_cta", "gather_flat", "gather_empty", "combine", "gemm_fp32",
                                        "gemm_tc", "gat_cta", "gat_flat", "gat_empty", "edge_messages", "aggregate_finish",
                                        "gemm2_tc"};
}  // namespace

it_prof_scope::it_prof_scope(int kid, double bytes, double flops, cudaStream_t st) : slot_(-1), st_(st) {
  std::lock_guard<std::mutex> lk(g_mu);
  ++g_launches;
  if (!g_on) return;
  Slot s;
  if (!g_pool.empty()) { s = g_pool.back(); g_pool.pop_back(); }
  else if (cudaEventCreate(&s.a) != cudaSuccess || cudaEventCreate(&s.b) != cudaSuccess) return;
  s.kid = kid; s.bytes = bytes; s.flops = flops;
  cudaEventRecord(s.a, st);
  g_slots.push_back(s);
  slot_ = (int)g_slots.size() - 1;
}

it_prof_scope::~it_prof_scope() {
  if (slot_ < 0) return;
  std::lock_guard<std::mutex> lk(g_mu);
  if (slot_ < (int)g_slots.size()) cudaEventRecord(g_slots[slot_].b, st_);
}

bool it_profile_is_on() {
  std::lock_guard<std::mutex> lk(g_mu);
  return g_on;
}

extern "C" int64_t it_kernel_launch_count(void) {
  std::lock_guard<std::mutex> lk(g_mu);
  return g_launches;
}

extern "C" it_status it_profile_begin(void) {
  std::lock_guard<std::mutex> lk(g_mu);
  for (auto &s : g_slots) g_pool.push_back(s);
  g_slots.clear();
  g_on = true;
  return IT_OK;
}

extern "C" it_status it_profile_end(it_kernel_stat *stats, int32_t capacity, int32_t *n_stats) {
  std::lock_guard<std::mutex> lk(g_mu);
  g_on = false;
  it_kernel_stat acc[IT_K_COUNT];
  memset(acc, 0, sizeof(acc));
  it_status rc = IT_OK;
  for (auto &s : g_slots) {
    float ms = 0.f;
    if (cudaEventSynchronize(s.b) != cudaSuccess || cudaEventElapsedTime(&ms, s.a, s.b) != cudaSuccess) {
      it_set_error("profile: reading an event failed");
      rc = IT_ERR_CUDA;
      ms = 0.f;
    }
    acc[s.kid].launches += 1;
    acc[s.kid].total_ms += ms;
    acc[s.kid].algo_bytes += s.bytes;
    acc[s.kid].algo_flops += s.flops;
    g_pool.push_back(s);
  }
  g_slots.clear();
  int32_t n = 0;
  for (int k = 0; k < IT_K_COUNT; ++k) {
    if (acc[k].launches == 0) continue;
    if (stats && n < capacity) {
      stats[n] = acc[k];
      strncpy(stats[n].name, kNames[k], sizeof(stats[n].name) - 1);
    }
    ++n;
  }
  if (n_stats) *n_stats = n;
  return rc;
}
