// Launch accounting for the benchmark: a per-kernel-class launch counter (always on) and, when
// enabled, a pair of CUDA events recorded on the launching stream around every launch so that
// the average device time of one kernel class can be read back after a timed region.
#include "common.cuh"

#include <atomic>
#include <mutex>
#include <vector>

namespace templora {
namespace {

std::atomic<int> g_timing_on{0};
std::atomic<long long> g_launches[kKindCount];
std::mutex g_mu;
struct Pair { cudaEvent_t a, b; };
std::vector<Pair> g_pending[kKindCount];
std::vector<Pair> g_free;

}  // namespace

LaunchScope::LaunchScope(int kind, cudaStream_t st) : kind_(kind), st_(st), a_(nullptr), b_(nullptr) {
  g_launches[kind].fetch_add(1, std::memory_order_relaxed);
  if (!((g_timing_on.load(std::memory_order_relaxed) >> kind) & 1)) return;
  std::lock_guard<std::mutex> lk(g_mu);
  Pair p{nullptr, nullptr};
  if (!g_free.empty()) {
    p = g_free.back();
    g_free.pop_back();
  } else if (cudaEventCreate(&p.a) != cudaSuccess || cudaEventCreate(&p.b) != cudaSuccess) {
    return;
  }
  a_ = p.a; b_ = p.b;
  cudaEventRecord(a_, st_);
}

LaunchScope::~LaunchScope() {
  if (!a_) return;
  cudaEventRecord(b_, st_);
  std::lock_guard<std::mutex> lk(g_mu);
  g_pending[kind_].push_back(Pair{a_, b_});
}

}  // namespace templora

using namespace templora;

extern "C" {

void templora_timing_enable(int32_t kind_mask) { g_timing_on.store(kind_mask); }

templora_status_t templora_timing_read(int32_t kind, double *total_ms, int64_t *timed_launches, int64_t *all_launches,
                                       int32_t reset) {
  if (kind < 0 || kind >= kKindCount) return TEMPLORA_ERR_INVALID_ARG;
  double total = 0.0;
  long long n = 0;
  std::lock_guard<std::mutex> lk(g_mu);
  for (const Pair &p : g_pending[kind]) {
    float ms = 0.f;
    if (cudaEventSynchronize(p.b) != cudaSuccess || cudaEventElapsedTime(&ms, p.a, p.b) != cudaSuccess)
      return TEMPLORA_ERR_CUDA;
    total += ms;
    ++n;
  }
  if (total_ms) *total_ms = total;
  if (timed_launches) *timed_launches = n;
  if (all_launches) *all_launches = g_launches[kind].load();
  if (reset) {
    for (const Pair &p : g_pending[kind]) g_free.push_back(p);
    g_pending[kind].clear();
    g_launches[kind].store(0);
  }
  return TEMPLORA_OK;
}

}  // extern "C"
