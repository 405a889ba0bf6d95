// Benchmark instrumentation: a process-wide launch counter and an optional event pair recorded
// around the dominant kernel of the next call.
#include <atomic>

#include "common.cuh"

namespace qb {
namespace {
std::atomic<uint64_t> g_launches{0};
thread_local cudaEvent_t t_start = nullptr;
thread_local cudaEvent_t t_stop = nullptr;
std::atomic<long long> g_wait_limit{0};   // 0 = default
std::atomic<int> g_drop_load{-1};
std::atomic<long long> g_hold_producer{0};
}  // namespace

long long wait_limit_cycles() {
  const long long v = g_wait_limit.load(std::memory_order_relaxed);
  return v > 0 ? v : kDefaultWaitLimitCycles;
}
int take_dropped_load() { return g_drop_load.exchange(-1, std::memory_order_relaxed); }
long long take_producer_hold() { return g_hold_producer.exchange(0, std::memory_order_relaxed); }

void count_launch(int n) { g_launches.fetch_add((uint64_t)n, std::memory_order_relaxed); }

DominantKernelTimer::DominantKernelTimer(cudaStream_t s) : st(s), stop(t_stop) {
  if (t_start) cudaEventRecord(t_start, st);
  t_start = nullptr;
  t_stop = nullptr;
}
DominantKernelTimer::~DominantKernelTimer() {
  if (stop) cudaEventRecord(stop, st);
}
}  // namespace qb

extern "C" {
uint64_t qblora_kernel_launches(void) { return qb::g_launches.load(std::memory_order_relaxed); }
int qblora_debug_set_wait_limit(int64_t cycles) {
  if (cycles < 0) return QBLORA_ERR_INVALID_ARG;
  qb::g_wait_limit.store((long long)cycles, std::memory_order_relaxed);
  return QBLORA_OK;
}
int qblora_debug_drop_load(int32_t iteration) {
  qb::g_drop_load.store(iteration < 0 ? -1 : (int)iteration, std::memory_order_relaxed);
  return QBLORA_OK;
}
int qblora_debug_hold_producer(int64_t cycles) {
  if (cycles < 0 || cycles > 100000000) return QBLORA_ERR_INVALID_ARG;
  qb::g_hold_producer.store((long long)cycles, std::memory_order_relaxed);
  return QBLORA_OK;
}
int qblora_set_timing_events(void* start_event, void* stop_event) {
  qb::t_start = static_cast<cudaEvent_t>(start_event);
  qb::t_stop = static_cast<cudaEvent_t>(stop_event);
  return QBLORA_OK;
}
}
