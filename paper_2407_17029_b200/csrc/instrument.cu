// Benchmark instrumentation: a process-wide launch counter and an optional event pair recorded
// around the dominant kernel of the next call.
#include <atomic>

#include "common.cuh"

namespace qb {
namespace {
std::atomic<uint64_t> g_launches{0};
thread_local cudaEvent_t t_start = nullptr;
thread_local cudaEvent_t t_stop = nullptr;
}  // namespace

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
int qblora_set_timing_events(void* start_event, void* stop_event) {
  qb::t_start = static_cast<cudaEvent_t>(start_event);
  qb::t_stop = static_cast<cudaEvent_t>(stop_event);
  return QBLORA_OK;
}
}
