// Host-only entry points of the C ABI: status read-back, version, launch accounting and tracing.
#include <atomic>
#include <mutex>
#include <vector>

#include "common.cuh"

namespace ocs {
namespace {

struct TraceRecord {
  const char* name;
  cudaEvent_t start, stop;
  bool closed = false;   // its stop event has been recorded
};

std::atomic<long long> g_launches{0};
std::mutex g_trace_mutex;
bool g_trace_on = false;
size_t g_trace_cap = 0;
std::vector<TraceRecord> g_records;      // records of the running trace
std::vector<cudaEvent_t> g_event_pool;   // events kept for reuse between traces

cudaEvent_t take_event() {
  if (!g_event_pool.empty()) {
    cudaEvent_t e = g_event_pool.back();
    g_event_pool.pop_back();
    return e;
  }
  cudaEvent_t e = nullptr;
  if (cudaEventCreate(&e) != cudaSuccess) return nullptr;
  return e;
}

}  // namespace

int trace_begin(const char* name, cudaStream_t stream) {
  g_launches.fetch_add(1, std::memory_order_relaxed);
  if (!g_trace_on) return -1;
  std::lock_guard<std::mutex> lock(g_trace_mutex);
  if (!g_trace_on || g_records.size() >= g_trace_cap) return -1;
  TraceRecord r{name, take_event(), take_event()};
  if (!r.start || !r.stop) {
    if (r.start) g_event_pool.push_back(r.start);
    if (r.stop) g_event_pool.push_back(r.stop);
    return -1;
  }
  cudaEventRecord(r.start, stream);
  g_records.push_back(r);
  return (int)g_records.size() - 1;
}

void trace_end(int record, cudaStream_t stream) {
  if (record < 0) return;
  std::lock_guard<std::mutex> lock(g_trace_mutex);
  if (!g_trace_on || (size_t)record >= g_records.size()) return;   // the trace ended, or a new one began, meanwhile
  cudaEventRecord(g_records[record].stop, stream);
  g_records[record].closed = true;
}

}  // namespace ocs

using namespace ocs;

extern "C" const char* ocs_version(void) { return "ocs-b200 0.2 (sm_100a)"; }

extern "C" ocs_status ocs_poll_status(const int* dev_status, void* stream, int* host_out) {
  if (!dev_status || !host_out) return OCS_ERR_INVALID_ARG;
  cudaStream_t s = reinterpret_cast<cudaStream_t>(stream);
  if (cudaMemcpyAsync(host_out, dev_status, sizeof(int), cudaMemcpyDeviceToHost, s) != cudaSuccess) return OCS_ERR_CUDA;
  return cudaStreamSynchronize(s) == cudaSuccess ? OCS_OK : OCS_ERR_CUDA;
}

extern "C" long long ocs_kernel_launches(void) { return g_launches.load(std::memory_order_relaxed); }

extern "C" ocs_status ocs_trace_start(int max_records) {
  if (max_records < 1) return OCS_ERR_INVALID_ARG;
  std::lock_guard<std::mutex> lock(g_trace_mutex);
  for (const TraceRecord& r : g_records) { g_event_pool.push_back(r.start); g_event_pool.push_back(r.stop); }
  g_records.clear();
  g_trace_cap = (size_t)max_records;
  g_trace_on = true;
  return OCS_OK;
}

extern "C" int ocs_trace_stop(ocs_trace_row* rows, int capacity) {
  std::lock_guard<std::mutex> lock(g_trace_mutex);
  g_trace_on = false;
  int n = 0;
  bool failed = false;
  for (const TraceRecord& r : g_records) {
    if (!r.closed) continue;   // its launch had not returned when the trace ended
    float ms = 0.0f;
    if (cudaEventSynchronize(r.stop) != cudaSuccess || cudaEventElapsedTime(&ms, r.start, r.stop) != cudaSuccess)
      failed = true;
    int i = 0;
    while (i < n && strncmp(rows[i].name, r.name, sizeof(rows[i].name) - 1) != 0) ++i;
    if (i == n) {
      if (!rows || n >= capacity) continue;
      memset(&rows[n], 0, sizeof(rows[n]));
      strncpy(rows[n].name, r.name, sizeof(rows[n].name) - 1);
      ++n;
    }
    rows[i].launches += 1;
    rows[i].total_ms += (double)ms;
  }
  for (const TraceRecord& r : g_records) { g_event_pool.push_back(r.start); g_event_pool.push_back(r.stop); }
  g_records.clear();
  return failed ? -1 : n;
}
