// Launch accounting and optional per-kernel device timing (profiling aid of the library; not on the data path).
#include <atomic>
#include <cstdio>
#include <cstring>
#include <map>
#include <mutex>
#include <string>
#include <vector>

#include "common.cuh"

namespace lawcat {
namespace {
struct Rec {
  const char* name;
  cudaEvent_t a, b;
};
std::atomic<unsigned long long> g_launches{0};
std::atomic<bool> g_on{false};
std::mutex g_mu;
std::vector<Rec> g_recs;
}  // namespace

LaunchScope::LaunchScope(const char* name, cudaStream_t s) : stream(s), idx(-1) {
  g_launches.fetch_add(1, std::memory_order_relaxed);
  if (!g_on.load(std::memory_order_relaxed)) return;
  Rec r{name, nullptr, nullptr};
  if (cudaEventCreate(&r.a) != cudaSuccess || cudaEventCreate(&r.b) != cudaSuccess) return;
  cudaEventRecord(r.a, s);
  std::lock_guard<std::mutex> lk(g_mu);
  idx = (int)g_recs.size();
  g_recs.push_back(r);
}

LaunchScope::~LaunchScope() {
  if (idx < 0) return;
  std::lock_guard<std::mutex> lk(g_mu);
  cudaEventRecord(g_recs[idx].b, stream);
}

static thread_local char t_cuda_error[256] = "";

void note_cuda_error(cudaError_t e, const char* file, int line) {
  const char* base = strrchr(file, '/');
  snprintf(t_cuda_error, sizeof(t_cuda_error), "%s (%s) at %s:%d", cudaGetErrorString(e), cudaGetErrorName(e),
           base ? base + 1 : file, line);
}
}  // namespace lawcat

using namespace lawcat;

extern "C" {

unsigned long long lawcat_launch_count(void) { return g_launches.load(); }

const char* lawcat_last_cuda_error(void) { return t_cuda_error; }

int lawcat_trace_begin(void) {
  std::lock_guard<std::mutex> lk(g_mu);
  for (Rec& r : g_recs) {
    cudaEventDestroy(r.a);
    cudaEventDestroy(r.b);
  }
  g_recs.clear();
  g_on.store(true);
  return LAWCAT_OK;
}

int lawcat_trace_end(char* buf, size_t buf_bytes) {
  g_on.store(false);
  std::lock_guard<std::mutex> lk(g_mu);
  std::map<std::string, std::pair<long, double>> agg;
  int status = LAWCAT_OK;
  for (Rec& r : g_recs) {
    float ms = 0.f;
    if (cudaEventSynchronize(r.b) != cudaSuccess || cudaEventElapsedTime(&ms, r.a, r.b) != cudaSuccess)
      status = LAWCAT_ERR_CUDA;
    auto& e = agg[r.name];
    e.first += 1;
    e.second += ms;
    cudaEventDestroy(r.a);
    cudaEventDestroy(r.b);
  }
  g_recs.clear();
  if (buf && buf_bytes) {
    size_t off = 0;
    buf[0] = 0;
    for (auto& kv : agg) {
      char line[256];
      int n = snprintf(line, sizeof line, "%s %ld %.6f\n", kv.first.c_str(), kv.second.first, kv.second.second);
      if (n < 0 || off + (size_t)n + 1 > buf_bytes) break;
      memcpy(buf + off, line, (size_t)n + 1);
      off += (size_t)n;
    }
  }
  return status;
}

}  // extern "C"
