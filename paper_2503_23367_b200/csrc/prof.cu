// Launch counting and optional per-kernel-class timing for the benchmark: how many of this library's
// kernels ran, the algorithmic work they were given, and (when enabled) the device time of each class
// measured with CUDA events recorded on the launching stream.
#include <atomic>
#include <mutex>
#include <vector>

#include "internal.h"

namespace fv {

namespace {
std::mutex g_mu;
bool g_timing = false;
uint64_t g_launches[KC_COUNT] = {0};
double g_work[KC_COUNT] = {0};
double g_dram[KC_COUNT] = {0};
struct Pair { cudaEvent_t a, b; int cls; };
std::vector<Pair> g_pairs;       // recorded since the last read
std::vector<Pair> g_free;        // reusable events
}  // namespace

LaunchScope::LaunchScope(KernelClass c, int kernels, double work, double dram_bytes, cudaStream_t s) : slot(-1), st(s) {
  std::lock_guard<std::mutex> lk(g_mu);
  g_launches[c] += kernels;
  g_work[c] += work;
  g_dram[c] += dram_bytes;
  if (!g_timing) return;
  Pair p;
  if (!g_free.empty()) { p = g_free.back(); g_free.pop_back(); }
  else if (cudaEventCreate(&p.a) != cudaSuccess || cudaEventCreate(&p.b) != cudaSuccess) return;
  p.cls = c;
  cudaEventRecord(p.a, st);
  g_pairs.push_back(p);
  slot = (int)g_pairs.size() - 1;
}

LaunchScope::~LaunchScope() {
  if (slot < 0) return;
  std::lock_guard<std::mutex> lk(g_mu);
  if (slot < (int)g_pairs.size()) cudaEventRecord(g_pairs[slot].b, st);
}

}  // namespace fv

using namespace fv;

extern "C" {

uint64_t fv_kernel_launches(void) {
  std::lock_guard<std::mutex> lk(g_mu);
  uint64_t t = 0;
  for (int i = 0; i < KC_COUNT; ++i) t += g_launches[i];
  return t;
}

fv_status fv_profile_enable(int32_t on) {
  std::lock_guard<std::mutex> lk(g_mu);
  g_timing = on != 0;
  return FV_OK;
}

fv_status fv_profile_read(double* ms_host, uint64_t* launches_host, double* work_host, double* dram_bytes_host) {
  if (cudaDeviceSynchronize() != cudaSuccess) return FV_ERR_CUDA;
  std::lock_guard<std::mutex> lk(g_mu);
  double ms[KC_COUNT] = {0};
  for (const Pair& p : g_pairs) {
    float t = 0.f;
    if (cudaEventElapsedTime(&t, p.a, p.b) == cudaSuccess) ms[p.cls] += t;
    g_free.push_back(p);
  }
  g_pairs.clear();
  for (int i = 0; i < KC_COUNT; ++i) {
    if (ms_host) ms_host[i] = ms[i];
    if (launches_host) launches_host[i] = g_launches[i];
    if (work_host) work_host[i] = g_work[i];
    if (dram_bytes_host) dram_bytes_host[i] = g_dram[i];
    g_launches[i] = 0;
    g_work[i] = 0;
    g_dram[i] = 0;
  }
  return FV_OK;
}

}  // extern "C"
