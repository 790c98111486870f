// fv_prune_select_static: Pivotal Token Selection for callers that cannot hand the library a scratch
// buffer because they cannot allocate one -- e.g. a serving loop whose device memory was carved up
// once at start-up (every byte belongs to a pool with a fixed budget), or a host plug-in that is not
// allowed to call the CUDA allocator, whose implicit device synchronisation would stall its pipeline.
// The selection kernels need scratch beyond their inputs and outputs (arrival counters, partial column
// sums, the scores); here that scratch is a fixed array that lives in the library's own device image.
//
// The array below exists once per GPU that loads this library and stays resident until the process
// exits.  In HOST code its name is only a handle (not a device address): the device address is
// obtained with cudaGetSymbolAddress, once per device, with that device current, and that pointer
// is what the kernels receive.
#include <cuda_runtime.h>

#include <mutex>

#include "internal.h"

namespace {

constexpr size_t kStaticScratchBytes = size_t(8) << 20;  // 8 MiB per GPU, resident until exit
constexpr int kMaxDevices = 64;

static __device__ __align__(256) unsigned char g_select_scratch[kStaticScratchBytes];

std::mutex g_mu;
void* g_scratch_ptr[kMaxDevices] = {nullptr};

// Device address of the scratch array on the CURRENT device (resolved on first use per device).
cudaError_t scratch_address(void** out) {
  int dev = -1;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return e;
  if (dev < 0 || dev >= kMaxDevices) return cudaErrorInvalidDevice;
  std::lock_guard<std::mutex> lk(g_mu);
  if (!g_scratch_ptr[dev]) {
    void* p = nullptr;
    e = cudaGetSymbolAddress(&p, g_select_scratch);
    if (e != cudaSuccess) return e;
    if (!p) return cudaErrorInvalidSymbol;
    g_scratch_ptr[dev] = p;
  }
  *out = g_scratch_ptr[dev];
  return cudaSuccess;
}

}  // namespace

extern "C" {

size_t fv_prune_select_static_capacity(void) { return kStaticScratchBytes; }

fv_status fv_prune_select_static(const float* x_dev, int32_t B, int32_t h, int32_t w, int32_t C, double keep_ratio,
                                 int32_t* idx_out_dev, int32_t* inv_out_dev, float* score_out_dev, int32_t* near_tie_dev,
                                 int32_t* k_out_host, void* stream) {
  if (!x_dev || !idx_out_dev || B <= 0 || h <= 0 || w <= 0 || C <= 0) return FV_ERR_INVALID_ARG;
  if (!(keep_ratio > 0.0) || keep_ratio > 1.0 || (C % 4) || (reinterpret_cast<uintptr_t>(x_dev) & 15u)) return FV_ERR_INVALID_ARG;
  const long n = (long)h * w;
  if (n > fv::kTopkMaxTokens || C > fv::kTopkMaxTokens) return FV_ERR_UNSUPPORTED;
  // The shape must fit the fixed scratch: this entry point never allocates, so it refuses instead.
  if (fv::select_workspace_bytes(B, (int)n, C) > kStaticScratchBytes) return FV_ERR_CAPACITY;
  if (fv::select_init() != cudaSuccess) return FV_ERR_CUDA;
  void* scratch = nullptr;
  if (scratch_address(&scratch) != cudaSuccess) return FV_ERR_CUDA;
  const int k = fv_k_for(keep_ratio, h, w);
  if (k_out_host) *k_out_host = k;
  // Of the scratch only the arrival counters at its head have to start at zero; they are cleared here on
  // every call (a memset node on the stream, no allocation).  Every other word the kernels read
  // (partial sums, scores) is written earlier in the same call, so the previous call's leftovers are harmless.
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  if (cudaMemsetAsync(scratch, 0, fv::select_ticket_bytes(B), st) != cudaSuccess) return FV_ERR_CUDA;
  cudaError_t e = fv::launch_select(x_dev, B, (int)n, C, k, idx_out_dev, inv_out_dev, score_out_dev, near_tie_dev, scratch,
                                    false, st);
  return e == cudaSuccess ? FV_OK : FV_ERR_CUDA;
}

}  // extern "C"
