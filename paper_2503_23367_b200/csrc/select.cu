// Pivotal Token Selection (Sec. 3.3, Eq. 4-5, Algorithm 1 first routine) on sm_100a.
//
//   colsum_partial -> mean_finalize : Eq. 4, the per-image mean token (deterministic two-stage sum)
//   score_rows                      : s[b,t] = sum_c (x[b,t,c] - mean[b,c])^2   (one warp per token)
//   topk_select                     : exact k largest per image, ties to the lowest index, ascending
//                                     output, inverse map (one CTA per image, radix select on the
//                                     fp32 bit patterns, which order like the values for s >= 0)
// All HBM access is 128-bit and coalesced; no float atomics anywhere (bit-reproducible).
#include "internal.h"

namespace fv {

namespace {

constexpr int kScoreRowsPerCta = 32;
constexpr int kTopkThreads = 1024;

__global__ void __launch_bounds__(512) colsum_partial_kernel(const float4* __restrict__ x, int n, int C4, int nchunks,
                                                             float4* __restrict__ partial) {
  const int b = blockIdx.y, chunk = blockIdx.x;
  const int r0 = chunk * kColsumRows;
  const int r1 = min(n, r0 + kColsumRows);
  const float4* base = x + (size_t)b * n * C4;
  for (int c4 = threadIdx.x; c4 < C4; c4 += blockDim.x) {
    float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
    int r = r0;
    for (; r + 4 <= r1; r += 4) {
      float4 v0 = __ldg(base + (size_t)(r + 0) * C4 + c4);
      float4 v1 = __ldg(base + (size_t)(r + 1) * C4 + c4);
      float4 v2 = __ldg(base + (size_t)(r + 2) * C4 + c4);
      float4 v3 = __ldg(base + (size_t)(r + 3) * C4 + c4);
      acc.x += v0.x; acc.y += v0.y; acc.z += v0.z; acc.w += v0.w;
      acc.x += v1.x; acc.y += v1.y; acc.z += v1.z; acc.w += v1.w;
      acc.x += v2.x; acc.y += v2.y; acc.z += v2.z; acc.w += v2.w;
      acc.x += v3.x; acc.y += v3.y; acc.z += v3.z; acc.w += v3.w;
    }
    for (; r < r1; ++r) {
      float4 v = __ldg(base + (size_t)r * C4 + c4);
      acc.x += v.x; acc.y += v.y; acc.z += v.z; acc.w += v.w;
    }
    partial[((size_t)b * nchunks + chunk) * C4 + c4] = acc;
  }
}

__global__ void mean_finalize_kernel(const float* __restrict__ partial, int nchunks, int C, int n, float* __restrict__ mean) {
  const int b = blockIdx.y;
  const int c = blockIdx.x * blockDim.x + threadIdx.x;
  if (c >= C) return;
  const float* p = partial + (size_t)b * nchunks * C + c;
  float acc = 0.f;
  for (int i = 0; i < nchunks; ++i) acc += p[(size_t)i * C];
  mean[(size_t)b * C + c] = acc / (float)n;
}

__global__ void __launch_bounds__(256) score_rows_kernel(const float4* __restrict__ x, const float4* __restrict__ mean, int n,
                                                         int C4, float* __restrict__ score) {
  extern __shared__ float4 s_mean[];
  const int b = blockIdx.y;
  for (int i = threadIdx.x; i < C4; i += blockDim.x) s_mean[i] = mean[(size_t)b * C4 + i];
  __syncthreads();
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int r0 = blockIdx.x * kScoreRowsPerCta;
  for (int rr = warp; rr < kScoreRowsPerCta; rr += 8) {
    const int r = r0 + rr;
    if (r >= n) break;
    const float4* row = x + ((size_t)b * n + r) * C4;
    float acc = 0.f;
    for (int c4 = lane; c4 < C4; c4 += 32) {
      float4 v = __ldg(row + c4);
      float4 m = s_mean[c4];
      float dx = v.x - m.x, dy = v.y - m.y, dz = v.z - m.z, dw = v.w - m.w;
      acc += dx * dx; acc += dy * dy; acc += dz * dz; acc += dw * dw;
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, o);
    if (lane == 0) score[(size_t)b * n + r] = acc;
  }
}

// Exclusive prefix sum of one value per thread over the whole CTA (1024 threads); returns the
// exclusive prefix and, through `total`, the CTA-wide sum.  s_warp is 32 words of scratch.
__device__ __forceinline__ uint32_t block_exclusive_scan(uint32_t v, uint32_t* s_warp, uint32_t* total) {
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  uint32_t inc = v;
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    uint32_t t = __shfl_up_sync(0xffffffffu, inc, o);
    if (lane >= o) inc += t;
  }
  __syncthreads();  // s_warp may still be read from a previous scan
  if (lane == 31) s_warp[warp] = inc;
  __syncthreads();
  uint32_t wv = s_warp[lane];  // blockDim.x == 1024 -> 32 warps
  uint32_t winc = wv;
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    uint32_t t = __shfl_up_sync(0xffffffffu, winc, o);
    if (lane >= o) winc += t;
  }
  uint32_t warp_excl = __shfl_sync(0xffffffffu, winc - wv, warp);
  *total = __shfl_sync(0xffffffffu, winc, 31);
  return warp_excl + inc - v;
}

__global__ void __launch_bounds__(kTopkThreads) topk_select_kernel(const float* __restrict__ score, int n, int k,
                                                                   int32_t* __restrict__ idx, int32_t* __restrict__ inv,
                                                                   int32_t* __restrict__ near_tie) {
  extern __shared__ uint32_t s_keys[];  // n keys
  __shared__ uint32_t s_hist[256];
  __shared__ uint32_t s_warp[32];
  __shared__ uint32_t s_prefix, s_remaining, s_near;
  const int b = blockIdx.x, tid = threadIdx.x, lane = tid & 31;
  const float* sc = score + (size_t)b * n;
  for (int i = tid; i < n; i += kTopkThreads) s_keys[i] = __float_as_uint(sc[i]) & 0x7FFFFFFFu;  // s >= 0; drops the sign of -0
  if (tid == 0) { s_prefix = 0u; s_remaining = (uint32_t)k; s_near = 0u; }
  __syncthreads();

  // Radix select, most significant byte first: after 4 passes s_prefix is the k-th largest key and
  // s_remaining how many keys equal to it belong to the kept set.
  for (int pass = 0; pass < 4; ++pass) {
    const int shift = 24 - 8 * pass;
    const uint32_t hi_mask = pass == 0 ? 0u : (0xFFFFFFFFu << (shift + 8));
    if (tid < 256) s_hist[tid] = 0u;
    __syncthreads();
    const uint32_t prefix = s_prefix;
    for (int i = tid; i < n; i += kTopkThreads) {
      uint32_t key = s_keys[i];
      if ((key & hi_mask) == prefix) atomicAdd(&s_hist[(key >> shift) & 255u], 1u);
    }
    __syncthreads();
    if (tid < 32) {
      // lane l owns bins 255-8l .. 248-8l (descending); find the bin where the running count from the
      // top reaches s_remaining.
      uint32_t local[8], sum = 0;
#pragma unroll
      for (int j = 0; j < 8; ++j) { local[j] = s_hist[255 - 8 * lane - j]; sum += local[j]; }
      uint32_t inc = sum;
#pragma unroll
      for (int o = 1; o < 32; o <<= 1) {
        uint32_t t = __shfl_up_sync(0xffffffffu, inc, o);
        if (lane >= o) inc += t;
      }
      const uint32_t rem = s_remaining;
      const uint32_t excl = inc - sum;
      const bool mine = (excl < rem) && (inc >= rem);  // exactly one lane
      if (mine) {
        uint32_t cum = excl;
#pragma unroll
        for (int j = 0; j < 8; ++j) {
          if (cum + local[j] >= rem) {
            s_prefix = prefix | ((uint32_t)(255 - 8 * lane - j) << shift);
            s_remaining = rem - cum;
            break;
          }
          cum += local[j];
        }
      }
    }
    __syncthreads();
  }
  const uint32_t tau = s_prefix;
  const uint32_t need_eq = s_remaining;

  // Ordered compaction: thread t owns the contiguous tokens [t*per, (t+1)*per).
  const int per = (n + kTopkThreads - 1) / kTopkThreads;
  const int i0 = min(n, tid * per), i1 = min(n, i0 + per);
  uint32_t eq = 0;
  for (int i = i0; i < i1; ++i) eq += (s_keys[i] == tau);
  uint32_t tot;
  uint32_t eq_before = block_exclusive_scan(eq, s_warp, &tot);
  uint32_t kept = 0, e = eq_before;
  for (int i = i0; i < i1; ++i) {
    uint32_t key = s_keys[i];
    if (key > tau) ++kept;
    else if (key == tau) { kept += (e < need_eq); ++e; }
  }
  uint32_t pos = block_exclusive_scan(kept, s_warp, &tot);
  e = eq_before;
  const float tau_f = __uint_as_float(tau);
  const float band = 1e-5f * tau_f;
  uint32_t near = 0;
  for (int i = i0; i < i1; ++i) {
    uint32_t key = s_keys[i];
    bool take = key > tau;
    if (key == tau) { take = (e < need_eq); ++e; }
    if (take) idx[(size_t)b * k + pos] = i;
    if (inv) inv[(size_t)b * n + i] = take ? (int32_t)pos : -1;
    pos += take;
    near += (fabsf(__uint_as_float(key) - tau_f) <= band);
  }
  if (near_tie) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) near += __shfl_xor_sync(0xffffffffu, near, o);
    if (lane == 0) atomicAdd(&s_near, near);
    __syncthreads();
    if (tid == 0) near_tie[b] = (int32_t)s_near;
  }
}

__global__ void inv_fill_kernel(int32_t* inv, size_t total) {
  size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (i < total) inv[i] = -1;
}
__global__ void inv_scatter_kernel(const int32_t* __restrict__ idx, int B, int k, int n, int32_t* __restrict__ inv) {
  int i = blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= B * k) return;
  int b = i / k, j = i - b * k;
  int t = idx[i];
  if (t >= 0 && t < n) inv[(size_t)b * n + t] = j;
}

}  // namespace

size_t select_workspace_bytes(int B, int n, int C) {
  const size_t nchunks = (n + kColsumRows - 1) / kColsumRows;
  size_t bytes = align_up((size_t)B * nchunks * C * sizeof(float), 256);  // partial column sums
  bytes += align_up((size_t)B * C * sizeof(float), 256);                   // mean token
  bytes += align_up((size_t)B * n * sizeof(float), 256);                   // scores
  return bytes;
}

cudaError_t select_init() {
  return cudaFuncSetAttribute(topk_select_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kTopkMaxTokens * 4);
}

cudaError_t launch_select(const float* x, int B, int n, int C, int k, int32_t* idx, int32_t* inv, float* score,
                          int32_t* near_tie, void* workspace, cudaStream_t st) {
  const int nchunks = (n + kColsumRows - 1) / kColsumRows;
  const int C4 = C / 4;
  char* ws = static_cast<char*>(workspace);
  float* partial = reinterpret_cast<float*>(ws);
  ws += align_up((size_t)B * nchunks * C * sizeof(float), 256);
  float* mean = reinterpret_cast<float*>(ws);
  ws += align_up((size_t)B * C * sizeof(float), 256);
  float* sc = score ? score : reinterpret_cast<float*>(ws);
  LaunchScope scope(KC_SELECT, 4, (double)B * n * C * 4.0 + 4.0 * B * n + 4.0 * B * ((double)k + n), st);
  const int cs_threads = C4 >= 512 ? 512 : ((C4 + 31) / 32 * 32);
  colsum_partial_kernel<<<dim3(nchunks, B), cs_threads, 0, st>>>(reinterpret_cast<const float4*>(x), n, C4, nchunks,
                                                                 reinterpret_cast<float4*>(partial));
  mean_finalize_kernel<<<dim3((C + 255) / 256, B), 256, 0, st>>>(partial, nchunks, C, n, mean);
  score_rows_kernel<<<dim3((n + kScoreRowsPerCta - 1) / kScoreRowsPerCta, B), 256, C * sizeof(float), st>>>(
      reinterpret_cast<const float4*>(x), reinterpret_cast<const float4*>(mean), n, C4, sc);
  topk_select_kernel<<<B, kTopkThreads, (size_t)n * 4, st>>>(sc, n, k, idx, inv, near_tie);
  return cudaGetLastError();
}

cudaError_t launch_inv_from_idx(const int32_t* idx, int B, int k, int n, int32_t* inv, cudaStream_t st) {
  const size_t total = (size_t)B * n;
  LaunchScope scope(KC_SELECT, 2, 4.0 * B * ((double)k + n), st);
  inv_fill_kernel<<<(unsigned)((total + 255) / 256), 256, 0, st>>>(inv, total);
  inv_scatter_kernel<<<(B * k + 255) / 256, 256, 0, st>>>(idx, B, k, n, inv);
  return cudaGetLastError();
}

}  // namespace fv
