// Pivotal Token Selection (Sec. 3.3, Eq. 4-5, Algorithm 1 first routine) on sm_100a.
//
//   colsum_chunk_kernel : Eq. 4's sum over tokens, one partial per chunk of 32 tokens, folded into at most
//                         16 group partials per image by the last CTA of each group (fixed order).  Skipped
//                         when the previous restore kernel has already left the partials of its output.
//   score_topk_kernel   : s[b,t] = sum_c (x[b,t,c] - mean[b,c])^2, one warp per token, the mean token
//                         rebuilt from the group partials in shared memory; the last CTA of each image to
//                         finish then runs the exact top-k of that image: radix select on the fp32 bit
//                         patterns (which order like the values for s >= 0), ties to the lowest index,
//                         ascending output, inverse map.
// Few launches and short chains of dependent loads matter more here than peak bandwidth: the maps are
// tens of MB, and every dependent global access costs about a microsecond.  All HBM access is 128-bit
// and coalesced; no float atomics anywhere (bit-reproducible).
#include "colsum_fold.cuh"
#include "internal.h"

namespace fv {

namespace {

constexpr int kTopkThreads = 512;
constexpr int kTopkWarps = kTopkThreads / 32;
// Keys sit in shared memory with one pad word per 32, so that both access patterns of the top-k are
// free of bank conflicts: consecutive lanes on consecutive tokens, and each lane on its own contiguous run.
__device__ __forceinline__ int KI(int i) { return i + (i >> 5); }
constexpr size_t kTopkMaxSmem = ((size_t)kTopkMaxTokens + kTopkMaxTokens / 32 + 1) * 4;

__global__ void __launch_bounds__(256) colsum_chunk_kernel(const float4* __restrict__ x, int n, int C4, int nchunks, int group,
                                                           int ngroups, float4* __restrict__ chunk_partial,
                                                           float4* __restrict__ group_partial, unsigned int* tickets) {
  pdl_trigger();
  pdl_wait();
  const int b = blockIdx.y, chunk = blockIdx.x;
  const int r0 = chunk * kColsumRows;
  const int r1 = min(n, r0 + kColsumRows);
  const float4* base = x + (size_t)b * n * C4;
  for (int c4 = threadIdx.x; c4 < C4; c4 += blockDim.x) {
    float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
    int r = r0;
    for (; r + 8 <= r1; r += 8) {
      float4 v[8];
#pragma unroll
      for (int i = 0; i < 8; ++i) v[i] = __ldg(base + (size_t)(r + i) * C4 + c4);
#pragma unroll
      for (int i = 0; i < 8; ++i) { acc.x += v[i].x; acc.y += v[i].y; acc.z += v[i].z; acc.w += v[i].w; }
    }
    for (; r < r1; ++r) {
      const float4 v = __ldg(base + (size_t)r * C4 + c4);
      acc.x += v.x; acc.y += v.y; acc.z += v.z; acc.w += v.w;
    }
    chunk_partial[((size_t)b * nchunks + chunk) * C4 + c4] = acc;
  }
  fold_group_partials(b, chunk, nchunks, group, ngroups, C4, chunk_partial, group_partial, tickets);
}

// Exclusive prefix sum of one value per thread over the whole CTA (kTopkThreads threads); returns the
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
  uint32_t wv = lane < kTopkWarps ? s_warp[lane] : 0u;
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

// grid (CTAs per image, B), 512 threads, sized to be resident all at once (two CTAs per SM); the warps of
// an image stride over its token rows.  Dynamic shared memory max(C, n + n/32) * 4 bytes (mean token, then keys).
__global__ void __launch_bounds__(kTopkThreads, 2) score_topk_kernel(const float4* __restrict__ x,
                                                                  const float4* __restrict__ group_partial, int ngroups, int n,
                                                                  int C4, int k, float* __restrict__ score,
                                                                  unsigned int* img_tickets, int32_t* __restrict__ idx,
                                                                  int32_t* __restrict__ inv, int32_t* __restrict__ near_tie) {
  extern __shared__ float4 s_dyn[];
  float4* s_mean = s_dyn;
  uint32_t* s_keys = reinterpret_cast<uint32_t*>(s_dyn);  // reused once the scores are out
  __shared__ uint32_t s_hist[256];
  __shared__ uint32_t s_warp[32];
  __shared__ uint32_t s_prefix, s_remaining, s_near;
  __shared__ int s_last;
  const int b = blockIdx.y, tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  pdl_trigger();
  pdl_wait();

  // ---- Eq. 4: the mean token of image b from the group partials (fixed order)
  {
    const float4* gp = group_partial + (size_t)b * ngroups * C4;
    const float fn = (float)n;
    for (int c4 = tid; c4 < C4; c4 += kTopkThreads) {
      float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
      for (int g = 0; g < ngroups; ++g) {
        const float4 v = __ldcg(gp + (size_t)g * C4 + c4);
        acc.x += v.x; acc.y += v.y; acc.z += v.z; acc.w += v.w;
      }
      s_mean[c4] = make_float4(acc.x / fn, acc.y / fn, acc.z / fn, acc.w / fn);
    }
  }
  __syncthreads();

  // ---- Eq. 5 / Algorithm 1: squared deviation from the mean, one warp per token row
  for (int r = blockIdx.x * kTopkWarps + warp; r < n; r += gridDim.x * kTopkWarps) {
    const float4* row = x + ((size_t)b * n + r) * C4;
    float acc = 0.f;
    int c4 = lane;
    for (; c4 + 32 * 7 < C4; c4 += 32 * 8) {
      float4 v[8];
#pragma unroll
      for (int i = 0; i < 8; ++i) v[i] = __ldg(row + c4 + 32 * i);
#pragma unroll
      for (int i = 0; i < 8; ++i) {
        const float4 m = s_mean[c4 + 32 * i];
        const float dx = v[i].x - m.x, dy = v[i].y - m.y, dz = v[i].z - m.z, dw = v[i].w - m.w;
        acc += dx * dx; acc += dy * dy; acc += dz * dz; acc += dw * dw;
      }
    }
    for (; c4 < C4; c4 += 32) {
      const float4 v = __ldg(row + c4);
      const float4 m = s_mean[c4];
      const float dx = v.x - m.x, dy = v.y - m.y, dz = v.z - m.z, dw = v.w - m.w;
      acc += dx * dx; acc += dy * dy; acc += dz * dz; acc += dw * dw;
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, o);
    if (lane == 0) score[(size_t)b * n + r] = acc;
  }
  __threadfence();  // this thread's scores are visible device-wide before the CTA takes its ticket

  // ---- the last CTA of this image to get here ranks the image
  __syncthreads();
  if (tid == 0) {
    const unsigned int prev = atomicAdd(img_tickets + b, 1u);
    s_last = (prev == gridDim.x - 1);
    if (s_last) img_tickets[b] = 0u;
    s_prefix = 0u; s_remaining = (uint32_t)k; s_near = 0u;
  }
  __syncthreads();
  if (!s_last) return;
  __threadfence();

  // Keys = fp32 bit patterns of the scores (s >= 0, so they order like the values) taken relative to the
  // smallest key of the image: the scores of one map share their leading bits, and ranking only the
  // bits that differ both skips passes and spreads the keys over the histogram bins.
  const float* sc = score + (size_t)b * n;
  uint32_t kmin = 0xFFFFFFFFu, kmax = 0u;
  for (int i = tid; i < n; i += kTopkThreads) {
    const uint32_t key = __float_as_uint(__ldcg(sc + i)) & 0x7FFFFFFFu;  // drops the sign of -0
    s_keys[KI(i)] = key;
    kmin = min(kmin, key); kmax = max(kmax, key);
  }
  kmin = __reduce_min_sync(0xffffffffu, kmin);
  kmax = __reduce_max_sync(0xffffffffu, kmax);
  if (lane == 0) { s_warp[warp] = kmin; s_hist[warp] = kmax; }
  __syncthreads();
  kmin = s_warp[lane < kTopkWarps ? lane : 0];
  kmax = s_hist[lane < kTopkWarps ? lane : 0];
  kmin = __reduce_min_sync(0xffffffffu, kmin);
  kmax = __reduce_max_sync(0xffffffffu, kmax);
  __syncthreads();
  for (int i = tid; i < n; i += kTopkThreads) s_keys[KI(i)] -= kmin;  // each thread rewrites its own keys
  const uint32_t range = kmax - kmin;
  const int npass = range ? (32 - __clz(range) + 7) / 8 : 0;

  // Radix select, most significant byte first: after the passes s_prefix is the k-th largest key and
  // s_remaining how many keys equal to it belong to the kept set.
  for (int pass = 0; pass < npass; ++pass) {
    const int shift = 8 * (npass - 1 - pass);
    const uint32_t hi_mask = shift + 8 >= 32 ? 0u : (0xFFFFFFFFu << (shift + 8));
    if (tid < 256) s_hist[tid] = 0u;
    __syncthreads();
    const uint32_t prefix = s_prefix;
    for (int i = tid; i < n; i += kTopkThreads) {
      const uint32_t key = s_keys[KI(i)];
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
  const uint32_t tau = s_prefix;  // relative to kmin
  const uint32_t need_eq = s_remaining;

  // Ordered compaction: thread t owns the contiguous tokens [t*per, (t+1)*per).
  const int per = (n + kTopkThreads - 1) / kTopkThreads;
  const int i0 = min(n, tid * per), i1 = min(n, i0 + per);
  // one scan for both counts a thread needs: keys above the threshold (low half) and keys equal to it (high
  // half) among the tokens before its own; n <= 49152 keeps either total below 2^16
  uint32_t cnt = 0;
  for (int i = i0; i < i1; ++i) {
    const uint32_t key = s_keys[KI(i)];
    cnt += (key > tau) + ((uint32_t)(key == tau) << 16);
  }
  uint32_t tot;
  const uint32_t before = block_exclusive_scan(cnt, s_warp, &tot);
  const uint32_t eq_before = before >> 16;
  uint32_t pos = (before & 0xFFFFu) + min(eq_before, need_eq);   // kept tokens before this thread's first
  uint32_t e;
  e = eq_before;
  const float tau_f = __uint_as_float(tau + kmin);
  const float band = 1e-5f * tau_f;
  uint32_t near = 0;
  for (int i = i0; i < i1; ++i) {
    uint32_t key = s_keys[KI(i)];
    bool take = key > tau;
    if (key == tau) { take = (e < need_eq); ++e; }
    if (take) idx[(size_t)b * k + pos] = i;
    if (inv) inv[(size_t)b * n + i] = take ? (int32_t)pos : -1;
    pos += take;
    near += (fabsf(__uint_as_float(key + kmin) - tau_f) <= band);
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
  pdl_trigger();
  pdl_wait();
  size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (i < total) inv[i] = -1;
}
__global__ void inv_scatter_kernel(const int32_t* __restrict__ idx, int B, int k, int n, int32_t* __restrict__ inv) {
  pdl_trigger();
  pdl_wait();
  int i = blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= B * k) return;
  int b = i / k, j = i - b * k;
  int t = idx[i];
  if (t >= 0 && t < n) inv[(size_t)b * n + t] = j;
}

}  // namespace

size_t select_ticket_bytes(int B) { return align_up((size_t)B * (kMaxGroups + 1) * sizeof(unsigned int), 256); }

static void chunking(int n, int* nchunks, int* group, int* ngroups) {
  *nchunks = (n + kColsumRows - 1) / kColsumRows;
  *group = (*nchunks + kMaxGroups - 1) / kMaxGroups;
  *ngroups = (*nchunks + *group - 1) / *group;
}

size_t select_workspace_bytes(int B, int n, int C) {
  int nchunks, group, ngroups;
  chunking(n, &nchunks, &group, &ngroups);
  size_t bytes = select_ticket_bytes(B);
  bytes += align_up((size_t)B * nchunks * C * sizeof(float), 256);  // chunk partials of the column sums
  bytes += align_up((size_t)B * ngroups * C * sizeof(float), 256);  // group partials
  bytes += align_up((size_t)B * n * sizeof(float), 256);            // scores
  return bytes;
}

SelectWs select_ws_carve(void* workspace, int B, int n, int C) {
  SelectWs w;
  chunking(n, &w.nchunks, &w.group, &w.ngroups);
  char* p = static_cast<char*>(workspace);
  w.tickets = reinterpret_cast<unsigned int*>(p);
  p += select_ticket_bytes(B);
  w.chunk_partial = reinterpret_cast<float*>(p);
  p += align_up((size_t)B * w.nchunks * C * sizeof(float), 256);
  w.group_partial = reinterpret_cast<float*>(p);
  p += align_up((size_t)B * w.ngroups * C * sizeof(float), 256);
  w.score = reinterpret_cast<float*>(p);
  return w;
}

static int g_num_sms = 148;

cudaError_t select_init() {
  int dev = 0;
  cudaError_t e = cudaGetDevice(&dev);
  if (e == cudaSuccess) e = cudaDeviceGetAttribute(&g_num_sms, cudaDevAttrMultiProcessorCount, dev);
  if (e != cudaSuccess) return e;
  return cudaFuncSetAttribute(score_topk_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kTopkMaxSmem);
}

cudaError_t launch_select(const float* x, int B, int n, int C, int k, int32_t* idx, int32_t* inv, float* score,
                          int32_t* near_tie, void* workspace, bool have_partials, cudaStream_t st) {
  const int C4 = C / 4;
  const SelectWs w = select_ws_carve(workspace, B, n, C);
  float* sc = score ? score : w.score;
  const double sel_bytes = (double)B * n * C * 4.0 + 4.0 * B * n + 4.0 * B * ((double)k + n);
  // the stand-alone column-sum pass reads the map a second time
  LaunchScope scope(KC_SELECT, have_partials ? 1 : 2, sel_bytes, sel_bytes + (have_partials ? 0.0 : (double)B * n * C * 4.0), st);
  if (!have_partials)
    launch_pdl(colsum_chunk_kernel, dim3(w.nchunks, B), dim3(256), 0, st, reinterpret_cast<const float4*>(x), n, C4, w.nchunks, w.group,
               w.ngroups, reinterpret_cast<float4*>(w.chunk_partial), reinterpret_cast<float4*>(w.group_partial), w.tickets);
  const size_t keys_smem = ((size_t)n + n / 32 + 1) * 4;
  const size_t smem = keys_smem > (size_t)C * 4 ? keys_smem : (size_t)C * 4;
  // all CTAs resident at once: two per SM over the B images, never more than one warp per token row
  int per_image = (2 * g_num_sms + B - 1) / B;
  const int need = (n + kTopkWarps - 1) / kTopkWarps;
  if (per_image > need) per_image = need;
  if (per_image < 1) per_image = 1;
  launch_pdl(score_topk_kernel, dim3(per_image, B), dim3(kTopkThreads), smem, st, reinterpret_cast<const float4*>(x),
             reinterpret_cast<const float4*>(w.group_partial), w.ngroups, n, C4, k, sc, w.tickets + (size_t)B * kMaxGroups, idx, inv,
             near_tie);
  return cudaGetLastError();
}

cudaError_t launch_inv_fill(int B, int n, int32_t* inv, cudaStream_t st) {
  const size_t total = (size_t)B * n;
  LaunchScope scope(KC_SELECT, 1, 4.0 * total, 4.0 * total, st);
  return launch_pdl(inv_fill_kernel, dim3((unsigned)((total + 255) / 256)), dim3(256), 0, st, inv, total);
}

cudaError_t launch_inv_from_idx(const int32_t* idx, int B, int k, int n, int32_t* inv, cudaStream_t st) {
  const size_t total = (size_t)B * n;
  LaunchScope scope(KC_SELECT, 2, 4.0 * B * ((double)k + n), 4.0 * B * ((double)k + n), st);
  launch_pdl(inv_fill_kernel, dim3((unsigned)((total + 255) / 256)), dim3(256), 0, st, inv, total);
  launch_pdl(inv_scatter_kernel, dim3((B * k + 255) / 256), dim3(256), 0, st, idx, B, k, n, inv);
  return cudaGetLastError();
}

}  // namespace fv
