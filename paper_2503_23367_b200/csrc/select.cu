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
#include <cuda_bf16.h>

#include "colsum_fold.cuh"
#include "internal.h"
#include "sm100.cuh"

namespace fv {

namespace {

constexpr int kSelectThreads = 1024;   // the stand-alone score + top-k kernel: one CTA per SM
constexpr int kSelectWarps = kSelectThreads / 32;
constexpr int kTopkThreads = 512;      // the fused kernel of a scale step (a thread may hold a whole row slice)
constexpr int kTopkWarps = kTopkThreads / 32;
constexpr size_t kTopkMaxSmem = (size_t)kTopkMaxTokens * 4;   // one key per token (consecutive lanes on consecutive tokens)

template <typename XT>
__global__ void __launch_bounds__(256) colsum_chunk_kernel(const XT* __restrict__ x, int n, int C4, int nchunks, int group,
                                                           int ngroups, float4* __restrict__ chunk_partial,
                                                           float4* __restrict__ group_partial, unsigned int* tickets) {
  pdl_trigger();
  pdl_wait();
  const int b = blockIdx.y, chunk = blockIdx.x;
  const int r0 = chunk * kColsumRows;
  const int r1 = min(n, r0 + kColsumRows);
  const XT* base = x + (size_t)b * n * C4 * 4;
  for (int c4 = threadIdx.x; c4 < C4; c4 += blockDim.x) {
    float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
    int r = r0;
    for (; r + 8 <= r1; r += 8) {
      float4 v[8];
#pragma unroll
      for (int i = 0; i < 8; ++i) v[i] = x_load4<true>(base + ((size_t)(r + i) * C4 + c4) * 4);
#pragma unroll
      for (int i = 0; i < 8; ++i) { acc.x += v[i].x; acc.y += v[i].y; acc.z += v[i].z; acc.w += v[i].w; }
    }
    for (; r < r1; ++r) {
      const float4 v = x_load4<true>(base + ((size_t)r * C4 + c4) * 4);
      acc.x += v.x; acc.y += v.y; acc.z += v.z; acc.w += v.w;
    }
    chunk_partial[((size_t)b * nchunks + chunk) * C4 + c4] = acc;
  }
  fold_group_partials(b, chunk, nchunks, group, ngroups, C4, chunk_partial, group_partial, tickets);
}

// Exclusive prefix sum of one value per thread over the whole CTA (T threads, the template argument); returns the
// exclusive prefix and, through `total`, the CTA-wide sum.  s_warp is 32 words of scratch.
template <int T>
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
  uint32_t wv = lane < (T / 32) ? s_warp[lane] : 0u;
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

// ---- Eq. 4: the mean token of image b from up to two sets of at most kMaxGroups partial column sums, added in a
// fixed order (set a, then set b).  The loads are requested eight at a time before the first of them is used.
__device__ __forceinline__ void add_partials(float4& acc, const float4* __restrict__ gp, int ng, int C4, int c4) {
#pragma unroll
  for (int g0 = 0; g0 < kMaxGroups; g0 += 8) {
    if (g0 >= ng) break;
    float4 v[8];
#pragma unroll
    for (int g = 0; g < 8; ++g)
      if (g0 + g < ng) v[g] = __ldcg(gp + (size_t)(g0 + g) * C4 + c4);
#pragma unroll
    for (int g = 0; g < 8; ++g)
      if (g0 + g < ng) { acc.x += v[g].x; acc.y += v[g].y; acc.z += v[g].z; acc.w += v[g].w; }
  }
}
template <int T>
__device__ __forceinline__ void mean_from_partials(float4* s_mean, const float4* __restrict__ gp_a, int nga,
                                                   const float4* __restrict__ gp_b, int ngb, int C4, int n) {
  const float fn = (float)n;
  for (int c4 = threadIdx.x; c4 < C4; c4 += T) {
    float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
    add_partials(acc, gp_a, nga, C4, c4);
    if (ngb > 0) add_partials(acc, gp_b, ngb, C4, c4);
    s_mean[c4] = make_float4(acc.x / fn, acc.y / fn, acc.z / fn, acc.w / fn);
  }
}

// The same sums in the same order by twice as many threads: the upper half of the CTA fetches the partials of the
// groups from 8 on into shared memory while the lower half adds the first 8; the lower half then continues with the
// staged values.  One round trip to L2 instead of two.  stage: 8 * C4 float4 words.
template <int T>
__device__ __forceinline__ void mean_from_partials_halves(float4* s_mean, float4* stage, const float4* __restrict__ gp, int ng, int C4, int n) {
  constexpr int H = T / 2;
  const int tid = threadIdx.x, half = tid / H, t = tid - half * H;
  const float fn = (float)n;
  for (int c0 = 0; c0 < C4; c0 += H) {
    const int c4 = c0 + t;
    float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
    if (c4 < C4) {
      float4 v[8];
      const int g_lo = half * 8;
#pragma unroll
      for (int g = 0; g < 8; ++g)
        if (g_lo + g < ng) v[g] = __ldcg(gp + (size_t)(g_lo + g) * C4 + c4);
      if (half == 0) {
#pragma unroll
        for (int g = 0; g < 8; ++g)
          if (g < ng) { acc.x += v[g].x; acc.y += v[g].y; acc.z += v[g].z; acc.w += v[g].w; }
      } else {
#pragma unroll
        for (int g = 0; g < 8; ++g)
          if (8 + g < ng) stage[(size_t)g * C4 + c4] = v[g];
      }
    }
    __syncthreads();
    if (half == 0 && c4 < C4) {
#pragma unroll
      for (int g = 0; g < 8; ++g)
        if (8 + g < ng) { const float4 u = stage[(size_t)g * C4 + c4]; acc.x += u.x; acc.y += u.y; acc.z += u.z; acc.w += u.w; }
      s_mean[c4] = make_float4(acc.x / fn, acc.y / fn, acc.z / fn, acc.w / fn);
    }
  }
}
static_assert(kMaxGroups == 16, "mean_from_partials_halves splits the groups 8 + 8");

// ---- Eq. 5 / Algorithm 1: squared deviation from the mean, one warp per token row; the warps of an image stride
// over its rows.  NC: the map was not written by this kernel, so its rows may take the read-only path; the fused
// kernel, whose other CTAs have just updated rows of it, reads them through L2.
// BATCH: 16-byte loads a lane requests together (8 with 64 registers per thread, 16 with 128).
// lo / hi: running smallest / largest score key (the bit pattern without its sign) of the rows this warp has scored.
// inv (may be null): the inverse map of the image is set to "not kept" for every row scored here, so that the CTA
// that ranks the image only has to write the entries of the kept rows (one SM stores slowly).
template <int T, bool NC, int BATCH, typename XT>
__device__ __forceinline__ void score_rows(const XT* x, const float4* s_mean, int b, int n, int C4, float* __restrict__ score,
                                           int32_t* __restrict__ inv, uint32_t& lo, uint32_t& hi) {
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  for (int r = blockIdx.x * (T / 32) + warp; r < n; r += gridDim.x * (T / 32)) {
    const XT* row = x + ((size_t)b * n + r) * C4 * 4;
    float acc = 0.f;
    int c4 = lane;
    for (; c4 + 32 * (BATCH - 1) < C4; c4 += 32 * BATCH) {
      float4 v[BATCH];
#pragma unroll
      for (int i = 0; i < BATCH; ++i) v[i] = x_load4<NC>(row + (size_t)(c4 + 32 * i) * 4);
#pragma unroll
      for (int i = 0; i < BATCH; ++i) {
        const float4 m = s_mean[c4 + 32 * i];
        const float dx = v[i].x - m.x, dy = v[i].y - m.y, dz = v[i].z - m.z, dw = v[i].w - m.w;
        acc += dx * dx; acc += dy * dy; acc += dz * dz; acc += dw * dw;
      }
    }
    for (; c4 < C4; c4 += 32) {
      const float4 v = x_load4<NC>(row + (size_t)c4 * 4);
      const float4 m = s_mean[c4];
      const float dx = v.x - m.x, dy = v.y - m.y, dz = v.z - m.z, dw = v.w - m.w;
      acc += dx * dx; acc += dy * dy; acc += dz * dz; acc += dw * dw;
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, o);
    if (lane == 0) {
      score[(size_t)b * n + r] = acc;
      if (inv) inv[(size_t)b * n + r] = -1;
    }
    const uint32_t key = __float_as_uint(acc) & 0x7FFFFFFFu;
    lo = min(lo, key); hi = max(hi, key);
  }
}

// Scratch of the top-k in static shared memory.
constexpr int kFirstDigitBits = 11;                 // the first radix digit: up to 2048 bins
constexpr int kHistBins = 1 << kFirstDigitBits;
constexpr int kCandMax = 1024;                      // longest candidate list kept beside the keys
constexpr int kCountMax = 128;                      // a list this short is finished by counting
struct TopkShared {
  uint32_t hist[kHistBins];      // radix histogram; afterwards the kept / equal counts per 128 tokens of the compaction
  uint32_t cand[2][kCandMax];    // keys that still share the threshold's leading digits
  uint32_t warp[32];
  uint32_t range[64];
  uint32_t prefix, remaining, nbin, near, ncand[2];
};
static_assert(kTopkMaxTokens / 128 <= 512 && kTopkMaxTokens % 4 == 0, "one count per 128 tokens and thread; keys in 16-byte words");

// Smallest and largest score key of the image, gathered while the scores are computed: every CTA folds the keys of
// its rows and adds them to two words per image with integer atomics (order-independent); the words hold ~min and
// max so that zero means "nothing yet", and the CTA that ranks the image zeroes them again.
template <int T>
__device__ __forceinline__ void publish_range(uint32_t lo, uint32_t hi, TopkShared& sh, unsigned int* range_b) {
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  if (lane == 0) { sh.range[warp] = lo; sh.range[32 + warp] = hi; }
  __syncthreads();
  if (threadIdx.x == 0) {
    for (int w = 1; w < (T / 32); ++w) { lo = min(lo, sh.range[w]); hi = max(hi, sh.range[32 + w]); }
    if (lo <= hi) { atomicMax(range_b, ~lo); atomicMax(range_b + 1, hi); }
  }
}

// The bin, counted from the top, in which the running count reaches sh.remaining: its index is added to sh.prefix at
// `shift`, sh.remaining becomes the rank inside the bin and sh.nbin the bin's count.  All threads; ends with a barrier.
template <int T>
__device__ __forceinline__ void threshold_bin(TopkShared& sh, int nbins, int shift) {
  const int tid = threadIdx.x;
  uint32_t local[4], sum = 0;
#pragma unroll
  for (int j = 0; j < 4; ++j) {
    const int bin = nbins - 1 - 4 * tid - j;
    local[j] = bin >= 0 ? sh.hist[bin] : 0u;
    sum += local[j];
  }
  const uint32_t rem = sh.remaining;   // read before the barriers of the scan, rewritten after them
  uint32_t tot;
  const uint32_t excl = block_exclusive_scan<T>(sum, sh.warp, &tot);
  if (excl < rem && excl + sum >= rem) {   // exactly one thread
    uint32_t cum = excl;
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      if (cum + local[j] >= rem) {
        sh.prefix |= (uint32_t)(nbins - 1 - 4 * tid - j) << shift;
        sh.remaining = rem - cum;
        sh.nbin = local[j];
        break;
      }
      cum += local[j];
    }
  }
  __syncthreads();
}

// ---- exact top-k of one image by one CTA (all T threads): radix select on the fp32 bit patterns of the
// scores (s >= 0, so they order like the values), ties to the lowest index, ascending output, inverse map.
// range_b: the image's two range words (see publish_range), complete when this is called.
//   1. one sweep brings the scores from L2 into shared memory as keys relative to the smallest, and counts the first
//      digit -- the top 11 bits of the range the keys really span, so that the counts spread over the bins;
//   2. the keys inside the threshold's bin (a few dozen on a map of distinct scores) are copied to a list, which
//      is finished by counting when it is short and by 8-bit digits otherwise; a bin too full for the list (many
//      equal scores) is refined with 8-bit digits over all keys until it fits;
//   3. ordered compaction: counts per 128 tokens, one scan over them, then every lane knows the output slots of its
//      four tokens.
// One SM does all of this while the others idle, and its instruction issue is what the sweeps wait for: they take
// four keys per lane and 16-byte shared-memory accesses.
template <int T>
__device__ __forceinline__ void topk_image(const float* __restrict__ sc, int n, int k, uint32_t* s_keys, TopkShared& sh,
                                           int32_t* __restrict__ idx_b, int32_t* __restrict__ inv_b, int32_t* near_tie_b,
                                           unsigned int* range_b) {
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const uint32_t kmin = ~__ldcg(range_b), kmax = __ldcg(range_b + 1);
  const uint32_t range = kmax >= kmin ? kmax - kmin : 0u;
  const int bits = range ? 32 - __clz(range) : 0;
  int width = min(bits, kFirstDigitBits);
  int shift = bits - width;
#pragma unroll
  for (int j = 0; j < kHistBins / T; ++j) sh.hist[tid + j * T] = 0u;
  if (tid == 0) { sh.prefix = 0u; sh.remaining = (uint32_t)k; sh.near = 0u; sh.ncand[0] = 0u; sh.ncand[1] = 0u; }
  __syncthreads();
  if (tid == 0) { range_b[0] = 0u; range_b[1] = 0u; }   // every thread has read them

  // ---- 1. scores -> keys, first digit counted on the way.  Up to eight 16-byte loads per thread are requested
  // before the first is used (one CTA fetching them one dependent load at a time took longer than the ranking).
  const int n4 = (n % 4 == 0 && (reinterpret_cast<uintptr_t>(sc) & 15u) == 0) ? n / 4 : 0;
  const uint32_t top = (1u << width) - 1u;
  for (int i0 = tid; i0 < n4; i0 += T * 8) {
    float4 v[8];
#pragma unroll
    for (int u = 0; u < 8; ++u)
      if (i0 + u * T < n4) v[u] = __ldcg(reinterpret_cast<const float4*>(sc) + i0 + u * T);
#pragma unroll
    for (int u = 0; u < 8; ++u) {
      const int i4 = i0 + u * T;
      if (i4 < n4) {
        uint4 key;
        key.x = (__float_as_uint(v[u].x) & 0x7FFFFFFFu) - kmin;   // the mask drops the sign of -0
        key.y = (__float_as_uint(v[u].y) & 0x7FFFFFFFu) - kmin;
        key.z = (__float_as_uint(v[u].z) & 0x7FFFFFFFu) - kmin;
        key.w = (__float_as_uint(v[u].w) & 0x7FFFFFFFu) - kmin;
        reinterpret_cast<uint4*>(s_keys)[i4] = key;
        // (the clamp only matters if the range words were damaged, e.g. by two launches sharing one workspace)
        atomicAdd(&sh.hist[min(key.x >> shift, top)], 1u); atomicAdd(&sh.hist[min(key.y >> shift, top)], 1u);
        atomicAdd(&sh.hist[min(key.z >> shift, top)], 1u); atomicAdd(&sh.hist[min(key.w >> shift, top)], 1u);
      }
    }
  }
  for (int i = 4 * n4 + tid; i < n; i += T) {
    const uint32_t key = (__float_as_uint(__ldcg(sc + i)) & 0x7FFFFFFFu) - kmin;
    s_keys[i] = key;
    atomicAdd(&sh.hist[min(key >> shift, top)], 1u);
  }
  __syncthreads();

  // ---- 2. the k-th largest key: after this sh.prefix is that key (relative to kmin) and sh.remaining how many of
  // the keys equal to it belong to the kept set.
  bool listed = false;
  int cur = 0;
  uint32_t nlist = 0;
  for (;;) {
    threshold_bin<T>(sh, 1 << width, shift);
    if (shift == 0) break;                        // every bit of the range is decided
    const uint32_t prefix = sh.prefix, nbin = sh.nbin;
    if (listed || nbin <= (uint32_t)kCandMax) {   // the keys of the threshold's bin, in any order
      const int nxt = listed ? cur ^ 1 : 0;
      if (listed) {
        for (uint32_t i = tid; i < nlist; i += T) {
          const uint32_t key = sh.cand[cur][i];
          if ((key >> shift) == (prefix >> shift)) sh.cand[nxt][atomicAdd(&sh.ncand[nxt], 1u)] = key;
        }
      } else {
        for (int i0 = tid * 4; i0 < n; i0 += T * 4) {
          const uint4 v = reinterpret_cast<const uint4*>(s_keys)[i0 >> 2];
          const uint32_t key[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
          for (int e = 0; e < 4; ++e)
            if (i0 + e < n && (key[e] >> shift) == (prefix >> shift)) sh.cand[nxt][atomicAdd(&sh.ncand[nxt], 1u)] = key[e];
        }
      }
      listed = true; cur = nxt; nlist = nbin;
      __syncthreads();
      if (nlist <= (uint32_t)kCountMax) {         // finish by counting: the key with fewer than `remaining` keys above
        const uint32_t rem = sh.remaining;        // it and at least `remaining` keys not below it
        __syncthreads();
        if ((uint32_t)tid < nlist) {
          const uint32_t key = sh.cand[cur][tid];
          uint32_t gt = 0, eq = 0;
          for (uint32_t j = 0; j < nlist; ++j) { const uint32_t c = sh.cand[cur][j]; gt += c > key; eq += c == key; }
          if (gt < rem && rem <= gt + eq) { sh.prefix = key; sh.remaining = rem - gt; }   // equal keys write the same
        }
        __syncthreads();
        break;
      }
    }
    // the next 8-bit digit of the keys that share the prefix
    width = min(shift, 8);
    shift -= width;
    if (tid < 256) sh.hist[tid] = 0u;
    if (tid == 0 && listed) sh.ncand[cur ^ 1] = 0u;
    __syncthreads();
    const uint32_t dmask = (1u << width) - 1u;
    if (listed) {
      for (uint32_t i = tid; i < nlist; i += T) atomicAdd(&sh.hist[(sh.cand[cur][i] >> shift) & dmask], 1u);
    } else {
      const int up = shift + width;               // <= 20: the first digit took at least one bit above it
      for (int i0 = tid * 4; i0 < n; i0 += T * 4) {
        const uint4 v = reinterpret_cast<const uint4*>(s_keys)[i0 >> 2];
        const uint32_t key[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
        for (int e = 0; e < 4; ++e)
          if (i0 + e < n && (key[e] >> up) == (prefix >> up)) atomicAdd(&sh.hist[(key[e] >> shift) & dmask], 1u);
      }
    }
    __syncthreads();
  }
  const uint32_t tau = sh.prefix;  // relative to kmin
  const uint32_t need_eq = sh.remaining;
  __syncthreads();                 // the histogram is reused below

  // ---- 3. ordered compaction, 128 consecutive tokens per warp step (four per lane).  Counts per 128 tokens of the
  // keys above the threshold (low half) and equal to it (high half; n <= 49152 keeps either total below 2^16), one
  // scan over them, then every lane knows the output slots of its tokens.
  uint32_t* seg = sh.hist;
  const int nchunk = (n + 127) / 128;      // <= 384: one per thread in the scan
  const uint4* s_keys4 = reinterpret_cast<const uint4*>(s_keys);   // the allocation is padded to whole 16-byte words
  for (int c = warp; c < nchunk; c += (T / 32)) {
    const int i0 = c * 128 + lane * 4;
    uint32_t p = 0;
    if (i0 < n) {
      const uint4 v = s_keys4[i0 >> 2];
      const uint32_t key[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
      for (int e = 0; e < 4; ++e)
        if (i0 + e < n) p += (uint32_t)(key[e] > tau) + ((uint32_t)(key[e] == tau) << 16);
    }
    p = __reduce_add_sync(0xffffffffu, p);
    if (lane == 0) seg[c] = p;
  }
  __syncthreads();
  {
    const uint32_t mine = tid < nchunk ? seg[tid] : 0u;
    uint32_t tot;
    const uint32_t before = block_exclusive_scan<T>(mine, sh.warp, &tot);
    if (tid < nchunk) seg[tid] = before;
  }
  __syncthreads();
  const float tau_f = __uint_as_float(tau + kmin);
  const float band = 1e-5f * tau_f;
  uint32_t near = 0;
  for (int c = warp; c < nchunk; c += (T / 32)) {
    const int i0 = c * 128 + lane * 4;
    uint32_t key[4] = {0u, 0u, 0u, 0u};
    uint32_t p = 0;
    if (i0 < n) {
      const uint4 v = s_keys4[i0 >> 2];
      key[0] = v.x; key[1] = v.y; key[2] = v.z; key[3] = v.w;
#pragma unroll
      for (int e = 0; e < 4; ++e)
        if (i0 + e < n) p += (uint32_t)(key[e] > tau) + ((uint32_t)(key[e] == tau) << 16);
    }
    uint32_t inc = p;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      const uint32_t t = __shfl_up_sync(0xffffffffu, inc, o);
      if (lane >= o) inc += t;
    }
    const uint32_t base = seg[c] + inc - p;
    uint32_t gt_before = base & 0xFFFFu, eq_before = base >> 16;
#pragma unroll
    for (int e = 0; e < 4; ++e) {
      if (i0 + e < n) {
        const bool is_gt = key[e] > tau, is_eq = key[e] == tau;
        if (is_gt || (is_eq && eq_before < need_eq)) {          // equal keys: the lowest indices
          const uint32_t pos = gt_before + min(eq_before, need_eq);   // kept tokens before this one
          idx_b[pos] = i0 + e;
          if (inv_b) inv_b[i0 + e] = (int32_t)pos;   // the other entries were set to -1 when the rows were scored
        }
        gt_before += is_gt; eq_before += is_eq;
        if (near_tie_b) near += (fabsf(__uint_as_float(key[e] + kmin) - tau_f) <= band);
      }
    }
  }
  if (near_tie_b) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) near += __shfl_xor_sync(0xffffffffu, near, o);
    if (lane == 0) atomicAdd(&sh.near, near);
    __syncthreads();
    if (tid == 0) *near_tie_b = (int32_t)sh.near;
  }
}

// grid (CTAs per image, B), 1024 threads, one CTA per SM (the CTA that ranks an image then has 32 warps to hide the
// latencies of its sweeps with); the warps of an image stride over its token rows.  Dynamic shared memory
// max(9 C, n) * 4 bytes (mean token and staged partial sums, then keys).
template <typename XT>
__global__ void __launch_bounds__(kSelectThreads, 1) score_topk_kernel(const XT* __restrict__ x,
                                                                  const float4* __restrict__ group_partial, int ngroups, int n,
                                                                  int C4, int k, int staged, float* __restrict__ score,
                                                                  unsigned int* img_tickets, unsigned int* img_range, int32_t* __restrict__ idx,
                                                                  int32_t* __restrict__ inv, int32_t* __restrict__ near_tie) {
  extern __shared__ float4 s_dyn[];
  float4* s_mean = s_dyn;
  uint32_t* s_keys = reinterpret_cast<uint32_t*>(s_dyn);  // reused once the scores are out
  __shared__ TopkShared sh;
  __shared__ int s_last;
  const int b = blockIdx.y, tid = threadIdx.x;
  pdl_trigger();
  pdl_wait();
  if (staged) mean_from_partials_halves<kSelectThreads>(s_mean, s_mean + C4, group_partial + (size_t)b * ngroups * C4, ngroups, C4, n);
  else mean_from_partials<kSelectThreads>(s_mean, group_partial + (size_t)b * ngroups * C4, ngroups, nullptr, 0, C4, n);   // very wide maps
  __syncthreads();
  uint32_t lo = 0xFFFFFFFFu, hi = 0u;
  score_rows<kSelectThreads, true, 8, XT>(x, s_mean, b, n, C4, score, inv, lo, hi);
  publish_range<kSelectThreads>(lo, hi, sh, img_range + 2 * b);
  __threadfence();  // this thread's scores (and range) are visible device-wide before the CTA takes its ticket

  // ---- the last CTA of this image to get here ranks the image
  __syncthreads();
  if (tid == 0) {
    const unsigned int prev = atomicAdd(img_tickets + b, 1u);
    s_last = (prev == gridDim.x - 1);
    if (s_last) img_tickets[b] = 0u;
  }
  __syncthreads();
  if (!s_last) return;
  __threadfence();
  topk_image<kSelectThreads>(score + (size_t)b * n, n, k, s_keys, sh, idx + (size_t)b * k, inv ? inv + (size_t)b * n : nullptr, near_tie ? near_tie + b : nullptr,
             img_range + 2 * b);
}

// ------------------------------------------------------------------------------------------------------------
// The selection of a wrapped sublayer inside a scale step, fused with what surrounds it on the kept rows:
//   phase 0  Cached Token Restoration of the PREVIOUS sublayer's kept rows (Eq. 6's scatter of the forwarded rows,
//            with gate and residual): x[idx_prev[j]] += gamma * y[j].  (The rows that were not kept were restored
//            from the cache by the restore kernel on the side stream, which also left their column sums.)  The
//            column sums of the rows updated here are folded CTA -> group of CTAs -> image, in a fixed order.
//   barrier  every CTA waits until all groups are folded (an arrival count in global memory; bounded wait).
//   phase 1  Eq. 4's mean token from the two sets of sums, Eq. 5's scores, and -- by the last CTA of an image to
//            finish -- the exact top-k (kept indices ascending, inverse map).
//   flag     the other CTAs of the image wait for its top-k (bounded).
//   phase 2  Algorithm 1's gather of the kept rows fused with LayerNorm and AdaLN modulation -> bf16 A operand.
// The grid never exceeds what the GPU holds at once (the launcher asks the occupancy calculator), so the waits
// cannot starve a CTA that has not started.  A wait that expires leaves a code in the status word and the CTA
// returns; nothing spins without a limit.
struct FusedSelectArgs {
  float4* x; int n, C4, k;
  // phase 0 (y == nullptr: no kept rows to restore; the given sums then cover the whole map)
  const uint4* y; const int32_t* idx_prev; const float* gamma_prev; int mod_stride; int k_prev;
  float4* kept_cta_partial; float4* kept_group; unsigned int* kept_tickets; int gs, ngk;
  unsigned int* done; unsigned int done_target;
  // phase 1
  const float4* group_partial; int ngroups;
  float* score; unsigned int* img_tickets; unsigned int* img_range; int32_t* idx; int32_t* inv;
  unsigned int* ready; unsigned int epoch;
  // phase 2
  const float* sigma; const float* beta; uint2* a_out;
  int32_t* status;
};

__device__ __forceinline__ unsigned int ld_acquire_u32(const unsigned int* p) {
  unsigned int v;
  asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
  return v;
}
// Waits until the counter at `w` has reached `target` (counters only grow; compared as a wrapping difference), for
// at most two seconds.
__device__ __forceinline__ bool wait_counter(const unsigned int* w, unsigned int target) {
  unsigned long long t0 = 0;
  for (unsigned int spins = 0;; ++spins) {
    if ((int)(ld_acquire_u32(w) - target) >= 0) return true;
    if (spins == 64) asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t0));
    if (spins > 64 && (spins & 63u) == 0) {
      unsigned long long t1;
      asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t1));
      if (t1 - t0 > 2000000000ull) return false;
    }
    if (spins > 16) __nanosleep(64);
  }
}

// LayerNorm (+ modulation) of one token row by one warp, the row held in registers (C <= 2048); same arithmetic and
// order of sums as the stand-alone gather kernel.  Rows of the map may have been updated by other CTAs of this
// kernel (before the grid-wide wait), so they are read through L2, not through the read-only path.
__device__ __forceinline__ void gather_ln_row(const float4* row, int C4, const float4* s_sigma, const float4* s_beta,
                                              uint2* __restrict__ dst) {
  constexpr int kVec = 16;
  const int lane = threadIdx.x & 31;
  float4 v[kVec];
  float sum = 0.f;
#pragma unroll
  for (int i = 0; i < kVec; ++i) {
    const int c4 = lane + 32 * i;
    if (c4 < C4) v[i] = __ldcg(row + c4);
  }
#pragma unroll
  for (int i = 0; i < kVec; ++i) {
    const int c4 = lane + 32 * i;
    if (c4 < C4) sum += (v[i].x + v[i].y) + (v[i].z + v[i].w);
  }
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) sum += __shfl_xor_sync(0xffffffffu, sum, o);
  const float inv_c = 1.0f / (float)(C4 * 4);
  const float mu = sum * inv_c;
  float var = 0.f;
#pragma unroll
  for (int i = 0; i < kVec; ++i) {
    const int c4 = lane + 32 * i;
    if (c4 < C4) {
      const float dx = v[i].x - mu, dy = v[i].y - mu, dz = v[i].z - mu, dw = v[i].w - mu;
      var += (dx * dx + dy * dy) + (dz * dz + dw * dw);
    }
  }
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) var += __shfl_xor_sync(0xffffffffu, var, o);
  const float rstd = rsqrtf(var * inv_c + 1e-6f);
#pragma unroll
  for (int i = 0; i < kVec; ++i) {
    const int c4 = lane + 32 * i;
    if (c4 < C4) {
      float4 a;
      a.x = (v[i].x - mu) * rstd; a.y = (v[i].y - mu) * rstd; a.z = (v[i].z - mu) * rstd; a.w = (v[i].w - mu) * rstd;
      if (s_sigma) {
        const float4 sg = s_sigma[c4], bb = s_beta[c4];
        a.x = fmaf(a.x, 1.f + sg.x, bb.x); a.y = fmaf(a.y, 1.f + sg.y, bb.y);
        a.z = fmaf(a.z, 1.f + sg.z, bb.z); a.w = fmaf(a.w, 1.f + sg.w, bb.w);
      }
      __nv_bfloat162 lo = __floats2bfloat162_rn(a.x, a.y), hi = __floats2bfloat162_rn(a.z, a.w);
      uint2 o;
      o.x = *reinterpret_cast<uint32_t*>(&lo);
      o.y = *reinterpret_cast<uint32_t*>(&hi);
      dst[c4] = o;
    }
  }
}

__device__ __forceinline__ void bf16x8_widen(const uint4& p, float (&f)[8]) {
  const uint32_t u[4] = {p.x, p.y, p.z, p.w};
#pragma unroll
  for (int i = 0; i < 4; ++i) { f[2 * i] = __uint_as_float(u[i] << 16); f[2 * i + 1] = __uint_as_float(u[i] & 0xFFFF0000u); }
}

// grid (CTAs per image, B), kTopkThreads threads, one CTA per SM (a thread may hold a token row's sixteen 16-byte
// words).  Dynamic shared memory: the largest of the mean token, the keys of the top-k, the row-parallel copies of
// phase 0's sums and the modulation vectors of phase 2.
__global__ void __launch_bounds__(kTopkThreads, 1) select_fused_kernel(const FusedSelectArgs a) {
  extern __shared__ float4 s_dyn[];
  __shared__ TopkShared sh;
  __shared__ int s_flag;
  const int b = blockIdx.y, cta = blockIdx.x, G = gridDim.x, tid = threadIdx.x;
  const int n = a.n, C4 = a.C4;
  pdl_trigger();
  pdl_wait();
  bool ok = true;

  // ---- phase 0: the previous sublayer's kept rows
  if (a.y) {
    const int C8 = C4 / 2;
    const int rows_par = kTopkThreads / C8;       // rows a CTA updates side by side (>= 2: C <= 2048)
    const int c8 = tid % C8, rp = tid / C8;
    float4 a0 = make_float4(0.f, 0.f, 0.f, 0.f), a1 = a0;
    if (rp < rows_par) {
      float4 g0 = make_float4(1.f, 1.f, 1.f, 1.f), g1 = g0;
      if (a.gamma_prev) {
        const float4* g = reinterpret_cast<const float4*>(a.gamma_prev + (size_t)b * a.mod_stride);
        g0 = __ldg(g + 2 * c8); g1 = __ldg(g + 2 * c8 + 1);
      }
      const int stride = G * rows_par;
      const int32_t* ip = a.idx_prev + (size_t)b * a.k_prev;
      const uint4* yb = a.y + (size_t)b * a.k_prev * C8;
      float4* xb = a.x + (size_t)b * n * C4;
      for (int j = cta + G * rp; j < a.k_prev; j += 2 * stride) {     // two rows in flight
        const int j2 = j + stride;
        const bool two = j2 < a.k_prev;
        const int t1 = min(max(__ldg(ip + j), 0), n - 1);
        const int t2 = two ? min(max(__ldg(ip + j2), 0), n - 1) : t1;
        float4* xr1 = xb + (size_t)t1 * C4 + 2 * c8;
        float4* xr2 = xb + (size_t)t2 * C4 + 2 * c8;
        float4 u0 = xr1[0], u1 = xr1[1];
        const uint4 p1 = __ldg(yb + (size_t)j * C8 + c8);
        float4 w0 = u0, w1 = u1;
        uint4 p2 = p1;
        if (two) { w0 = xr2[0]; w1 = xr2[1]; p2 = __ldg(yb + (size_t)j2 * C8 + c8); }
        float f[8];
        bf16x8_widen(p1, f);
        if (a.gamma_prev) {
          u0.x = fmaf(g0.x, f[0], u0.x); u0.y = fmaf(g0.y, f[1], u0.y); u0.z = fmaf(g0.z, f[2], u0.z); u0.w = fmaf(g0.w, f[3], u0.w);
          u1.x = fmaf(g1.x, f[4], u1.x); u1.y = fmaf(g1.y, f[5], u1.y); u1.z = fmaf(g1.z, f[6], u1.z); u1.w = fmaf(g1.w, f[7], u1.w);
        } else {
          u0.x += f[0]; u0.y += f[1]; u0.z += f[2]; u0.w += f[3];
          u1.x += f[4]; u1.y += f[5]; u1.z += f[6]; u1.w += f[7];
        }
        xr1[0] = u0; xr1[1] = u1;
        a0.x += u0.x; a0.y += u0.y; a0.z += u0.z; a0.w += u0.w;
        a1.x += u1.x; a1.y += u1.y; a1.z += u1.z; a1.w += u1.w;
        if (two) {
          bf16x8_widen(p2, f);
          if (a.gamma_prev) {
            w0.x = fmaf(g0.x, f[0], w0.x); w0.y = fmaf(g0.y, f[1], w0.y); w0.z = fmaf(g0.z, f[2], w0.z); w0.w = fmaf(g0.w, f[3], w0.w);
            w1.x = fmaf(g1.x, f[4], w1.x); w1.y = fmaf(g1.y, f[5], w1.y); w1.z = fmaf(g1.z, f[6], w1.z); w1.w = fmaf(g1.w, f[7], w1.w);
          } else {
            w0.x += f[0]; w0.y += f[1]; w0.z += f[2]; w0.w += f[3];
            w1.x += f[4]; w1.y += f[5]; w1.z += f[6]; w1.w += f[7];
          }
          xr2[0] = w0; xr2[1] = w1;
          a0.x += w0.x; a0.y += w0.y; a0.z += w0.z; a0.w += w0.w;
          a1.x += w1.x; a1.y += w1.y; a1.z += w1.z; a1.w += w1.w;
        }
      }
    }
    // the row-parallel copies of the sums, added in a fixed order -> this CTA's partial
    if (rp > 0 && rp < rows_par) { s_dyn[((size_t)(rp - 1) * C8 + c8) * 2] = a0; s_dyn[((size_t)(rp - 1) * C8 + c8) * 2 + 1] = a1; }
    __syncthreads();
    if (rp == 0) {
      for (int r = 1; r < rows_par; ++r) {
        const float4 v0 = s_dyn[((size_t)(r - 1) * C8 + c8) * 2], v1 = s_dyn[((size_t)(r - 1) * C8 + c8) * 2 + 1];
        a0.x += v0.x; a0.y += v0.y; a0.z += v0.z; a0.w += v0.w;
        a1.x += v1.x; a1.y += v1.y; a1.z += v1.z; a1.w += v1.w;
      }
      float4* cp = a.kept_cta_partial + ((size_t)b * G + cta) * C4 + 2 * c8;
      cp[0] = a0; cp[1] = a1;
    }
    const bool folded = fold_group_partials(b, cta, G, a.gs, a.ngk, C4, a.kept_cta_partial, a.kept_group, a.kept_tickets);
    if (folded) {      // uniform over the CTA
      __threadfence();
      __syncthreads();
      if (tid == 0) atomicAdd(a.done, 1u);
    }
    // ---- every group of every image folded?
    if (tid == 0) {
      const bool w = wait_counter(a.done, a.done_target);
      if (!w && a.status) atomicCAS(a.status, 0, DEV_TIMEOUT_GRID);
      s_flag = w;
    }
    __syncthreads();
    ok = s_flag != 0;
    __syncthreads();      // s_flag is reused below
    __threadfence();
  }
  if (!ok) return;

  // ---- phase 1: mean token, scores, top-k
  mean_from_partials<kTopkThreads>(s_dyn, a.group_partial + (size_t)b * a.ngroups * C4, a.ngroups,
                     a.y ? a.kept_group + (size_t)b * a.ngk * C4 : nullptr, a.y ? a.ngk : 0, C4, n);
  __syncthreads();
  uint32_t lo = 0xFFFFFFFFu, hi = 0u;
  score_rows<kTopkThreads, false, 16, float>(reinterpret_cast<const float*>(a.x), s_dyn, b, n, C4, a.score, a.inv, lo, hi);
  publish_range<kTopkThreads>(lo, hi, sh, a.img_range + 2 * b);
  __threadfence();
  __syncthreads();
  if (tid == 0) {
    const unsigned int prev = atomicAdd(a.img_tickets + b, 1u);
    const int last = (prev == (unsigned int)G - 1u);
    if (last) a.img_tickets[b] = 0u;
    s_flag = last;
  }
  __syncthreads();
  const bool last = s_flag != 0;
  float4* s_sigma = nullptr;
  float4* s_beta = nullptr;
  if (last) {
    __threadfence();
    topk_image<kTopkThreads>(a.score + (size_t)b * n, n, a.k, reinterpret_cast<uint32_t*>(s_dyn), sh, a.idx + (size_t)b * a.k, a.inv + (size_t)b * n, nullptr,
               a.img_range + 2 * b);
    __threadfence();
    __syncthreads();
    if (tid == 0) asm volatile("st.release.gpu.global.u32 [%0], %1;" ::"l"(a.ready + b), "r"(a.epoch) : "memory");
  }
  // the modulation vectors of the image (they do not depend on the selection: fetched before the wait)
  if (a.sigma) {
    s_sigma = s_dyn; s_beta = s_dyn + C4;
    const float4* sg = reinterpret_cast<const float4*>(a.sigma + (size_t)b * a.mod_stride);
    const float4* bt = reinterpret_cast<const float4*>(a.beta + (size_t)b * a.mod_stride);
    for (int i = tid; i < C4; i += kTopkThreads) { s_sigma[i] = __ldg(sg + i); s_beta[i] = __ldg(bt + i); }
  }
  if (!last) {
    if (tid == 0) {
      const bool w = wait_counter(a.ready + b, a.epoch);
      if (!w && a.status) atomicCAS(a.status, 0, DEV_TIMEOUT_GRID);
      s_flag = w;
    }
    __syncthreads();
    if (s_flag == 0) return;
    __threadfence();
  } else {
    __syncthreads();
  }

  // ---- phase 2: gather + LayerNorm + modulation of the kept rows, one warp per row
  const int warp = tid >> 5;
  const int32_t* ib = a.idx + (size_t)b * a.k;
  for (int j = cta * kTopkWarps + warp; j < a.k; j += G * kTopkWarps) {
    const int t = min(max(__ldcg(ib + j), 0), n - 1);
    gather_ln_row(a.x + ((size_t)b * n + t) * C4, C4, s_sigma, s_beta, a.a_out + ((size_t)b * a.k + j) * C4);
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

// group arrival counters [B, kMaxGroups], image arrival counters [B], score range words [B, 2]
size_t select_ticket_bytes(int B) { return align_up((size_t)B * (kMaxGroups + 3) * sizeof(unsigned int), 256); }

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
  e = cudaFuncSetAttribute(score_topk_kernel<float>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kTopkMaxSmem);
  if (e == cudaSuccess) e = cudaFuncSetAttribute(score_topk_kernel<__nv_bfloat16>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kTopkMaxSmem);
  if (e != cudaSuccess) return e;
  return cudaFuncSetAttribute(select_fused_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kTopkMaxSmem);
}

template <typename XT>
static cudaError_t launch_select_t(const XT* x, int B, int n, int C, int k, int32_t* idx, int32_t* inv, float* sc, int32_t* near_tie,
                                   const SelectWs& w, bool have_partials, cudaStream_t st) {
  const int C4 = C / 4;
  if (!have_partials)
    launch_pdl(colsum_chunk_kernel<XT>, dim3(w.nchunks, B), dim3(256), 0, st, x, n, C4, w.nchunks, w.group,
               w.ngroups, reinterpret_cast<float4*>(w.chunk_partial), reinterpret_cast<float4*>(w.group_partial), w.tickets);
  const size_t keys_smem = ((size_t)n + 3) / 4 * 16;   // whole 16-byte words
  const int staged = (size_t)C * 4 * 9 <= kTopkMaxSmem;  // room for the mean token and eight staged partial sums
  const size_t mean_smem = (size_t)C * 4 * (staged ? 9 : 1);
  const size_t smem = keys_smem > mean_smem ? keys_smem : mean_smem;
  // one CTA per SM over the B images, never more than one warp per token row
  int per_image = g_num_sms / B;
  const int need = (n + kSelectWarps - 1) / kSelectWarps;
  if (per_image > need) per_image = need;
  if (per_image < 1) per_image = 1;
  unsigned int* img_tickets = w.tickets + (size_t)B * kMaxGroups;
  unsigned int* img_range = w.tickets + (size_t)B * (kMaxGroups + 1);
  const float4* gp = reinterpret_cast<const float4*>(w.group_partial);
  launch_pdl(score_topk_kernel<XT>, dim3(per_image, B), dim3(kSelectThreads), smem, st, x, gp, w.ngroups, n, C4, k, staged, sc, img_tickets,
             img_range, idx, inv, near_tie);
  return cudaGetLastError();
}

cudaError_t launch_select(const void* x, int B, int n, int C, int k, int32_t* idx, int32_t* inv, float* score,
                          int32_t* near_tie, void* workspace, bool have_partials, cudaStream_t st, bool x_bf16) {
  const SelectWs w = select_ws_carve(workspace, B, n, C);
  float* sc = score ? score : w.score;
  const double es = x_bf16 ? 2.0 : 4.0;
  const double sel_bytes = (double)B * n * C * es + 4.0 * B * n + 4.0 * B * ((double)k + n);
  // the stand-alone column-sum pass reads the map a second time
  LaunchScope scope(KC_SELECT, have_partials ? 1 : 2, sel_bytes, sel_bytes + (have_partials ? 0.0 : (double)B * n * C * es), st);
  if (x_bf16) return launch_select_t(static_cast<const __nv_bfloat16*>(x), B, n, C, k, idx, inv, sc, near_tie, w, have_partials, st);
  return launch_select_t(static_cast<const float*>(x), B, n, C, k, idx, inv, sc, near_tie, w, have_partials, st);
}

// ---- the fused selection of a scale step
constexpr int kFusedMaxCtas = 320;     // CTAs per image the kept-row partials have room for
size_t select_fused_sync_bytes(int B) { return align_up((size_t)B * (kMaxGroups + 1) * sizeof(unsigned int) + 64, 256); }
size_t select_fused_ws_bytes(int B, int C) {
  return select_fused_sync_bytes(B) + align_up((size_t)B * kFusedMaxCtas * C * sizeof(float), 256) +
         align_up((size_t)B * kMaxGroups * C * sizeof(float), 256);
}

static size_t fused_smem_bytes(int n, int C) {
  const size_t keys = ((size_t)n + 3) / 4 * 16;
  const size_t vec = (size_t)C * 4;                       // the mean token
  const int rows_par = kTopkThreads / (C / 8);
  const size_t comb = (size_t)(rows_par > 1 ? rows_par - 1 : 0) * C * 4;
  size_t m = keys > 2 * vec ? keys : 2 * vec;             // keys | sigma + beta
  return m > comb ? m : comb;
}

// CTAs per image of the fused kernel: never more than the GPU holds at once (its CTAs wait on one another), never
// more than one warp per token row.  0: the shape cannot take the fused path.
static int fused_ctas_per_image(int B, int n, int C) {
  if (C % 8 || C / 8 > kTopkThreads / 2 || C > 2048 || n > kTopkMaxTokens) return 0;
  int per_sm = 0;
  if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, select_fused_kernel, kTopkThreads, fused_smem_bytes(n, C)) != cudaSuccess) {
    (void)cudaGetLastError();
    return 0;
  }
  long g = (long)per_sm * g_num_sms / B;
  const long need = (n + kTopkWarps - 1) / kTopkWarps;
  if (g > need) g = need;
  if (g > kFusedMaxCtas) g = kFusedMaxCtas;
  return (int)g;
}
bool select_fused_supported(int B, int n, int C) { return fused_ctas_per_image(B, n, C) >= 1; }

cudaError_t launch_select_fused(const FusedSelect& f, cudaStream_t st) {
  const int G = fused_ctas_per_image(f.B, f.n, f.C);
  if (G < 1) return cudaErrorInvalidConfiguration;
  const SelectWs w = select_ws_carve(f.sel_ws, f.B, f.n, f.C);
  char* fw = static_cast<char*>(f.fused_ws);
  FusedSelectArgs a{};
  a.x = reinterpret_cast<float4*>(f.x); a.n = f.n; a.C4 = f.C / 4; a.k = f.k;
  a.y = reinterpret_cast<const uint4*>(f.y); a.idx_prev = f.idx_prev; a.gamma_prev = f.gamma_prev; a.mod_stride = f.mod_stride; a.k_prev = f.k;
  a.kept_tickets = reinterpret_cast<unsigned int*>(fw);
  a.done = a.kept_tickets + (size_t)f.B * kMaxGroups;
  a.ready = a.done + 16;                                   // one word per image
  a.kept_cta_partial = reinterpret_cast<float4*>(fw + select_fused_sync_bytes(f.B));
  a.kept_group = reinterpret_cast<float4*>(fw + select_fused_sync_bytes(f.B) + align_up((size_t)f.B * kFusedMaxCtas * f.C * sizeof(float), 256));
  a.gs = (G + kMaxGroups - 1) / kMaxGroups;
  a.ngk = (G + a.gs - 1) / a.gs;
  if (f.y) *f.done_total += (unsigned int)(f.B * a.ngk);
  a.done_target = *f.done_total;
  a.epoch = ++*f.epoch;
  a.group_partial = reinterpret_cast<const float4*>(w.group_partial); a.ngroups = w.ngroups;
  a.score = w.score; a.img_tickets = w.tickets + (size_t)f.B * kMaxGroups;
  a.img_range = w.tickets + (size_t)f.B * (kMaxGroups + 1); a.idx = f.idx; a.inv = f.inv;
  a.sigma = f.sigma; a.beta = f.beta; a.a_out = reinterpret_cast<uint2*>(f.a_out);
  a.status = f.status;
  // algorithmic bytes: the selection (x once, scores, indices), the gather (kept rows in, bf16 out) and, when it
  // carries the previous sublayer's kept rows, their restoration (x read + written, y read)
  const double rows = (double)f.B * f.k;
  const double sel_bytes = (double)f.B * f.n * f.C * 4.0 + 4.0 * f.B * f.n + 4.0 * f.B * ((double)f.k + f.n);
  const double gat_bytes = rows * f.C * 6.0;
  const double res_bytes = f.y ? rows * f.C * 10.0 : 0.0;
  LaunchScope scope(KC_SELECT, 1, sel_bytes + gat_bytes + res_bytes, sel_bytes + gat_bytes + res_bytes, st);
  return launch_pdl(select_fused_kernel, dim3(G, f.B), dim3(kTopkThreads), fused_smem_bytes(f.n, f.C), st, a);
}

cudaError_t launch_colsum(const float* x, int B, int n, int C, void* workspace, cudaStream_t st) {
  const SelectWs w = select_ws_carve(workspace, B, n, C);
  LaunchScope scope(KC_SELECT, 1, (double)B * n * C * 4.0, (double)B * n * C * 4.0, st);
  return launch_pdl(colsum_chunk_kernel<float>, dim3(w.nchunks, B), dim3(256), 0, st, x, n, C / 4, w.nchunks, w.group,
                    w.ngroups, reinterpret_cast<float4*>(w.chunk_partial), reinterpret_cast<float4*>(w.group_partial), w.tickets);
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
