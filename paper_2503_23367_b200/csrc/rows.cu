// Row-wise HBM-bound kernels of the pruned step:
//   gather_ln        : Algorithm 1's gather of the kept rows fused with the block's pre-LayerNorm and
//                      AdaLN modulation; writes the bf16 A operand of the following GEMM.
//   restore_residual : Cached Token Restoration (Eq. 6, Algorithm 1 second routine) written as a
//                      gather through the inverse index map (no scatter, so no write races), fused
//                      with the gate and the residual add.
//   restore_bf16     : the plain restoration, bf16 in / bf16 out, bit-exact copy.
// Every global access is a 128-bit vector, consecutive lanes touching consecutive 16-byte words.  The
// kernels are short, so they are arranged to keep the chain of dependent global accesses short (index
// -> row -> store) with everything else (modulation vectors, the residual rows) fetched beside it.
#include <cuda_bf16.h>

#include "colsum_fold.cuh"
#include "internal.h"
#include "sm100.cuh"

namespace fv {

namespace {

constexpr int kMaxVec = 16;  // float4 per lane -> C <= 2048

// grid (ceil(k / 8), B): one warp per kept row; sigma / beta of the image staged in shared memory while
// the row index and the row itself are in flight.
template <typename XT>
__global__ void __launch_bounds__(256) gather_ln_kernel(const XT* __restrict__ x, const int32_t* __restrict__ idx, int n,
                                                        int k, int C4, const float* __restrict__ sigma,
                                                        const float* __restrict__ beta, int mod_stride,
                                                        uint2* __restrict__ a_out, int32_t* status) {
  extern __shared__ float4 s_mod[];  // sigma [C4] then beta [C4]
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int b = blockIdx.y, j = blockIdx.x * 8 + warp;
  const bool live = j < k;
  pdl_trigger();
  pdl_wait();
  int t = live ? (idx ? __ldg(idx + (size_t)b * k + j) : j) : 0;
  if (t < 0 || t >= n) {   // a caller's index outside the map: stay inside it and say so
    if (status && lane == 0) atomicCAS(status, 0, DEV_BAD_ROW_INDEX);
    t = min(max(t, 0), n - 1);
  }
  if (sigma) {
    const float4* sg = reinterpret_cast<const float4*>(sigma + (size_t)b * mod_stride);
    const float4* bt = reinterpret_cast<const float4*>(beta + (size_t)b * mod_stride);
    for (int i = threadIdx.x; i < C4; i += 256) { s_mod[i] = __ldg(sg + i); s_mod[C4 + i] = __ldg(bt + i); }
  }
  const XT* row = x + ((size_t)b * n + t) * C4 * 4;
  float4 v[kMaxVec];
  float sum = 0.f;
  if (live) {
#pragma unroll
    for (int i = 0; i < kMaxVec; ++i) {
      const int c4 = lane + 32 * i;
      if (c4 < C4) v[i] = x_load4<true>(row + (size_t)c4 * 4);
    }
#pragma unroll
    for (int i = 0; i < kMaxVec; ++i) {
      const int c4 = lane + 32 * i;
      if (c4 < C4) sum += (v[i].x + v[i].y) + (v[i].z + v[i].w);
    }
  }
  __syncthreads();
  if (!live) return;
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) sum += __shfl_xor_sync(0xffffffffu, sum, o);
  const float inv_c = 1.0f / (float)(C4 * 4);
  const float mu = sum * inv_c;
  float var = 0.f;
#pragma unroll
  for (int i = 0; i < kMaxVec; ++i) {
    const int c4 = lane + 32 * i;
    if (c4 < C4) {
      float dx = v[i].x - mu, dy = v[i].y - mu, dz = v[i].z - mu, dw = v[i].w - mu;
      var += (dx * dx + dy * dy) + (dz * dz + dw * dw);
    }
  }
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) var += __shfl_xor_sync(0xffffffffu, var, o);
  const float rstd = rsqrtf(var * inv_c + 1e-6f);
  uint2* dst = a_out + ((size_t)b * k + j) * C4;
#pragma unroll
  for (int i = 0; i < kMaxVec; ++i) {
    const int c4 = lane + 32 * i;
    if (c4 < C4) {
      float4 a;
      a.x = (v[i].x - mu) * rstd; a.y = (v[i].y - mu) * rstd; a.z = (v[i].z - mu) * rstd; a.w = (v[i].w - mu) * rstd;
      if (sigma) {
        const float4 sg = s_mod[c4], bb = s_mod[C4 + c4];
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

__device__ __forceinline__ int nearest_src(int t, int h, int w, int hc, int wc) {
  const int y = t / w, xx = t - y * w;
  return ((y * hc) / h) * wc + (xx * wc) / w;
}

// interpolate(.) of Eq. 6 beyond nearest neighbour, half-pixel centres (source coordinate
// (dst + 0.5) * in / out - 0.5 per axis): the source tokens of destination token t and their weights.
//   TAPS 4 : bilinear (coordinate clamped to the map, two taps per axis);
//   TAPS 16: bicubic, separable cubic convolution (Keys' kernel, a = -0.75), four taps per axis with the
//            tap indices clamped to the map.
template <int TAPS> struct InterpTaps { int src[TAPS]; float wt[TAPS]; };

__device__ __forceinline__ void cubic_axis(int o, int n_out, int n_in, int (&idx)[4], float (&wt)[4]) {
  const double a = -0.75;
  const double s = (o + 0.5) * (double)n_in / n_out - 0.5;
  const int i0 = (int)floor(s);
#pragma unroll
  for (int q = 0; q < 4; ++q) {
    const int pos = i0 - 1 + q;
    const double d = fabs(s - pos);
    const double wv = d <= 1.0 ? ((a + 2.0) * d - (a + 3.0)) * d * d + 1.0 : (d < 2.0 ? ((a * d - 5.0 * a) * d + 8.0 * a) * d - 4.0 * a : 0.0);
    idx[q] = min(max(pos, 0), n_in - 1);
    wt[q] = (float)wv;
  }
}

template <int TAPS>
__device__ __forceinline__ InterpTaps<TAPS> interp_taps(int t, int h, int w, int hc, int wc) {
  const int y = t / w, xx = t - y * w;
  InterpTaps<TAPS> b;
  if constexpr (TAPS == 4) {
    double sy = (y + 0.5) * (double)hc / h - 0.5, sx = (xx + 0.5) * (double)wc / w - 0.5;
    sy = fmin(fmax(sy, 0.0), (double)(hc - 1)); sx = fmin(fmax(sx, 0.0), (double)(wc - 1));
    const int y0 = (int)floor(sy), x0 = (int)floor(sx);
    const int y1 = min(y0 + 1, hc - 1), x1 = min(x0 + 1, wc - 1);
    const float ty = (float)(sy - y0), tx = (float)(sx - x0);
    b.src[0] = y0 * wc + x0; b.src[1] = y0 * wc + x1; b.src[2] = y1 * wc + x0; b.src[3] = y1 * wc + x1;
    b.wt[0] = (1.f - ty) * (1.f - tx); b.wt[1] = (1.f - ty) * tx; b.wt[2] = ty * (1.f - tx); b.wt[3] = ty * tx;
  } else {
    int yi[4], xi[4];
    float yw[4], xw[4];
    cubic_axis(y, h, hc, yi, yw);
    cubic_axis(xx, w, wc, xi, xw);
#pragma unroll
    for (int qy = 0; qy < 4; ++qy)
#pragma unroll
      for (int qx = 0; qx < 4; ++qx) { b.src[4 * qy + qx] = yi[qy] * wc + xi[qx]; b.wt[4 * qy + qx] = yw[qy] * xw[qx]; }
  }
  return b;
}

__device__ __forceinline__ void bf16x8_to_float(const uint4& p, float (&f)[8]) {
  const uint32_t u[4] = {p.x, p.y, p.z, p.w};
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    f[2 * i] = __uint_as_float(u[i] << 16);
    f[2 * i + 1] = __uint_as_float(u[i] & 0xFFFF0000u);
  }
}

// x[b,t,:] += gamma[b,:] * (inv[b,t] >= 0 ? y[b*k + inv[b,t], :] : cache[b, src(t), :])
// grid (chunks of 32 tokens, B), 256 threads; a thread owns 8 channels (one 16-byte bf16 word of the
// source, two float4 of x) for all rows of the chunk, so the column sums of the updated rows -- the
// next sublayer's Eq. 4 -- fall out of the same registers with no cross-thread reduction.  The source
// row of every token is resolved once into shared memory; the x rows do not wait for it.
// `part` splits the work so that the bulk of it can run beside the sublayer's GEMMs and attention:
//   0 : every row;  1 : only the rows that were NOT kept (they depend on the selection and the cache alone:
//   column sums start at zero and are left as the chunk partial);  2 : only the kept rows (after the
//   branch has produced y: column sums continue from the chunk partial of part 1, then the group fold);
//   3 : as 1, but the sums of the rows that were not kept are folded here (the kept rows are then restored, and
//   summed, by the next selection's kernel).
// RF: rows in flight per thread (4, or 2 in the build that fits four CTAs per SM: 64 registers).
template <typename XT, int RF>
__global__ void __launch_bounds__(256, RF == 2 ? 4 : 3) restore_residual_kernel(XT* __restrict__ x, const uint4* __restrict__ y,
                                                               const uint4* __restrict__ cache, const int32_t* __restrict__ inv,
                                                               const float* __restrict__ gamma, int mod_stride, int n, int k,
                                                               int h, int w, int hc, int wc, int C8, int nchunks, int group,
                                                               int ngroups, float4* __restrict__ chunk_partial,
                                                               float4* __restrict__ group_partial, unsigned int* tickets,
                                                               int part) {
  __shared__ const uint4* s_src[kColsumRows];
  __shared__ int s_on[kColsumRows];
  pdl_trigger();
  pdl_wait();
  const int b = blockIdx.y, chunk = blockIdx.x;
  const int t0 = chunk * kColsumRows;
  const int rows = min(kColsumRows, n - t0);
  if (threadIdx.x < rows) {
    const int t = t0 + threadIdx.x;
    const int j = __ldg(inv + (size_t)b * n + t);
    s_src[threadIdx.x] = (j >= 0) ? y + ((size_t)b * k + j) * C8
                                  : cache + ((size_t)b * hc * wc + nearest_src(t, h, w, hc, wc)) * C8;
    s_on[threadIdx.x] = part == 0 || (part == 1 || part == 3) == (j < 0);
  }
  __syncthreads();
  XT* xbase = x + ((size_t)b * n + t0) * C8 * 8;
  for (int c8 = threadIdx.x; c8 < C8; c8 += 256) {
    float4 g0 = make_float4(1.f, 1.f, 1.f, 1.f), g1 = g0;
    if (gamma) {
      const float4* g = reinterpret_cast<const float4*>(gamma + (size_t)b * mod_stride);
      g0 = __ldg(g + 2 * c8); g1 = __ldg(g + 2 * c8 + 1);
    }
    float4 a0 = make_float4(0.f, 0.f, 0.f, 0.f), a1 = a0;
    if (part == 2 && chunk_partial) {  // continue the sums of the rows updated by part 1
      const float4* cp = chunk_partial + ((size_t)b * nchunks + chunk) * C8 * 2 + 2 * c8;
      a0 = __ldcg(cp); a1 = __ldcg(cp + 1);
    }
    for (int r = 0; r < rows; r += RF) {
      uint4 p[RF];
      float xv[RF][8];
#pragma unroll
      for (int i = 0; i < RF; ++i) {
        if (r + i < rows && s_on[r + i]) {
          x_load8(xbase + ((size_t)(r + i) * C8 + c8) * 8, xv[i]);
          p[i] = __ldg(s_src[r + i] + c8);
        }
      }
#pragma unroll
      for (int i = 0; i < RF; ++i) {
        if (r + i < rows && s_on[r + i]) {
          float f[8];
          bf16x8_to_float(p[i], f);
          float (&u)[8] = xv[i];
          if (gamma) {
            u[0] = fmaf(g0.x, f[0], u[0]); u[1] = fmaf(g0.y, f[1], u[1]); u[2] = fmaf(g0.z, f[2], u[2]); u[3] = fmaf(g0.w, f[3], u[3]);
            u[4] = fmaf(g1.x, f[4], u[4]); u[5] = fmaf(g1.y, f[5], u[5]); u[6] = fmaf(g1.z, f[6], u[6]); u[7] = fmaf(g1.w, f[7], u[7]);
          } else {
#pragma unroll
            for (int e = 0; e < 8; ++e) u[e] += f[e];
          }
          x_store8(xbase + ((size_t)(r + i) * C8 + c8) * 8, u);     // a bf16 stream: u now holds the stored (rounded) values
          a0.x += u[0]; a0.y += u[1]; a0.z += u[2]; a0.w += u[3];
          a1.x += u[4]; a1.y += u[5]; a1.z += u[6]; a1.w += u[7];
        }
      }
    }
    if (chunk_partial) {
      float4* cp = chunk_partial + ((size_t)b * nchunks + chunk) * C8 * 2 + 2 * c8;
      cp[0] = a0; cp[1] = a1;
    }
  }
  if (chunk_partial && part != 1)
    fold_group_partials(b, chunk, nchunks, group, ngroups, C8 * 2, chunk_partial, group_partial, tickets);
}

__global__ void __launch_bounds__(256) restore_bf16_kernel(const uint4* __restrict__ cache, int hc, int wc,
                                                           const uint4* __restrict__ pivots, const int32_t* __restrict__ inv,
                                                           int n, int k, int h, int w, int C8, uint4* __restrict__ out,
                                                           int total_rows) {
  pdl_trigger();
  pdl_wait();
  const int warp = (blockIdx.x * blockDim.x + threadIdx.x) >> 5, lane = threadIdx.x & 31;
  if (warp >= total_rows) return;
  const int b = warp / n, t = warp - b * n;
  const int j = inv[warp];
  const uint4* src = (j >= 0) ? pivots + ((size_t)b * k + j) * C8
                              : cache + ((size_t)b * hc * wc + nearest_src(t, h, w, hc, wc)) * C8;
  uint4* dst = out + (size_t)warp * C8;
  for (int c8 = lane; c8 < C8; c8 += 32) dst[c8] = __ldg(src + c8);
}

// Per-step granularity: compact copy of the kept rows of the fp32 token map (Algorithm 1's gather).
// grid (ceil(k / 8), B): one warp per kept row.
__global__ void __launch_bounds__(256) gather_rows_kernel(const float4* __restrict__ x, const int32_t* __restrict__ idx, int n,
                                                          int k, int C4, float4* __restrict__ out, int32_t* status) {
  pdl_trigger();
  pdl_wait();
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int b = blockIdx.y, j = blockIdx.x * 8 + warp;
  if (j >= k) return;
  int t = __ldg(idx + (size_t)b * k + j);
  if (t < 0 || t >= n) {
    if (status && lane == 0) atomicCAS(status, 0, DEV_BAD_ROW_INDEX);
    t = min(max(t, 0), n - 1);
  }
  const float4* src = x + ((size_t)b * n + t) * C4;
  float4* dst = out + ((size_t)b * k + j) * C4;
  for (int c4 = lane; c4 < C4; c4 += 32) dst[c4] = __ldg(src + c4);
}

// Per-step granularity: Cached Token Restoration of the step's output map (Eq. 6), fp32, a copy:
// out[b,t,:] = inv[b,t] >= 0 ? pivots[b, inv[b,t], :] : cache[b, src(t), :].
__global__ void __launch_bounds__(256) restore_rows_f32_kernel(const float4* __restrict__ cache, int hc, int wc,
                                                               const float4* __restrict__ pivots, const int32_t* __restrict__ inv,
                                                               int n, int k, int h, int w, int C4, float4* __restrict__ out,
                                                               int total_rows) {
  pdl_trigger();
  pdl_wait();
  const int warp = (blockIdx.x * blockDim.x + threadIdx.x) >> 5, lane = threadIdx.x & 31;
  if (warp >= total_rows) return;
  const int b = warp / n, t = warp - b * n;
  const int j = __ldg(inv + warp);
  const float4* src = (j >= 0) ? pivots + ((size_t)b * k + j) * C4
                               : cache + ((size_t)b * hc * wc + nearest_src(t, h, w, hc, wc)) * C4;
  float4* dst = out + (size_t)warp * C4;
  for (int c4 = lane; c4 < C4; c4 += 32) dst[c4] = __ldg(src + c4);
}


// The kept rows of a restoration (part 2) with the group fold of the column sums done inside a thread-block
// cluster: the chunks of one group are the CTAs of one cluster, every CTA sends its chunk sums to the CTA that
// owns the channel slice (distributed shared memory), and after one cluster barrier every CTA adds the chunks of
// its slice in chunk order and writes the group partial.  Same values and the same order of additions as the
// fold through global memory (chunk partial -> ticket -> last arriver), without its chain of round trips.
// grid (group * ngroups, B), cluster (group, 1, 1), 256 threads; C8 <= 256.
constexpr int kFoldEntries = 256 + 16;   // group * ceil(C8 / group) <= C8 + group
__global__ void __launch_bounds__(256) restore_kept_cluster_kernel(float4* __restrict__ x, const uint4* __restrict__ y,
                                                                   const int32_t* __restrict__ inv, const float* __restrict__ gamma,
                                                                   int mod_stride, int n, int k, int C8, int nchunks, int group, int ngroups,
                                                                   const float4* __restrict__ chunk_partial, float4* __restrict__ group_partial) {
  __shared__ const uint4* s_src[kColsumRows];
  __shared__ int s_on[kColsumRows];
  __shared__ __align__(16) float s_fold[kFoldEntries * 8];   // [chunk of the group][channel group of this CTA's slice][8]
  pdl_trigger();
  cluster_arrive_relaxed();   // first half of the start-up barrier (completed before the remote stores below)
  pdl_wait();
  const int b = blockIdx.y;
  const int rank = (int)cluster_ctarank();
  const int g = blockIdx.x / group;
  const int chunk = blockIdx.x;                     // = g * group + rank
  const bool valid = chunk < nchunks;
  const int members = min(group, nchunks - g * group);
  const int slice = (C8 + group - 1) / group;       // channel groups (of 8) per owner
  const int t0 = chunk * kColsumRows;
  const int rows = valid ? min(kColsumRows, n - t0) : 0;
  if ((int)threadIdx.x < rows) {
    const int j = __ldg(inv + (size_t)b * n + t0 + threadIdx.x);
    s_src[threadIdx.x] = y + ((size_t)b * k + max(j, 0)) * C8;
    s_on[threadIdx.x] = j >= 0;
  }
  __syncthreads();
  const int c8 = threadIdx.x;
  float4 a0 = make_float4(0.f, 0.f, 0.f, 0.f), a1 = a0;
  if (valid && c8 < C8) {
    float4 g0 = make_float4(1.f, 1.f, 1.f, 1.f), g1 = g0;
    if (gamma) {
      const float4* gp = reinterpret_cast<const float4*>(gamma + (size_t)b * mod_stride);
      g0 = __ldg(gp + 2 * c8); g1 = __ldg(gp + 2 * c8 + 1);
    }
    // continue the sums of the rows the first part updated
    const float4* cp = chunk_partial + ((size_t)b * nchunks + chunk) * C8 * 2 + 2 * c8;
    a0 = __ldcg(cp); a1 = __ldcg(cp + 1);
    float4* xbase = x + ((size_t)b * n + t0) * C8 * 2;
    for (int r = 0; r < rows; r += 4) {
      uint4 p[4];
      float4 x0[4], x1[4];
#pragma unroll
      for (int i = 0; i < 4; ++i) {
        if (r + i < rows && s_on[r + i]) {
          float4* xr = xbase + (size_t)(r + i) * C8 * 2 + 2 * c8;
          x0[i] = xr[0]; x1[i] = xr[1];
          p[i] = __ldg(s_src[r + i] + c8);
        }
      }
#pragma unroll
      for (int i = 0; i < 4; ++i) {
        if (r + i < rows && s_on[r + i]) {
          float f[8];
          bf16x8_to_float(p[i], f);
          float4 u0 = x0[i], u1 = x1[i];
          if (gamma) {
            u0.x = fmaf(g0.x, f[0], u0.x); u0.y = fmaf(g0.y, f[1], u0.y); u0.z = fmaf(g0.z, f[2], u0.z); u0.w = fmaf(g0.w, f[3], u0.w);
            u1.x = fmaf(g1.x, f[4], u1.x); u1.y = fmaf(g1.y, f[5], u1.y); u1.z = fmaf(g1.z, f[6], u1.z); u1.w = fmaf(g1.w, f[7], u1.w);
          } else {
            u0.x += f[0]; u0.y += f[1]; u0.z += f[2]; u0.w += f[3];
            u1.x += f[4]; u1.y += f[5]; u1.z += f[6]; u1.w += f[7];
          }
          float4* xr = xbase + (size_t)(r + i) * C8 * 2 + 2 * c8;
          xr[0] = u0; xr[1] = u1;
          a0.x += u0.x; a0.y += u0.y; a0.z += u0.z; a0.w += u0.w;
          a1.x += u1.x; a1.y += u1.y; a1.z += u1.z; a1.w += u1.w;
        }
      }
    }
  }
  cluster_wait();    // every CTA of the cluster has started: their shared memory may be written
  if (valid && c8 < C8) {
    // the chunk's sums of this thread's 8 channels go to the CTA that owns the channel slice
    const int owner = c8 / slice, local = c8 - owner * slice;
    uint32_t dst;
    asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(dst) : "r"(smem_u32(s_fold + ((size_t)rank * slice + local) * 8)), "r"(owner));
    asm volatile("st.shared::cluster.v4.f32 [%0], {%1, %2, %3, %4};" ::"r"(dst), "f"(a0.x), "f"(a0.y), "f"(a0.z), "f"(a0.w) : "memory");
    asm volatile("st.shared::cluster.v4.f32 [%0], {%1, %2, %3, %4};" ::"r"(dst + 16), "f"(a1.x), "f"(a1.y), "f"(a1.z), "f"(a1.w) : "memory");
  }
  cluster_sync_all();
  // this CTA's slice of the group partial: the group's chunks in chunk order
  const int lc = threadIdx.x;
  const int my_c8 = rank * slice + lc;
  if (lc < slice && my_c8 < C8) {
    float4 s0 = make_float4(0.f, 0.f, 0.f, 0.f), s1 = s0;
    for (int m = 0; m < members; ++m) {
      const float4* e = reinterpret_cast<const float4*>(s_fold + ((size_t)m * slice + lc) * 8);
      const float4 v0 = e[0], v1 = e[1];
      s0.x += v0.x; s0.y += v0.y; s0.z += v0.z; s0.w += v0.w;
      s1.x += v1.x; s1.y += v1.y; s1.z += v1.z; s1.w += v1.w;
    }
    float4* gp = group_partial + ((size_t)b * ngroups + g) * C8 * 2 + 2 * my_c8;
    gp[0] = s0; gp[1] = s1;
  }
}

// restore_residual_kernel with bilinear (TAPS 4) or bicubic (TAPS 16) interpolation of the cache: an unkept
// token blends TAPS cached rows (fp32), a kept token takes its forwarded row.  Same CTA shape, row ownership
// and column-sum handling; fewer rows in flight (two, or one with sixteen source rows).  part 2 (kept rows only) never interpolates and
// runs the kernel above.
template <int TAPS>
__global__ void __launch_bounds__(256) restore_residual_interp_kernel(float* __restrict__ xf, const uint4* __restrict__ y,
                                                                        const uint4* __restrict__ cache, const int32_t* __restrict__ inv,
                                                                        const float* __restrict__ gamma, int mod_stride, int n, int k,
                                                                        int h, int w, int hc, int wc, int C8, int nchunks, int group,
                                                                        int ngroups, float4* __restrict__ chunk_partial,
                                                                        float4* __restrict__ group_partial, unsigned int* tickets,
                                                                        int part) {
  constexpr int ROWS = TAPS == 4 ? 2 : 1;   // rows in flight per thread
  float4* x = reinterpret_cast<float4*>(xf);
  __shared__ const uint4* s_src[kColsumRows][TAPS];
  __shared__ float s_wt[kColsumRows][TAPS];
  __shared__ int s_on[kColsumRows];
  pdl_trigger();
  pdl_wait();
  const int b = blockIdx.y, chunk = blockIdx.x;
  const int t0 = chunk * kColsumRows;
  const int rows = min(kColsumRows, n - t0);
  if (threadIdx.x < rows) {
    const int t = t0 + threadIdx.x;
    const int j = __ldg(inv + (size_t)b * n + t);
    if (j >= 0) {
      for (int q = 0; q < TAPS; ++q) { s_src[threadIdx.x][q] = y + ((size_t)b * k + j) * C8; s_wt[threadIdx.x][q] = q == 0 ? 1.f : 0.f; }
    } else {
      const InterpTaps<TAPS> bt = interp_taps<TAPS>(t, h, w, hc, wc);
      for (int q = 0; q < TAPS; ++q) { s_src[threadIdx.x][q] = cache + ((size_t)b * hc * wc + bt.src[q]) * C8; s_wt[threadIdx.x][q] = bt.wt[q]; }
    }
    s_on[threadIdx.x] = part == 0 || (part == 1 || part == 3) == (j < 0);
  }
  __syncthreads();
  float4* xbase = x + ((size_t)b * n + t0) * C8 * 2;
  for (int c8 = threadIdx.x; c8 < C8; c8 += 256) {
    float4 g0 = make_float4(1.f, 1.f, 1.f, 1.f), g1 = g0;
    if (gamma) {
      const float4* g = reinterpret_cast<const float4*>(gamma + (size_t)b * mod_stride);
      g0 = __ldg(g + 2 * c8); g1 = __ldg(g + 2 * c8 + 1);
    }
    float4 a0 = make_float4(0.f, 0.f, 0.f, 0.f), a1 = a0;
    for (int r = 0; r < rows; r += ROWS) {
      uint4 p[ROWS][TAPS];
      float4 x0[ROWS], x1[ROWS];
#pragma unroll
      for (int i = 0; i < ROWS; ++i) {
        if (r + i < rows && s_on[r + i]) {
          float4* xr = xbase + (size_t)(r + i) * C8 * 2 + 2 * c8;
          x0[i] = xr[0]; x1[i] = xr[1];
#pragma unroll
          for (int q = 0; q < TAPS; ++q) p[i][q] = __ldg(s_src[r + i][q] + c8);
        }
      }
#pragma unroll
      for (int i = 0; i < ROWS; ++i) {
        if (r + i < rows && s_on[r + i]) {
          float f[8] = {0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f};
#pragma unroll
          for (int q = 0; q < TAPS; ++q) {
            float fq[8];
            bf16x8_to_float(p[i][q], fq);
            const float wq = s_wt[r + i][q];
#pragma unroll
            for (int e = 0; e < 8; ++e) f[e] = fmaf(wq, fq[e], f[e]);
          }
          float4 u0 = x0[i], u1 = x1[i];
          u0.x = fmaf(g0.x, f[0], u0.x); u0.y = fmaf(g0.y, f[1], u0.y); u0.z = fmaf(g0.z, f[2], u0.z); u0.w = fmaf(g0.w, f[3], u0.w);
          u1.x = fmaf(g1.x, f[4], u1.x); u1.y = fmaf(g1.y, f[5], u1.y); u1.z = fmaf(g1.z, f[6], u1.z); u1.w = fmaf(g1.w, f[7], u1.w);
          float4* xr = xbase + (size_t)(r + i) * C8 * 2 + 2 * c8;
          xr[0] = u0; xr[1] = u1;
          a0.x += u0.x; a0.y += u0.y; a0.z += u0.z; a0.w += u0.w;
          a1.x += u1.x; a1.y += u1.y; a1.z += u1.z; a1.w += u1.w;
        }
      }
    }
    if (chunk_partial) {
      float4* cp = chunk_partial + ((size_t)b * nchunks + chunk) * C8 * 2 + 2 * c8;
      cp[0] = a0; cp[1] = a1;
    }
  }
  if (chunk_partial && part != 1)
    fold_group_partials(b, chunk, nchunks, group, ngroups, C8 * 2, chunk_partial, group_partial, tickets);
}

// Plain restoration (no residual) with bilinear / bicubic interpolation, one warp per output row; bf16 rows
// (8 per uint4, blended in fp32 and rounded once) or fp32 rows.
template <int TAPS>
__global__ void __launch_bounds__(256) restore_bf16_interp_kernel(const uint4* __restrict__ cache, int hc, int wc,
                                                                    const uint4* __restrict__ pivots, const int32_t* __restrict__ inv,
                                                                    int n, int k, int h, int w, int C8, uint4* __restrict__ out,
                                                                    int total_rows) {
  pdl_trigger();
  pdl_wait();
  const int warp = (blockIdx.x * blockDim.x + threadIdx.x) >> 5, lane = threadIdx.x & 31;
  if (warp >= total_rows) return;
  const int b = warp / n, t = warp - b * n;
  const int j = inv[warp];
  uint4* dst = out + (size_t)warp * C8;
  if (j >= 0) {
    const uint4* src = pivots + ((size_t)b * k + j) * C8;
    for (int c8 = lane; c8 < C8; c8 += 32) dst[c8] = __ldg(src + c8);
    return;
  }
  const InterpTaps<TAPS> bt = interp_taps<TAPS>(t, h, w, hc, wc);
  const uint4* base = cache + (size_t)b * hc * wc * C8;
  for (int c8 = lane; c8 < C8; c8 += 32) {
    float f[8] = {0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f};
#pragma unroll
    for (int q = 0; q < TAPS; ++q) {
      float fq[8];
      bf16x8_to_float(__ldg(base + (size_t)bt.src[q] * C8 + c8), fq);
#pragma unroll
      for (int e = 0; e < 8; ++e) f[e] = fmaf(bt.wt[q], fq[e], f[e]);
    }
    __nv_bfloat162 o[4] = {__floats2bfloat162_rn(f[0], f[1]), __floats2bfloat162_rn(f[2], f[3]), __floats2bfloat162_rn(f[4], f[5]),
                           __floats2bfloat162_rn(f[6], f[7])};
    dst[c8] = *reinterpret_cast<uint4*>(o);
  }
}

template <int TAPS>
__global__ void __launch_bounds__(256) restore_rows_f32_interp_kernel(const float4* __restrict__ cache, int hc, int wc,
                                                                        const float4* __restrict__ pivots, const int32_t* __restrict__ inv,
                                                                        int n, int k, int h, int w, int C4, float4* __restrict__ out,
                                                                        int total_rows) {
  pdl_trigger();
  pdl_wait();
  const int warp = (blockIdx.x * blockDim.x + threadIdx.x) >> 5, lane = threadIdx.x & 31;
  if (warp >= total_rows) return;
  const int b = warp / n, t = warp - b * n;
  const int j = __ldg(inv + warp);
  float4* dst = out + (size_t)warp * C4;
  if (j >= 0) {
    const float4* src = pivots + ((size_t)b * k + j) * C4;
    for (int c4 = lane; c4 < C4; c4 += 32) dst[c4] = __ldg(src + c4);
    return;
  }
  const InterpTaps<TAPS> bt = interp_taps<TAPS>(t, h, w, hc, wc);
  const float4* base = cache + (size_t)b * hc * wc * C4;
  for (int c4 = lane; c4 < C4; c4 += 32) {
    float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
    for (int q = 0; q < TAPS; ++q) {
      const float4 v = __ldg(base + (size_t)bt.src[q] * C4 + c4);
      acc.x = fmaf(bt.wt[q], v.x, acc.x); acc.y = fmaf(bt.wt[q], v.y, acc.y); acc.z = fmaf(bt.wt[q], v.z, acc.z); acc.w = fmaf(bt.wt[q], v.w, acc.w);
    }
    dst[c4] = acc;
  }
}

// (cos, sin) of the rotary angles of every token of one scale; double precision (a few hundred thousand
// evaluations per scale, once per context).
__global__ void rope_table_kernel(float2* __restrict__ table, int h, int w, int h_last, int w_last, int half, double log2_base) {
  const long total = (long)h * w * half;
  const int quarter = half / 2;
  for (long i = (long)blockIdx.x * blockDim.x + threadIdx.x; i < total; i += (long)gridDim.x * blockDim.x) {
    const int j = (int)(i % half);
    const int t = (int)(i / half);
    const int y = t / w, x = t - y * w;
    const double pos = j < quarter ? (double)y * h_last / h : (double)x * w_last / w;
    const double omega = exp2(-(double)(j % quarter) / quarter * log2_base);
    double sn, cs;
    sincos(pos * omega, &sn, &cs);
    table[i] = make_float2((float)cs, (float)sn);
  }
}
// One warp waits on an mbarrier that nothing arrives at: the wait expires after limit_ns and the code is recorded.
__global__ void expired_wait_kernel(int32_t* status, unsigned long long limit_ns) {
  __shared__ uint64_t bar;
  if (threadIdx.x == 0) { mbar_init(&bar, 1); mbar_fence_init(); }
  __syncwarp();
  if (threadIdx.x == 0 && !mbar_wait(&bar, 0, limit_ns)) atomicCAS(status, 0, DEV_TIMEOUT_SELFTEST);
}
}  // namespace

cudaError_t launch_expired_wait(int32_t* status, unsigned long long limit_ns, cudaStream_t st) {
  expired_wait_kernel<<<1, 32, 0, st>>>(status, limit_ns);
  return cudaGetLastError();
}

// How the kept-row part of a restoration folds its column sums: 0 by shape, 1 global memory, 2 clusters.
static int g_fold_mode = 0;
static bool g_cluster_fold_ok = false;
static int g_rows_sms = 148;
void restore_force_fold(int mode) { g_fold_mode = mode; }
cudaError_t rows_init() {
  g_cluster_fold_ok = cudaFuncSetAttribute(restore_kept_cluster_kernel, cudaFuncAttributeNonPortableClusterSizeAllowed, 1) == cudaSuccess;
  (void)cudaGetLastError();
  int dev = 0;
  if (cudaGetDevice(&dev) == cudaSuccess) (void)cudaDeviceGetAttribute(&g_rows_sms, cudaDevAttrMultiProcessorCount, dev);
  return cudaSuccess;
}

cudaError_t launch_gather_ln(const void* x, const int32_t* idx, int B, int n, int k, int C, const float* sigma,
                             const float* beta, int mod_stride, void* a_out, int32_t* status, cudaStream_t st, bool x_bf16) {
  const int rows = B * k;
  const double bytes = (double)rows * C * (x_bf16 ? 4.0 : 6.0);
  LaunchScope scope(KC_GATHER_LN, 1, bytes, bytes, st);
  if (x_bf16)
    return launch_pdl(gather_ln_kernel<__nv_bfloat16>, dim3((k + 7) / 8, B), dim3(256), sigma ? (size_t)C * 8 : 0, st,
                      static_cast<const __nv_bfloat16*>(x), idx, n, k, C / 4, sigma, beta, mod_stride, reinterpret_cast<uint2*>(a_out), status);
  return launch_pdl(gather_ln_kernel<float>, dim3((k + 7) / 8, B), dim3(256), sigma ? (size_t)C * 8 : 0, st, static_cast<const float*>(x),
                    idx, n, k, C / 4, sigma, beta, mod_stride, reinterpret_cast<uint2*>(a_out), status);
}

cudaError_t launch_restore_residual(void* x, const void* y, const void* cache, const int32_t* inv, const float* gamma,
                                    int mod_stride, int B, int k, int h, int w, int hc, int wc, int C, void* colsum_ws,
                                    int part, int interp_mode, cudaStream_t st, bool x_bf16) {
  const int n = h * w;
  SelectWs ws{};
  if (colsum_ws) ws = select_ws_carve(colsum_ws, B, n, C);
  const int nchunks = (n + kColsumRows - 1) / kColsumRows;
  // algorithmic bytes of the part: x read + written for its rows, its source rows
  const bool unkept_only = part == 1 || part == 3;
  const double rows_x = part == 0 ? (double)n : (unkept_only ? (double)(n - k) : (double)k);
  const double rr_bytes = (double)B * C * ((x_bf16 ? 4.0 : 8.0) * rows_x + (!unkept_only ? 2.0 * k : 0.0) + (part != 2 ? 2.0 * hc * wc : 0.0));
  LaunchScope scope(KC_RESTORE, 1, rr_bytes, rr_bytes, st);
  if (x_bf16) {   // bf16 residual stream: the generic kernel (nearest interpolation, fold through global memory)
    if (interp_mode != 0) return cudaErrorNotSupported;
    restore_residual_kernel<__nv_bfloat16, 4><<<dim3(nchunks, B), 256, 0, st>>>(
        static_cast<__nv_bfloat16*>(x), reinterpret_cast<const uint4*>(y), reinterpret_cast<const uint4*>(cache), inv, gamma, mod_stride, n, k, h, w,
        hc, wc, C / 8, nchunks, ws.group, ws.ngroups, reinterpret_cast<float4*>(ws.chunk_partial), reinterpret_cast<float4*>(ws.group_partial),
        ws.tickets, part);
    return cudaGetLastError();
  }
  // kept rows + group fold inside clusters (one cluster per group of chunks) where the group fits a cluster
  if (part == 2 && colsum_ws && g_cluster_fold_ok && g_fold_mode != 1 && ws.group >= 1 && ws.group <= 8 && C / 8 <= 256) {
    cudaLaunchConfig_t cfg{};
    cfg.gridDim = dim3(ws.group * ws.ngroups, B); cfg.blockDim = dim3(256); cfg.dynamicSmemBytes = 0; cfg.stream = st;
    cudaLaunchAttribute at[1];
    at[0].id = cudaLaunchAttributeClusterDimension;
    at[0].val.clusterDim.x = ws.group; at[0].val.clusterDim.y = 1; at[0].val.clusterDim.z = 1;
    cfg.attrs = at; cfg.numAttrs = 1;
    const cudaError_t e = cudaLaunchKernelEx(&cfg, restore_kept_cluster_kernel, reinterpret_cast<float4*>(x), reinterpret_cast<const uint4*>(y),
                                             inv, gamma, mod_stride, n, k, C / 8, nchunks, ws.group, ws.ngroups,
                                             reinterpret_cast<const float4*>(ws.chunk_partial), reinterpret_cast<float4*>(ws.group_partial));
    if (e == cudaSuccess || g_fold_mode == 2) return e;
    (void)cudaGetLastError();      // this cluster size cannot be scheduled here: the fold through global memory instead
  }
  // more chunks than three CTAs per SM hold at once (the 128 x 128 map): the kept-row part takes the build that fits four
  const bool small_build = part != 0 && (long)nchunks * B > 3L * g_rows_sms && (long)nchunks * B <= 4L * g_rows_sms;
  auto* kern = (interp_mode == 0 || part == 2) ? (small_build ? restore_residual_kernel<float, 2> : restore_residual_kernel<float, 4>)
               : (interp_mode == 1 ? restore_residual_interp_kernel<4> : restore_residual_interp_kernel<16>);
  if (part == 0)
    return launch_pdl(kern, dim3(nchunks, B), dim3(256), 0, st, static_cast<float*>(x),
                      reinterpret_cast<const uint4*>(y), reinterpret_cast<const uint4*>(cache), inv, gamma, mod_stride, n, k, h, w, hc, wc,
                      C / 8, nchunks, ws.group, ws.ngroups, reinterpret_cast<float4*>(ws.chunk_partial),
                      reinterpret_cast<float4*>(ws.group_partial), ws.tickets, part);
  // The two halves of a split restoration are ordered against another stream by events: they are
  // launched as ordinary stream work, not as programmatic dependents.
  kern<<<dim3(nchunks, B), 256, 0, st>>>(static_cast<float*>(x), reinterpret_cast<const uint4*>(y),
                                         reinterpret_cast<const uint4*>(cache), inv, gamma, mod_stride, n, k, h, w, hc, wc, C / 8, nchunks,
                                         ws.group, ws.ngroups, reinterpret_cast<float4*>(ws.chunk_partial),
                                         reinterpret_cast<float4*>(ws.group_partial), ws.tickets, part);
  return cudaGetLastError();
}

cudaError_t launch_restore_bf16(const void* cache, int hc, int wc, const void* pivots, const int32_t* inv, int B, int k,
                                int h, int w, int C, void* out, int interp_mode, cudaStream_t st) {
  const int rows = B * h * w;
  const double rb_bytes = (double)B * C * (2.0 * h * w + 2.0 * k + 2.0 * hc * wc);
  LaunchScope scope(KC_RESTORE, 1, rb_bytes, rb_bytes, st);
  return launch_pdl(interp_mode == 0 ? restore_bf16_kernel : (interp_mode == 1 ? restore_bf16_interp_kernel<4> : restore_bf16_interp_kernel<16>), dim3((rows + 7) / 8), dim3(256), 0, st, reinterpret_cast<const uint4*>(cache), hc, wc,
                    reinterpret_cast<const uint4*>(pivots), inv, h * w, k, h, w, C / 8, reinterpret_cast<uint4*>(out), rows);
}

cudaError_t launch_gather_rows(const float* x, const int32_t* idx, int B, int n, int k, int C, float* out, int32_t* status, cudaStream_t st) {
  LaunchScope scope(KC_GATHER_LN, 1, (double)B * k * C * 8.0, (double)B * k * C * 8.0, st);
  return launch_pdl(gather_rows_kernel, dim3((k + 7) / 8, B), dim3(256), 0, st, reinterpret_cast<const float4*>(x), idx, n, k, C / 4,
                    reinterpret_cast<float4*>(out), status);
}

cudaError_t launch_restore_rows_f32(const float* cache, int hc, int wc, const float* pivots, const int32_t* inv, int B, int k,
                                    int h, int w, int C, float* out, int interp_mode, cudaStream_t st) {
  const int rows = B * h * w;
  const double bytes = (double)B * C * 4.0 * ((double)h * w + k + (double)hc * wc);
  LaunchScope scope(KC_RESTORE, 1, bytes, bytes, st);
  return launch_pdl(interp_mode == 0 ? restore_rows_f32_kernel
                                     : (interp_mode == 1 ? restore_rows_f32_interp_kernel<4> : restore_rows_f32_interp_kernel<16>), dim3((rows + 7) / 8), dim3(256), 0, st, reinterpret_cast<const float4*>(cache), hc, wc,
                    reinterpret_cast<const float4*>(pivots), inv, h * w, k, h, w, C / 4, reinterpret_cast<float4*>(out), rows);
}

cudaError_t launch_rope_table(float* table, int h, int w, int h_last, int w_last, int head_dim, float base, cudaStream_t st) {
  const long total = (long)h * w * (head_dim / 2);
  const long blocks = (total + 255) / 256;
  rope_table_kernel<<<(unsigned)(blocks < 4096 ? blocks : 4096), 256, 0, st>>>(reinterpret_cast<float2*>(table), h, w, h_last, w_last,
                                                                                head_dim / 2, log2((double)base));
  return cudaGetLastError();
}

}  // namespace fv
