// Row-wise HBM-bound kernels of the pruned step:
//   gather_ln        : Algorithm 1's gather of the kept rows fused with the block's pre-LayerNorm and
//                      AdaLN modulation; writes the bf16 A operand of the following GEMM.
//   restore_residual : Cached Token Restoration (Eq. 6, Algorithm 1 second routine) written as a
//                      gather through the inverse index map (no scatter, so no write races), fused
//                      with the gate and the residual add.
//   restore_bf16     : the plain restoration, bf16 in / bf16 out, bit-exact copy.
// One warp owns one token row; every global access is a 128-bit vector, consecutive lanes touching
// consecutive 16-byte words.
#include <cuda_bf16.h>

#include "internal.h"

namespace fv {

namespace {

constexpr int kMaxVec = 16;  // float4 per lane -> C <= 2048

__global__ void __launch_bounds__(256) gather_ln_kernel(const float4* __restrict__ x, const int32_t* __restrict__ idx, int n,
                                                        int k, int C4, const float* __restrict__ sigma,
                                                        const float* __restrict__ beta, int mod_stride,
                                                        uint2* __restrict__ a_out, int total_rows) {
  const int warp = (blockIdx.x * blockDim.x + threadIdx.x) >> 5, lane = threadIdx.x & 31;
  if (warp >= total_rows) return;
  const int b = warp / k, j = warp - b * k;
  const int t = idx ? idx[warp] : j;
  const float4* row = x + ((size_t)b * n + t) * C4;
  float4 v[kMaxVec];
  float sum = 0.f;
#pragma unroll
  for (int i = 0; i < kMaxVec; ++i) {
    const int c4 = lane + 32 * i;
    if (c4 < C4) {
      v[i] = __ldg(row + c4);
      sum += (v[i].x + v[i].y) + (v[i].z + v[i].w);
    }
  }
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
  const float4* sg = sigma ? reinterpret_cast<const float4*>(sigma + (size_t)b * mod_stride) : nullptr;
  const float4* bt = beta ? reinterpret_cast<const float4*>(beta + (size_t)b * mod_stride) : nullptr;
  uint2* dst = a_out + (size_t)warp * C4;
#pragma unroll
  for (int i = 0; i < kMaxVec; ++i) {
    const int c4 = lane + 32 * i;
    if (c4 < C4) {
      float4 a;
      a.x = (v[i].x - mu) * rstd; a.y = (v[i].y - mu) * rstd; a.z = (v[i].z - mu) * rstd; a.w = (v[i].w - mu) * rstd;
      if (sg) {
        float4 s = __ldg(sg + c4), bb = __ldg(bt + c4);
        a.x = fmaf(a.x, 1.f + s.x, bb.x); a.y = fmaf(a.y, 1.f + s.y, bb.y);
        a.z = fmaf(a.z, 1.f + s.z, bb.z); a.w = fmaf(a.w, 1.f + s.w, bb.w);
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

__device__ __forceinline__ void bf16x8_to_float(const uint4& p, float (&f)[8]) {
  const uint32_t u[4] = {p.x, p.y, p.z, p.w};
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    f[2 * i] = __uint_as_float(u[i] << 16);
    f[2 * i + 1] = __uint_as_float(u[i] & 0xFFFF0000u);
  }
}

// x[b,t,:] += gamma[b,:] * (inv[b,t] >= 0 ? y[b*k + inv[b,t], :] : cache[b, src(t), :])
__global__ void __launch_bounds__(256) restore_residual_kernel(float4* __restrict__ x, const uint4* __restrict__ y,
                                                               const uint4* __restrict__ cache, const int32_t* __restrict__ inv,
                                                               const float* __restrict__ gamma, int mod_stride, int n, int k,
                                                               int h, int w, int hc, int wc, int C8, int total_rows) {
  const int warp = (blockIdx.x * blockDim.x + threadIdx.x) >> 5, lane = threadIdx.x & 31;
  if (warp >= total_rows) return;
  const int b = warp / n, t = warp - b * n;
  const int j = inv[warp];
  const uint4* src = (j >= 0) ? y + ((size_t)b * k + j) * C8
                              : cache + ((size_t)b * hc * wc + nearest_src(t, h, w, hc, wc)) * C8;
  float4* xr = x + (size_t)warp * C8 * 2;
  const float4* g = gamma ? reinterpret_cast<const float4*>(gamma + (size_t)b * mod_stride) : nullptr;
  for (int c8 = lane; c8 < C8; c8 += 32) {
    float f[8];
    bf16x8_to_float(__ldg(src + c8), f);
    float4 x0 = xr[2 * c8], x1 = xr[2 * c8 + 1];
    if (g) {
      float4 g0 = __ldg(g + 2 * c8), g1 = __ldg(g + 2 * c8 + 1);
      x0.x = fmaf(g0.x, f[0], x0.x); x0.y = fmaf(g0.y, f[1], x0.y); x0.z = fmaf(g0.z, f[2], x0.z); x0.w = fmaf(g0.w, f[3], x0.w);
      x1.x = fmaf(g1.x, f[4], x1.x); x1.y = fmaf(g1.y, f[5], x1.y); x1.z = fmaf(g1.z, f[6], x1.z); x1.w = fmaf(g1.w, f[7], x1.w);
    } else {
      x0.x += f[0]; x0.y += f[1]; x0.z += f[2]; x0.w += f[3];
      x1.x += f[4]; x1.y += f[5]; x1.z += f[6]; x1.w += f[7];
    }
    xr[2 * c8] = x0;
    xr[2 * c8 + 1] = x1;
  }
}

__global__ void __launch_bounds__(256) restore_bf16_kernel(const uint4* __restrict__ cache, int hc, int wc,
                                                           const uint4* __restrict__ pivots, const int32_t* __restrict__ inv,
                                                           int n, int k, int h, int w, int C8, uint4* __restrict__ out,
                                                           int total_rows) {
  const int warp = (blockIdx.x * blockDim.x + threadIdx.x) >> 5, lane = threadIdx.x & 31;
  if (warp >= total_rows) return;
  const int b = warp / n, t = warp - b * n;
  const int j = inv[warp];
  const uint4* src = (j >= 0) ? pivots + ((size_t)b * k + j) * C8
                              : cache + ((size_t)b * hc * wc + nearest_src(t, h, w, hc, wc)) * C8;
  uint4* dst = out + (size_t)warp * C8;
  for (int c8 = lane; c8 < C8; c8 += 32) dst[c8] = __ldg(src + c8);
}

}  // namespace

cudaError_t launch_gather_ln(const float* x, const int32_t* idx, int B, int n, int k, int C, const float* sigma,
                             const float* beta, int mod_stride, void* a_out, cudaStream_t st) {
  const int rows = B * k;
  const int blocks = (rows + 7) / 8;
  LaunchScope scope(KC_GATHER_LN, 1, (double)rows * C * 6.0, st);
  gather_ln_kernel<<<blocks, 256, 0, st>>>(reinterpret_cast<const float4*>(x), idx, n, k, C / 4, sigma, beta, mod_stride,
                                           reinterpret_cast<uint2*>(a_out), rows);
  return cudaGetLastError();
}

cudaError_t launch_restore_residual(float* x, const void* y, const void* cache, const int32_t* inv, const float* gamma,
                                    int mod_stride, int B, int k, int h, int w, int hc, int wc, int C, cudaStream_t st) {
  const int rows = B * h * w;
  LaunchScope scope(KC_RESTORE, 1, (double)B * C * (8.0 * h * w + 2.0 * k + 2.0 * hc * wc), st);
  restore_residual_kernel<<<(rows + 7) / 8, 256, 0, st>>>(reinterpret_cast<float4*>(x), reinterpret_cast<const uint4*>(y),
                                                          reinterpret_cast<const uint4*>(cache), inv, gamma, mod_stride,
                                                          h * w, k, h, w, hc, wc, C / 8, rows);
  return cudaGetLastError();
}

cudaError_t launch_restore_bf16(const void* cache, int hc, int wc, const void* pivots, const int32_t* inv, int B, int k,
                                int h, int w, int C, void* out, cudaStream_t st) {
  const int rows = B * h * w;
  LaunchScope scope(KC_RESTORE, 1, (double)B * C * (2.0 * h * w + 2.0 * k + 2.0 * hc * wc), st);
  restore_bf16_kernel<<<(rows + 7) / 8, 256, 0, st>>>(reinterpret_cast<const uint4*>(cache), hc, wc,
                                                      reinterpret_cast<const uint4*>(pivots), inv, h * w, k, h, w, C / 8,
                                                      reinterpret_cast<uint4*>(out), rows);
  return cudaGetLastError();
}

}  // namespace fv
