// Device-side pieces shared by the GEMM kernels: the argument block and the fused epilogues (bias, GELU,
// gate + residual with the sublayer-cache copy, and the Q | K-cache | V^T-cache split of the QKV projection).
#pragma once
#include <cuda_bf16.h>

#include "internal.h"
#include "sm100.cuh"

namespace fv {
namespace gemm_detail {

struct GemmDev {
  const __nv_bfloat16* bias;
  int M, N, K;
  int epilogue;
  void* out;
  void* aux;
  const float* gamma;
  int mod_stride, rows_per_image;
  int q_cols, C;
  __nv_bfloat16* k_cache;
  __nv_bfloat16* vt_cache;
  int kv_capacity, kv_offset;
  int32_t* status;
  int splits, kb_per_split;   // K slices per tile (1 = no split) and 64-wide k-blocks per slice
  float* sk_partial;          // [tile][slice][128][BN] fp32 partial accumulators
  unsigned int* sk_tickets;   // [tile] arrival counters, zero between launches
};

__device__ __forceinline__ float gelu_tanh_fast(float v) {
  const float u = 0.7978845608028654f * fmaf(0.044715f * v * v, v, v);
  float t;
  asm("tanh.approx.f32 %0, %1;" : "=f"(t) : "f"(u));
  return 0.5f * v * (1.f + t);
}

__device__ __forceinline__ void report(int32_t* status, int code) {
  if (status) atomicCAS(status, 0, code);
}

// One 32-column chunk of one accumulator row: bias, optional GELU, then the epilogue's store.
__device__ __forceinline__ void epilogue_chunk(const GemmDev& p, const uint32_t (&r)[32], int row, int img, int jrow, int col) {
  float v[32];
  if (p.bias) {
    const uint4* bp = reinterpret_cast<const uint4*>(p.bias + col);
#pragma unroll
    for (int g = 0; g < 4; ++g) {
      if (col + 8 * g < p.N) {
        uint4 bb = __ldg(bp + g);
        const uint32_t u[4] = {bb.x, bb.y, bb.z, bb.w};
#pragma unroll
        for (int i = 0; i < 4; ++i) {
          v[8 * g + 2 * i] = __uint_as_float(r[8 * g + 2 * i]) + __uint_as_float(u[i] << 16);
          v[8 * g + 2 * i + 1] = __uint_as_float(r[8 * g + 2 * i + 1]) + __uint_as_float(u[i] & 0xFFFF0000u);
        }
      } else {
#pragma unroll
        for (int i = 0; i < 8; ++i) v[8 * g + i] = 0.f;
      }
    }
  } else {
#pragma unroll
    for (int i = 0; i < 32; ++i) v[i] = __uint_as_float(r[i]);
  }
  if (p.epilogue == EPI_GELU_BF16) {
#pragma unroll
    for (int i = 0; i < 32; ++i) v[i] = gelu_tanh_fast(v[i]);
  }
  if (p.epilogue == EPI_BF16 || p.epilogue == EPI_GELU_BF16 || (p.epilogue == EPI_QKV_SPLIT && col < p.q_cols)) {
    const int ld = (p.epilogue == EPI_QKV_SPLIT) ? p.q_cols : p.N;
    uint4* dst = reinterpret_cast<uint4*>(static_cast<__nv_bfloat16*>(p.out) + (size_t)row * ld + col);
#pragma unroll
    for (int g = 0; g < 4; ++g) {
      if (col + 8 * g < p.N) {
        uint4 o;
        o.x = pack_bf16x2(v[8 * g + 0], v[8 * g + 1]); o.y = pack_bf16x2(v[8 * g + 2], v[8 * g + 3]);
        o.z = pack_bf16x2(v[8 * g + 4], v[8 * g + 5]); o.w = pack_bf16x2(v[8 * g + 6], v[8 * g + 7]);
        dst[g] = o;
      }
    }
  } else if (p.epilogue == EPI_RESIDUAL) {
    float4* xr = reinterpret_cast<float4*>(static_cast<float*>(p.out) + (size_t)row * p.N + col);
    const float4* gp = p.gamma ? reinterpret_cast<const float4*>(p.gamma + (size_t)img * p.mod_stride + col) : nullptr;
    uint4* ap = p.aux ? reinterpret_cast<uint4*>(static_cast<__nv_bfloat16*>(p.aux) + (size_t)row * p.N + col) : nullptr;
#pragma unroll
    for (int g = 0; g < 8; ++g) {
      if (col + 4 * g < p.N) {
        float4 xv = xr[g];
        if (gp) {
          float4 gg = __ldg(gp + g);
          xv.x = fmaf(gg.x, v[4 * g + 0], xv.x); xv.y = fmaf(gg.y, v[4 * g + 1], xv.y);
          xv.z = fmaf(gg.z, v[4 * g + 2], xv.z); xv.w = fmaf(gg.w, v[4 * g + 3], xv.w);
        } else {
          xv.x += v[4 * g + 0]; xv.y += v[4 * g + 1]; xv.z += v[4 * g + 2]; xv.w += v[4 * g + 3];
        }
        xr[g] = xv;
      }
    }
    if (ap) {
#pragma unroll
      for (int g = 0; g < 4; ++g) {
        if (col + 8 * g < p.N) {
          uint4 o;
          o.x = pack_bf16x2(v[8 * g + 0], v[8 * g + 1]); o.y = pack_bf16x2(v[8 * g + 2], v[8 * g + 3]);
          o.z = pack_bf16x2(v[8 * g + 4], v[8 * g + 5]); o.w = pack_bf16x2(v[8 * g + 6], v[8 * g + 7]);
          ap[g] = o;
        }
      }
    }
  } else {  // EPI_QKV_SPLIT, K or V part
    const int kc = col - p.q_cols;
    const size_t krow = (size_t)img * p.kv_capacity + p.kv_offset + jrow;
    if (kc < p.C) {
      uint4* dst = reinterpret_cast<uint4*>(p.k_cache + krow * p.C + kc);
#pragma unroll
      for (int g = 0; g < 4; ++g) {
        uint4 o;
        o.x = pack_bf16x2(v[8 * g + 0], v[8 * g + 1]); o.y = pack_bf16x2(v[8 * g + 2], v[8 * g + 3]);
        o.z = pack_bf16x2(v[8 * g + 4], v[8 * g + 5]); o.w = pack_bf16x2(v[8 * g + 6], v[8 * g + 7]);
        dst[g] = o;
      }
    } else {
      // V is kept transposed ([image, channel, key]) so that P*V reads it K-major; for a fixed
      // channel the 32 lanes write 32 consecutive keys.
      __nv_bfloat16* dst = p.vt_cache + ((size_t)img * p.C + (kc - p.C)) * p.kv_capacity + p.kv_offset + jrow;
#pragma unroll
      for (int i = 0; i < 32; ++i) dst[(size_t)i * p.kv_capacity] = __float2bfloat16_rn(v[i]);
    }
  }
}

}  // namespace gemm_detail

// gemm_pair.cu: the CTA-pair kernel (256 x bn tiles, bn in {128, 256}); same argument block and epilogues.
cudaError_t gemm_pair_init();
cudaError_t launch_gemm_pair(const GemmArgs& g, const gemm_detail::GemmDev& p, int bn, cudaStream_t st);

}  // namespace fv
