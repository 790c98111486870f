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
  // EPI_QKV_SPLIT extras on the Q and K columns (the instantiation of their own, KIND 2):
  const float* qk_scale;      // [H] per-head query scale of cosine attention (q, k divided by their norm), or null
  const float2* rope_table;   // [tokens of the scale][head_dim / 2] (cos, sin), or null
  const int32_t* rope_idx;    // [B, rows_per_image] original token index of every row, or null (row j = token j)
  int head_dim;
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

// The epilogue warps copy the bias slice of a tile (BN bf16 <= 512 bytes) into shared memory while they wait
// for its accumulator, so that no chunk stalls on a global load of 64 bytes of bias.
constexpr int kBiasSmemBytes = 4 * 512;   // one slice per epilogue warp
__device__ __forceinline__ void stage_bias(const GemmDev& p, uint4* bias_w, int lane, int n0, int bn) {
  if (p.bias && lane * 8 < bn && n0 + lane * 8 < p.N) bias_w[lane] = __ldg(reinterpret_cast<const uint4*>(p.bias + n0) + lane);
  __syncwarp();
}

// acc + bias (+ GELU) of one 32-column chunk of one accumulator row; bias4 = the chunk's 32 bias values
// in shared memory (ignored when the GEMM has no bias).
__device__ __forceinline__ void chunk_values(const GemmDev& p, const uint32_t (&r)[32], int col, float (&v)[32], const uint4* bias4) {
  if (p.bias) {
#pragma unroll
    for (int g = 0; g < 4; ++g) {
      if (col + 8 * g < p.N) {
        uint4 bb = bias4[g];
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
}

// ---- residual epilogue: out[row, :] += gamma[image of row] * (acc + bias), fp32 in place (+ bf16 copy);
// also the plain fp32 result (EPI_F32: out = acc + bias, gamma and aux unused) ----
// The accumulator comes out of TMEM one row per thread; read-modify-writing the fp32 stream that way would
// touch 32 different rows per instruction.  Each 32 x 32 chunk is therefore turned through the warp's
// shared-memory tile (row pitch 36 floats: conflict-free both ways) so that lane l works on columns
// 4 * (l & 7) .. +3 of rows (l >> 3) + 4 * i, i = 0..7: 8 lanes cover the 128 contiguous bytes of one row, and
// a lane's column group is the same for all its rows, so the gate is one float4 per chunk.  One warp issues
// the whole epilogue of its 32 rows with nothing to hide its instruction latencies behind, so the number
// of instructions per chunk is what bounds it (measured: taking the loads and stores out changed nothing):
// everything that does not depend on the chunk (row validity, the image boundary, the row pointers) is
// set up once per tile.
constexpr int kResidTilePitch = 36;
constexpr int kResidSmemBytes = 4 * 32 * kResidTilePitch * 4;   // one tile per epilogue warp

struct ResidRows {
  float* out0;             // &out[first row of the lane, 4 * (lane & 7)] (column offset of the chunk not included)
  __nv_bfloat16* aux0;     // same position in the bf16 copy, or nullptr
  const float* gam0;       // gate vector of the image of the warp's first row (+ the lane's column offset), or nullptr
  const float* gam1;       // gate vector of the next image
  int n_rows;              // the lane's rows i < n_rows exist
  int n_load;              // ... and are read before they are written (n_rows, or 0 for the plain fp32 result: a
                           // count, not a branch, so that the reads stay plain predicated loads issued together)
  int n_first;             // the lane's rows i < n_first belong to the first image, the others to the next one
};

// Valid when an image has at least 32 rows (a warp's 32 rows then span at most two images).
__device__ __forceinline__ ResidRows resid_rows(const GemmDev& p, int lane, int row0) {
  ResidRows rr;
  const int r = row0 + (lane >> 3);
  const int cl = 4 * (lane & 7);
  rr.out0 = static_cast<float*>(p.out) + (size_t)r * p.N + cl;
  rr.aux0 = p.aux ? static_cast<__nv_bfloat16*>(p.aux) + (size_t)r * p.N + cl : nullptr;
  rr.n_rows = max(0, min(8, (p.M - r + 3) >> 2));
  rr.n_load = p.epilogue == EPI_F32 ? 0 : rr.n_rows;
  const int img0 = min(row0, p.M - 1) / p.rows_per_image;
  rr.n_first = max(0, min(8, ((img0 + 1) * p.rows_per_image - r + 3) >> 2));
  rr.gam0 = p.gamma ? p.gamma + (size_t)img0 * p.mod_stride + cl : nullptr;
  rr.gam1 = p.gamma ? rr.gam0 + p.mod_stride : nullptr;
  return rr;
}

// The lane's 8 float4 of `out` for the chunk at column `col`; fetched one chunk ahead of its use.
__device__ __forceinline__ void residual_load_x(const GemmDev& p, const ResidRows& rr, float4 (&x)[8], int lane, int col) {
  const bool col_ok = col + 4 * (lane & 7) < p.N;
#pragma unroll
  for (int i = 0; i < 8; ++i)
    if (col_ok && i < rr.n_load) x[i] = *reinterpret_cast<const float4*>(rr.out0 + (size_t)(4 * i) * p.N + col);
}

__device__ __forceinline__ void residual_chunk(const GemmDev& p, const ResidRows& rr, const uint32_t (&r)[32], const float4 (&x)[8],
                                               float* tile, int lane, int col, const uint4* bias4) {
  float v[32];
  chunk_values(p, r, col, v, bias4);
#pragma unroll
  for (int g = 0; g < 8; ++g)
    *reinterpret_cast<float4*>(tile + lane * kResidTilePitch + 4 * g) = make_float4(v[4 * g], v[4 * g + 1], v[4 * g + 2], v[4 * g + 3]);
  __syncwarp();
  if (col + 4 * (lane & 7) < p.N) {
    float4 g0 = make_float4(1.f, 1.f, 1.f, 1.f), g1 = g0;
    if (rr.gam0) {
      g0 = __ldg(reinterpret_cast<const float4*>(rr.gam0 + col));
      if (rr.n_first < rr.n_rows) g1 = __ldg(reinterpret_cast<const float4*>(rr.gam1 + col));
    }
    const float* trow = tile + (lane >> 3) * kResidTilePitch + 4 * (lane & 7);
#pragma unroll
    for (int i = 0; i < 8; ++i) {
      if (i < rr.n_rows) {
        const float4 a = *reinterpret_cast<const float4*>(trow + 4 * i * kResidTilePitch);
        const float4 gg = i < rr.n_first ? g0 : g1;
        float4 xv = i < rr.n_load ? x[i] : make_float4(0.f, 0.f, 0.f, 0.f);
        xv.x = fmaf(gg.x, a.x, xv.x); xv.y = fmaf(gg.y, a.y, xv.y); xv.z = fmaf(gg.z, a.z, xv.z); xv.w = fmaf(gg.w, a.w, xv.w);
        *reinterpret_cast<float4*>(rr.out0 + (size_t)(4 * i) * p.N + col) = xv;
        if (rr.aux0) {
          uint2 o;
          o.x = pack_bf16x2(a.x, a.y); o.y = pack_bf16x2(a.z, a.w);
          *reinterpret_cast<uint2*>(rr.aux0 + (size_t)(4 * i) * p.N + col) = o;
        }
      }
    }
  }
  __syncwarp();
}

// One 32-column chunk of one accumulator row: bias, optional GELU, then the epilogue's store.
__device__ __forceinline__ void store_chunk(const GemmDev& p, const float (&v)[32], int row, int img, int jrow, int col);
__device__ __forceinline__ void epilogue_chunk(const GemmDev& p, const uint32_t (&r)[32], int row, int img, int jrow, int col,
                                               const uint4* bias4) {
  float v[32];
  chunk_values(p, r, col, v, bias4);
  store_chunk(p, v, row, img, jrow, col);
}

// The epilogue's store of 32 finished fp32 values of one row.
__device__ __forceinline__ void store_chunk(const GemmDev& p, const float (&v)[32], int row, int img, int jrow, int col) {
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
  } else if (p.epilogue == EPI_F32) {
    float4* xr = reinterpret_cast<float4*>(static_cast<float*>(p.out) + (size_t)row * p.N + col);
#pragma unroll
    for (int g = 0; g < 8; ++g)
      if (col + 4 * g < p.N) xr[g] = make_float4(v[4 * g + 0], v[4 * g + 1], v[4 * g + 2], v[4 * g + 3]);
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
  } else if (p.epilogue == EPI_RESIDUAL_XBF16) {
    // gate + residual into a bf16 residual stream: out = bf16(float(out) + gamma * v), rounded once (+ bf16 copy of v)
    uint4* xr = reinterpret_cast<uint4*>(static_cast<__nv_bfloat16*>(p.out) + (size_t)row * p.N + col);
    const float4* gp = p.gamma ? reinterpret_cast<const float4*>(p.gamma + (size_t)img * p.mod_stride + col) : nullptr;
    uint4* ap = p.aux ? reinterpret_cast<uint4*>(static_cast<__nv_bfloat16*>(p.aux) + (size_t)row * p.N + col) : nullptr;
#pragma unroll
    for (int g = 0; g < 4; ++g) {
      if (col + 8 * g < p.N) {
        const uint4 xo = xr[g];
        const uint32_t u[4] = {xo.x, xo.y, xo.z, xo.w};
        float xv[8];
#pragma unroll
        for (int i = 0; i < 4; ++i) { xv[2 * i] = __uint_as_float(u[i] << 16); xv[2 * i + 1] = __uint_as_float(u[i] & 0xFFFF0000u); }
        if (gp) {
          const float4 ga = __ldg(gp + 2 * g), gb = __ldg(gp + 2 * g + 1);
          xv[0] = fmaf(ga.x, v[8 * g + 0], xv[0]); xv[1] = fmaf(ga.y, v[8 * g + 1], xv[1]); xv[2] = fmaf(ga.z, v[8 * g + 2], xv[2]); xv[3] = fmaf(ga.w, v[8 * g + 3], xv[3]);
          xv[4] = fmaf(gb.x, v[8 * g + 4], xv[4]); xv[5] = fmaf(gb.y, v[8 * g + 5], xv[5]); xv[6] = fmaf(gb.z, v[8 * g + 6], xv[6]); xv[7] = fmaf(gb.w, v[8 * g + 7], xv[7]);
        } else {
#pragma unroll
          for (int i = 0; i < 8; ++i) xv[i] += v[8 * g + i];
        }
        uint4 o;
        o.x = pack_bf16x2(xv[0], xv[1]); o.y = pack_bf16x2(xv[2], xv[3]); o.z = pack_bf16x2(xv[4], xv[5]); o.w = pack_bf16x2(xv[6], xv[7]);
        xr[g] = o;
        if (ap) {
          uint4 c;
          c.x = pack_bf16x2(v[8 * g + 0], v[8 * g + 1]); c.y = pack_bf16x2(v[8 * g + 2], v[8 * g + 3]);
          c.z = pack_bf16x2(v[8 * g + 4], v[8 * g + 5]); c.w = pack_bf16x2(v[8 * g + 6], v[8 * g + 7]);
          ap[g] = c;
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


// ---- Q / K columns of the QKV projection with cosine attention and / or rotary positions (KIND 2) ----
// One head's columns [col, col + head_dim) of one accumulator row (thread = row).  Cosine attention needs
// the head's norm before any value can be stored, so the head's chunks are read from TMEM twice (the read is
// cheap): once to sum the squares of acc + bias, once to scale, rotate and store.  The rotation angle belongs
// to the token's ORIGINAL slot in the map (rope_idx), not to its row in the compact tensor.
// Called by the whole warp (the TMEM loads are warp-wide); rows past M take part in the loads only.
__device__ __forceinline__ void qk_head_epilogue(const GemmDev& p, uint32_t taddr, int row, bool row_ok, int img, int jrow, int col,
                                                 const uint4* bias4, bool is_query) {
  const int hd = p.head_dim;
  float scale = 1.f;
  if (p.qk_scale) {
    float ss = 0.f;
    for (int c = 0; c < hd; c += 32) {
      uint32_t r[32];
      float v[32];
      tmem_ld32(taddr + c, r);
      tmem_wait_ld();
      chunk_values(p, r, col + c, v, bias4 + c / 8);
#pragma unroll
      for (int i = 0; i < 32; ++i) ss = fmaf(v[i], v[i], ss);
    }
    scale = 1.f / fmaxf(sqrtf(ss), 1e-12f);
    if (is_query) scale *= __ldg(p.qk_scale + (col % p.C) / hd);
  }
  const int token = (p.rope_idx && row_ok) ? __ldg(p.rope_idx + (size_t)img * p.rows_per_image + jrow) : jrow;
  const float4* tab = (p.rope_table && row_ok) ? reinterpret_cast<const float4*>(p.rope_table + (size_t)token * (hd / 2)) : nullptr;
  for (int c = 0; c < hd; c += 32) {
    uint32_t r[32];
    float v[32];
    tmem_ld32(taddr + c, r);
    tmem_wait_ld();
    chunk_values(p, r, col + c, v, bias4 + c / 8);
    if (p.qk_scale) {
#pragma unroll
      for (int i = 0; i < 32; ++i) v[i] *= scale;
    }
    if (tab) {
#pragma unroll
      for (int g = 0; g < 8; ++g) {   // two channel pairs per float4 of (cos, sin, cos, sin)
        const float4 cs = __ldg(tab + c / 4 + g);
        const float a0 = v[4 * g], b0 = v[4 * g + 1], a1 = v[4 * g + 2], b1 = v[4 * g + 3];
        v[4 * g] = a0 * cs.x - b0 * cs.y;
        v[4 * g + 1] = a0 * cs.y + b0 * cs.x;
        v[4 * g + 2] = a1 * cs.z - b1 * cs.w;
        v[4 * g + 3] = a1 * cs.w + b1 * cs.z;
      }
    }
    if (row_ok) store_chunk(p, v, row, img, jrow, col + c);
  }
}

// All columns of one tile for KIND 2: Q and K heads through qk_head_epilogue, V columns as usual.
template <int BN>
__device__ __forceinline__ void qkv_extras_tile(const GemmDev& p, uint32_t t0, int row, bool row_ok, int img, int jrow, int n0,
                                                const uint4* bias_w) {
  const int hd = p.head_dim;
  for (int c0 = 0; c0 < BN; c0 += hd) {
    const int col = n0 + c0;
    if (col >= p.N) break;
    if (col < p.q_cols + p.C) {
      qk_head_epilogue(p, t0 + c0, row, row_ok, img, jrow, col, bias_w + c0 / 8, col < p.q_cols);
    } else {
      for (int c = 0; c < hd; c += 32) {
        uint32_t r[32];
        tmem_ld32(t0 + c0 + c, r);
        tmem_wait_ld();
        if (row_ok) epilogue_chunk(p, r, row, img, jrow, col + c, bias_w + (c0 + c) / 8);
      }
    }
  }
}

}  // namespace gemm_detail

// gemm_cluster.cu: K split inside a cluster of `slices` CTAs per tile (partials reduced through distributed
// shared memory); bn in {64, 128}, slices in {2, 4}, p.kb_per_split k-blocks per CTA.
cudaError_t gemm_cluster_init();
cudaError_t launch_gemm_cluster(const GemmArgs& g, const gemm_detail::GemmDev& p, int bn, int slices, cudaStream_t st);

// gemm_pair.cu: the CTA-pair kernel (256 x bn tiles, bn in {128, 256}); same argument block and epilogues.
cudaError_t gemm_pair_init();
cudaError_t launch_gemm_pair(const GemmArgs& g, const gemm_detail::GemmDev& p, int bn, cudaStream_t st);

}  // namespace fv
