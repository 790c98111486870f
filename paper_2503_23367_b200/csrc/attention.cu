// Flash-style attention of the kept queries over the KV cache (Sec. 3.1: the KV cache of previous
// scale steps; Sec. 3.3: at pruned steps the cache holds only pivotal keys, and FastVAR never reads
// the attention map, so a fused kernel applies).  Within a scale step there is no mask: a query sees
// every cached key of the earlier scales and all keys appended by its own step.
//
// One CTA = 128 queries of one head of one image.  Keys are consumed in tiles of 128:
//   warp 0   : TMA producer (Q once; K tiles [128 keys x hd]; V^T tiles [hd x 128 keys]).
//   warp 1   : one lane issues tcgen05.mma:  S = Q K^T into one of two TMEM score buffers, and
//              O += P V with P read from shared memory; S of tile j+1 is issued before P V of tile j
//              so the tensor core works while the softmax warps handle tile j.
//   warps 2-5: online softmax, thread = query row: tcgen05.ld the 128 scores, running max / sum in
//              fp32 (base-2 exponent), bf16 probabilities written to shared memory in the 128-byte
//              swizzled K-major layout the MMA reads; the O accumulator in TMEM is rescaled in place
//              when the running max moves; final O / l is written as bf16.
// V is read transposed ([channel, key], keys contiguous), which makes it a K-major B operand.
// Every wait is bounded (status word + normal unwind on expiry).
#include <cuda.h>
#include <cuda_bf16.h>

#include "internal.h"
#include "sm100.cuh"

namespace fv {

namespace {

constexpr int QT = 128;  // queries per CTA
constexpr int KT = 128;  // keys per tile
constexpr int kAttnThreads = 192;

template <int HD> struct AttnCfg {
  static constexpr int kStages = (HD == 128) ? 2 : 3;
  static constexpr int kQBytes = QT * HD * 2;
  static constexpr int kKBytes = KT * HD * 2;
  static constexpr int kVBytes = HD * KT * 2;
  static constexpr int kPBytes = QT * KT * 2;
  static constexpr int kSmemBytes = kQBytes + kStages * (kKBytes + kVBytes) + kPBytes + 1024 + 256;
  static constexpr int kTmemCols = 512;  // S0 [0,128) S1 [128,256) O [256, 256+HD)
};

struct AttnDev {
  __nv_bfloat16* out;
  int rows, C, kv_len, kv_capacity;
  float scale_log2;  // log2(e) / sqrt(hd)
  int32_t* status;
};

__device__ __forceinline__ void report(int32_t* status, int code) {
  if (status) atomicCAS(status, 0, code);
}

__device__ __forceinline__ float fast_exp2(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}

template <int HD>
__global__ void __launch_bounds__(kAttnThreads, 1)
attention_kernel(const __grid_constant__ CUtensorMap tmQ, const __grid_constant__ CUtensorMap tmK,
                 const __grid_constant__ CUtensorMap tmV, const AttnDev p) {
  using Cfg = AttnCfg<HD>;
  constexpr int NS = Cfg::kStages;
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  uint8_t* q_s = smem;
  uint8_t* k_s = q_s + Cfg::kQBytes;
  uint8_t* v_s = k_s + NS * Cfg::kKBytes;
  uint8_t* p_s = v_s + NS * Cfg::kVBytes;
  uint64_t* bars = reinterpret_cast<uint64_t*>(p_s + Cfg::kPBytes);
  uint64_t* q_full = bars;
  uint64_t* k_full = bars + 1;
  uint64_t* k_empty = k_full + NS;
  uint64_t* v_full = k_empty + NS;
  uint64_t* v_empty = v_full + NS;
  uint64_t* s_full = v_empty + NS;   // [2]
  uint64_t* s_free = s_full + 2;     // [2]
  uint64_t* p_full = s_free + 2;
  uint64_t* p_free = p_full + 1;
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(p_free + 1);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int q0 = blockIdx.x * QT, head = blockIdx.y, img = blockIdx.z;
  const int T = (p.kv_len + KT - 1) / KT;

  if (threadIdx.x == 0) {
    mbar_init(q_full, 1);
    for (int s = 0; s < NS; ++s) { mbar_init(&k_full[s], 1); mbar_init(&k_empty[s], 1); mbar_init(&v_full[s], 1); mbar_init(&v_empty[s], 1); }
    for (int s = 0; s < 2; ++s) { mbar_init(&s_full[s], 1); mbar_init(&s_free[s], 128); }
    mbar_init(p_full, 128);
    mbar_init(p_free, 1);
    mbar_fence_init();
    tma_prefetch_desc(&tmQ); tma_prefetch_desc(&tmK); tma_prefetch_desc(&tmV);
  }
  if (warp == 1) { tmem_alloc(tmem_slot, Cfg::kTmemCols); tmem_relinquish(); }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;
  const uint32_t tmem_o = tmem_base + 256;

  if (warp == 0) {
    if (lane == 0) {
      mbar_expect_tx(q_full, Cfg::kQBytes);
      for (int a = 0; a < HD / 64; ++a) tma_load_2d(q_s + a * (QT * 128), &tmQ, head * HD + a * 64, img * p.rows + q0, q_full);
      for (int j = 0; j < T; ++j) {
        const int s = j % NS;
        const uint32_t ph = (j / NS) & 1;
        if (!mbar_wait(&k_empty[s], ph ^ 1)) { report(p.status, DEV_TIMEOUT_TMA); break; }
        mbar_expect_tx(&k_full[s], Cfg::kKBytes);
        for (int a = 0; a < HD / 64; ++a)
          tma_load_2d(k_s + s * Cfg::kKBytes + a * (KT * 128), &tmK, head * HD + a * 64, img * p.kv_capacity + j * KT, &k_full[s]);
        if (!mbar_wait(&v_empty[s], ph ^ 1)) { report(p.status, DEV_TIMEOUT_TMA); break; }
        mbar_expect_tx(&v_full[s], Cfg::kVBytes);
        for (int a = 0; a < KT / 64; ++a)
          tma_load_2d(v_s + s * Cfg::kVBytes + a * (HD * 128), &tmV, j * KT + a * 64, img * p.C + head * HD, &v_full[s]);
      }
    }
  } else if (warp == 1) {
    if (lane == 0) {
      constexpr uint32_t idesc_qk = umma_idesc_bf16(QT, KT);
      constexpr uint32_t idesc_pv = umma_idesc_bf16(QT, HD);
      bool ok = mbar_wait(q_full, 0);
      if (!ok) report(p.status, DEV_TIMEOUT_MMA);
      const uint32_t q_addr = smem_u32(q_s), p_addr = smem_u32(p_s);
      for (int j = 0; ok && j <= T; ++j) {
        if (j < T) {
          const int s = j % NS;
          if (!mbar_wait(&k_full[s], (j / NS) & 1) || !mbar_wait(&s_free[j & 1], ((j >> 1) & 1) ^ 1)) {
            report(p.status, DEV_TIMEOUT_MMA); ok = false; break;
          }
          tc_fence_after();
          const uint32_t k_addr = smem_u32(k_s + s * Cfg::kKBytes);
          const uint32_t d = tmem_base + (j & 1) * KT;
#pragma unroll
          for (int kk = 0; kk < HD / 16; ++kk) {
            const uint32_t off = (kk >> 2) * (QT * 128) + (kk & 3) * 32;
            umma_bf16(d, umma_desc_k_sw128(q_addr + off), umma_desc_k_sw128(k_addr + off), idesc_qk, kk != 0);
          }
          umma_commit(&k_empty[s]);
          umma_commit(&s_full[j & 1]);
        }
        if (j > 0) {
          const int jj = j - 1, s = jj % NS;
          if (!mbar_wait(&v_full[s], (jj / NS) & 1) || !mbar_wait(p_full, jj & 1)) {
            report(p.status, DEV_TIMEOUT_MMA); ok = false; break;
          }
          tc_fence_after();
          const uint32_t v_addr = smem_u32(v_s + s * Cfg::kVBytes);
#pragma unroll
          for (int kk = 0; kk < KT / 16; ++kk) {
            const uint32_t a_off = (kk >> 2) * (QT * 128) + (kk & 3) * 32;
            const uint32_t b_off = (kk >> 2) * (HD * 128) + (kk & 3) * 32;
            umma_bf16(tmem_o, umma_desc_k_sw128(p_addr + a_off), umma_desc_k_sw128(v_addr + b_off), idesc_pv, (jj | kk) != 0);
          }
          umma_commit(&v_empty[s]);
          umma_commit(p_free);
        }
      }
    }
  } else {
    // ---- softmax + output: thread = one query row ----
    const int quarter = warp & 3;
    const int r = quarter * 32 + lane;
    const uint32_t lane_off = uint32_t(quarter * 32) << 16;
    float m_run = -INFINITY, l_run = 0.f;
    bool ok = true;
    for (int j = 0; j < T; ++j) {
      if (!mbar_wait(&s_full[j & 1], (j >> 1) & 1)) { report(p.status, DEV_TIMEOUT_SOFTMAX); ok = false; break; }
      tc_fence_after();
      float sc[KT];
#pragma unroll
      for (int c = 0; c < KT / 32; ++c) {
        uint32_t t[32];
        tmem_ld32(tmem_base + lane_off + (j & 1) * KT + c * 32, t);
#pragma unroll
        for (int i = 0; i < 32; ++i) sc[c * 32 + i] = __uint_as_float(t[i]);
      }
      tmem_wait_ld();
      tc_fence_before();
      mbar_arrive(&s_free[j & 1]);
      const int valid = p.kv_len - j * KT;  // >= 1
      float mx = -INFINITY;
#pragma unroll
      for (int i = 0; i < KT; ++i) {
        if (i >= valid) sc[i] = -INFINITY;
        mx = fmaxf(mx, sc[i]);
      }
      const float m_new = fmaxf(m_run, mx * p.scale_log2);
      const float alpha = fast_exp2(m_run - m_new);  // 0 on the first tile (m_run = -inf)
      float rs = 0.f;
#pragma unroll
      for (int i = 0; i < KT; ++i) {
        sc[i] = fast_exp2(fmaf(sc[i], p.scale_log2, -m_new));
        rs += sc[i];
      }
      l_run = fmaf(l_run, alpha, rs);
      m_run = m_new;
      // P buffer free and O stable once P V of the previous tile has completed
      if (!mbar_wait(p_free, (j & 1) ^ 1)) { report(p.status, DEV_TIMEOUT_SOFTMAX); ok = false; break; }
      tc_fence_after();
      if (j > 0 && __any_sync(0xffffffffu, alpha != 1.f)) {
#pragma unroll
        for (int c = 0; c < HD / 32; ++c) {
          uint32_t t[32];
          tmem_ld32(tmem_o + lane_off + c * 32, t);
          tmem_wait_ld();
#pragma unroll
          for (int i = 0; i < 32; ++i) t[i] = __float_as_uint(__uint_as_float(t[i]) * alpha);
          tmem_st32(tmem_o + lane_off + c * 32, t);
        }
        tmem_wait_st();
      }
      // bf16 probabilities -> shared memory, K-major rows of 128 bytes with the 128-byte swizzle
#pragma unroll
      for (int c8 = 0; c8 < KT / 8; ++c8) {
        uint4 o;
        o.x = pack_bf16x2(sc[8 * c8 + 0], sc[8 * c8 + 1]); o.y = pack_bf16x2(sc[8 * c8 + 2], sc[8 * c8 + 3]);
        o.z = pack_bf16x2(sc[8 * c8 + 4], sc[8 * c8 + 5]); o.w = pack_bf16x2(sc[8 * c8 + 6], sc[8 * c8 + 7]);
        const int atom = c8 >> 3, chunk = c8 & 7;
        *reinterpret_cast<uint4*>(p_s + atom * (QT * 128) + r * 128 + ((chunk ^ (r & 7)) << 4)) = o;
      }
      fence_async_smem();
      tc_fence_before();
      mbar_arrive(p_full);
    }
    if (ok) {
      if (!mbar_wait(p_free, (T - 1) & 1)) { report(p.status, DEV_TIMEOUT_SOFTMAX); ok = false; }
    }
    tc_fence_after();
    if (ok) {
      const float inv_l = 1.f / l_run;
      const int row = q0 + r;
      __nv_bfloat16* dst = p.out + ((size_t)img * p.rows + row) * p.C + head * HD;
#pragma unroll
      for (int c = 0; c < HD / 32; ++c) {
        uint32_t t[32];
        tmem_ld32(tmem_o + lane_off + c * 32, t);
        tmem_wait_ld();
        if (row < p.rows) {
#pragma unroll
          for (int g = 0; g < 4; ++g) {
            uint4 o;
            o.x = pack_bf16x2(__uint_as_float(t[8 * g + 0]) * inv_l, __uint_as_float(t[8 * g + 1]) * inv_l);
            o.y = pack_bf16x2(__uint_as_float(t[8 * g + 2]) * inv_l, __uint_as_float(t[8 * g + 3]) * inv_l);
            o.z = pack_bf16x2(__uint_as_float(t[8 * g + 4]) * inv_l, __uint_as_float(t[8 * g + 5]) * inv_l);
            o.w = pack_bf16x2(__uint_as_float(t[8 * g + 6]) * inv_l, __uint_as_float(t[8 * g + 7]) * inv_l);
            reinterpret_cast<uint4*>(dst + c * 32)[g] = o;
          }
        }
      }
    }
  }
  tc_fence_before();
  __syncthreads();
  if (warp == 1) {
    __syncwarp();
    tmem_dealloc(tmem_base, Cfg::kTmemCols);
  }
}

bool make_tmap_rows(void* out, const void* base, uint64_t rows, uint64_t cols, uint32_t box_rows) {
  return make_tmap_bf16_2d(out, base, rows, cols, box_rows);
}

template <int HD> fv_status launch_hd(const AttnArgs& a, cudaStream_t st) {
  alignas(64) CUtensorMap tmQ, tmK, tmV;
  if (!make_tmap_rows(&tmQ, a.q, (uint64_t)a.B * a.rows, a.C, QT)) return FV_ERR_CUDA;
  if (!make_tmap_rows(&tmK, a.k, (uint64_t)a.B * a.kv_capacity, a.C, KT)) return FV_ERR_CUDA;
  if (!make_tmap_rows(&tmV, a.vt, (uint64_t)a.B * a.C, a.kv_capacity, HD)) return FV_ERR_CUDA;
  AttnDev p;
  p.out = static_cast<__nv_bfloat16*>(a.out);
  p.rows = a.rows; p.C = a.C; p.kv_len = a.kv_len; p.kv_capacity = a.kv_capacity;
  p.scale_log2 = 1.4426950408889634f / sqrtf((float)HD);
  p.status = a.status;
  dim3 grid((a.rows + QT - 1) / QT, a.H, a.B);
  LaunchScope scope(KC_ATTENTION, 1, 4.0 * a.B * (double)a.rows * a.kv_len * a.C, st);
  attention_kernel<HD><<<grid, kAttnThreads, AttnCfg<HD>::kSmemBytes, st>>>(tmQ, tmK, tmV, p);
  return cudaGetLastError() == cudaSuccess ? FV_OK : FV_ERR_CUDA;
}

}  // namespace

cudaError_t attention_init() {
  cudaError_t e = cudaFuncSetAttribute(attention_kernel<64>, cudaFuncAttributeMaxDynamicSharedMemorySize, AttnCfg<64>::kSmemBytes);
  if (e != cudaSuccess) return e;
  return cudaFuncSetAttribute(attention_kernel<128>, cudaFuncAttributeMaxDynamicSharedMemorySize, AttnCfg<128>::kSmemBytes);
}

fv_status launch_attention(const AttnArgs& a, cudaStream_t st) {
  if (!a.q || !a.k || !a.vt || !a.out || a.B <= 0 || a.rows <= 0 || a.H <= 0 || a.kv_len <= 0) return FV_ERR_INVALID_ARG;
  if (a.C % a.H || a.kv_capacity % 8 || a.kv_len > a.kv_capacity) return FV_ERR_INVALID_ARG;
  const int hd = a.C / a.H;
  if (hd == 64) return launch_hd<64>(a, st);
  if (hd == 128) return launch_hd<128>(a, st);
  return FV_ERR_UNSUPPORTED;
}

}  // namespace fv
