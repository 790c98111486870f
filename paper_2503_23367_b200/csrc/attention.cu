// Flash-style attention of the kept queries over the KV cache (Sec. 3.1: the KV cache of previous
// scale steps; Sec. 3.3: at pruned steps the cache holds only pivotal keys, and FastVAR never reads
// the attention map, so a fused kernel applies).  Within a scale step there is no mask: a query sees
// every cached key of the earlier scales and all keys appended by its own step.
//
// One CTA = 256 queries (two tiles of 128) of one head of one image; keys are consumed in tiles of 128.
// The two query tiles take turns on the tensor core: while the softmax warps of one tile work on its
// scores, the MMAs of the other tile run.
//   warp 8   : TMA producer (both Q tiles once; K tiles [128 keys x hd]; V^T tiles [hd x 128 keys]).
//   warp 9   : one lane issues tcgen05.mma.  Per key tile j and query tile t:  O_t += P_t V_j  with P_t
//              read from TENSOR MEMORY (it overwrites the first 64 columns of S_t), then
//              S_t = Q_t K_{j+1}^T.  MMAs of one thread execute in issue order, which is what makes
//              the P_t / S_t aliasing safe.
//   warps 0-3, 4-7: online softmax of tile 0 / tile 1, thread = query row: the 128 scores of the row come
//              out of TMEM in one go (four loads, one wait; the register file is re-divided between the
//              warpgroups with setmaxnreg so that a thread can hold them), row maximum, base-2
//              exponentials, row sum, and the bf16 probabilities go back to TMEM.  The running maximum is only raised when
//              it would grow by more than 2^8, so the O accumulator (TMEM) is rescaled in place only
//              on the rare tiles where that happens; the final O / l is written as bf16.
// V is read transposed ([channel, key], keys contiguous), which makes it a K-major B operand.
// Every wait is bounded (status word + normal unwind on expiry).
#include <cuda.h>
#include <cuda_bf16.h>

#include "internal.h"
#include "sm100.cuh"

namespace fv {

namespace {

constexpr int QT = 128;   // queries per tile (two tiles per CTA)
constexpr int KT = 128;   // keys per tile
constexpr int kAttnThreads = 384;   // warps 0-3 / 4-7: softmax of query tile 0 / 1; warp 8: TMA; warp 9: MMA; 10-11: idle
constexpr float kRescaleThreshold = 8.f;  // log2 units

template <int HD> struct AttnCfg {
  static constexpr int kStages = (HD == 128) ? 2 : 4;
  static constexpr int kQBytes = QT * HD * 2;   // one query tile
  static constexpr int kKBytes = KT * HD * 2;
  static constexpr int kVBytes = HD * KT * 2;
  static constexpr int kSmemBytes = 2 * kQBytes + kStages * (kKBytes + kVBytes) + 1024 + 256;
  static constexpr int kTmemCols = 512;  // S0 [0,128) S1 [128,256) O0 [256,256+HD) O1 [384,384+HD)
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

// The 128 scores of one row: TMEM -> registers (one wait for all four loads).  MASK: keys >= valid read -inf.
template <bool MASK>
__device__ __forceinline__ void tile_load_scores(uint32_t s_addr, int valid, float (&sc)[KT]) {
  uint32_t a[32], b[32], c[32], d[32];
  tmem_ld32(s_addr, a);
  tmem_ld32(s_addr + 32, b);
  tmem_ld32(s_addr + 64, c);
  tmem_ld32(s_addr + 96, d);
  tmem_wait_ld();
#pragma unroll
  for (int i = 0; i < 32; ++i) {
    sc[i] = __uint_as_float(a[i]); sc[32 + i] = __uint_as_float(b[i]);
    sc[64 + i] = __uint_as_float(c[i]); sc[96 + i] = __uint_as_float(d[i]);
  }
  if (MASK) {
#pragma unroll
    for (int i = 0; i < KT; ++i)
      if (i >= valid) sc[i] = -INFINITY;
  }
}

// p = 2^(s * scale - m) for the 128 scores of a row; bf16 pairs written to TMEM columns [p_addr, +64);
// returns the row sum of the UNROUNDED probabilities.  Masked scores are -inf and give p = 0.
__device__ __forceinline__ float tile_exp_store(const float (&sc)[KT], uint32_t p_addr, float scale, float m) {
  float rs0 = 0.f, rs1 = 0.f;
#pragma unroll
  for (int c = 0; c < KT / 32; ++c) {
    uint32_t pk[16];
#pragma unroll
    for (int i = 0; i < 16; ++i) {
      const float p0 = fast_exp2(fmaf(sc[c * 32 + 2 * i], scale, -m));
      const float p1 = fast_exp2(fmaf(sc[c * 32 + 2 * i + 1], scale, -m));
      rs0 += p0; rs1 += p1;
      pk[i] = pack_bf16x2(p0, p1);
    }
    tmem_st16(p_addr + c * 16, pk);
  }
  return rs0 + rs1;
}

template <int HD>
__global__ void __launch_bounds__(kAttnThreads, 1)
attention_kernel(const __grid_constant__ CUtensorMap tmQ, const __grid_constant__ CUtensorMap tmK,
                 const __grid_constant__ CUtensorMap tmV, const AttnDev p) {
  using Cfg = AttnCfg<HD>;
  constexpr int NS = Cfg::kStages;
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  uint8_t* q_s = smem;                          // two query tiles
  uint8_t* k_s = q_s + 2 * Cfg::kQBytes;
  uint8_t* v_s = k_s + NS * Cfg::kKBytes;
  uint64_t* bars = reinterpret_cast<uint64_t*>(v_s + NS * Cfg::kVBytes);
  uint64_t* q_full = bars;
  uint64_t* k_full = bars + 1;
  uint64_t* k_empty = k_full + NS;
  uint64_t* v_full = k_empty + NS;
  uint64_t* v_empty = v_full + NS;
  uint64_t* s_full = v_empty + NS;   // [2] scores of query tile t are in TMEM
  uint64_t* p_full = s_full + 2;     // [2] probabilities of query tile t are in TMEM (128 arrivals)
  uint64_t* o_done = p_full + 2;     // [2] the latest P V of query tile t has completed
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(o_done + 2);

  pdl_trigger();
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int q0 = blockIdx.x * (2 * QT), head = blockIdx.y, img = blockIdx.z;
  const int T = (p.kv_len + KT - 1) / KT;
  const int ntiles = (p.rows - q0 > QT) ? 2 : 1;

  if (threadIdx.x == 0) {
    mbar_init(q_full, 1);
    for (int s = 0; s < NS; ++s) { mbar_init(&k_full[s], 1); mbar_init(&k_empty[s], 1); mbar_init(&v_full[s], 1); mbar_init(&v_empty[s], 1); }
    for (int t = 0; t < 2; ++t) { mbar_init(&s_full[t], 1); mbar_init(&p_full[t], QT); mbar_init(&o_done[t], 1); }
    mbar_fence_init();
    tma_prefetch_desc(&tmQ); tma_prefetch_desc(&tmK); tma_prefetch_desc(&tmV);
  }
  if (warp == 9) { tmem_alloc(tmem_slot, Cfg::kTmemCols); tmem_relinquish(); }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;
  pdl_wait();  // set-up above overlaps the previous kernel; Q / K / V and the output are touched only from here

  // A softmax thread holds a whole score row (128 fp32) in registers, so the register file is re-divided
  // between the warpgroups: 2 x 128 x 216 + 128 x 40 <= 64 K registers.
  if (warp >= 8) {
   asm volatile("setmaxnreg.dec.sync.aligned.u32 40;");
   if (warp == 8) {
    if (lane == 0) {
      mbar_expect_tx(q_full, ntiles * Cfg::kQBytes);
      for (int t = 0; t < ntiles; ++t)
        for (int a = 0; a < HD / 64; ++a)
          tma_load_2d(q_s + t * Cfg::kQBytes + a * (QT * 128), &tmQ, head * HD + a * 64, img * p.rows + q0 + t * QT, q_full);
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
  } else if (warp == 9) {
    if (lane == 0) {
      constexpr uint32_t idesc_qk = umma_idesc_bf16(QT, KT);
      constexpr uint32_t idesc_pv = umma_idesc_bf16(QT, HD);
      const uint32_t q_addr = smem_u32(q_s);
      // S_t = Q_t K^T for the key tile in stage s
      auto issue_qk = [&](int t, int s) {
        const uint32_t k_addr = smem_u32(k_s + s * Cfg::kKBytes);
        const uint32_t qa = q_addr + t * Cfg::kQBytes;
#pragma unroll
        for (int kk = 0; kk < HD / 16; ++kk) {
          const uint32_t off = (kk >> 2) * (QT * 128) + (kk & 3) * 32;
          umma_bf16(tmem_base + t * KT, umma_desc_k_sw128(qa + off), umma_desc_k_sw128(k_addr + off), idesc_qk, kk != 0);
        }
        umma_commit(&s_full[t]);
      };
      bool ok = mbar_wait(q_full, 0) && mbar_wait(&k_full[0], 0);
      if (!ok) report(p.status, DEV_TIMEOUT_MMA);
      if (ok) {
        tc_fence_after();
        for (int t = 0; t < ntiles; ++t) issue_qk(t, 0);
        umma_commit(&k_empty[0]);
      }
      for (int j = 0; ok && j < T; ++j) {
        const int s = j % NS, sn = (j + 1) % NS;
        const bool more = j + 1 < T;
        if (!mbar_wait(&v_full[s], (j / NS) & 1) || (more && !mbar_wait(&k_full[sn], ((j + 1) / NS) & 1))) {
          report(p.status, DEV_TIMEOUT_MMA); ok = false; break;
        }
        const uint32_t v_addr = smem_u32(v_s + s * Cfg::kVBytes);
        for (int t = 0; t < ntiles; ++t) {
          if (!mbar_wait(&p_full[t], j & 1)) { report(p.status, DEV_TIMEOUT_MMA); ok = false; break; }
          tc_fence_after();
          const uint32_t p_tmem = tmem_base + t * KT;              // P_t over the first 64 columns of S_t
          const uint32_t o_tmem = tmem_base + 256 + t * 128;
#pragma unroll
          for (int kk = 0; kk < KT / 16; ++kk) {
            const uint32_t b_off = (kk >> 2) * (HD * 128) + (kk & 3) * 32;
            umma_bf16_ts(o_tmem, p_tmem + kk * 8, umma_desc_k_sw128(v_addr + b_off), idesc_pv, (j | kk) != 0);
          }
          umma_commit(&o_done[t]);
          if (more) issue_qk(t, sn);
        }
        if (!ok) break;
        umma_commit(&v_empty[s]);
        if (more) umma_commit(&k_empty[sn]);
      }
    }
   }
  } else {
    asm volatile("setmaxnreg.inc.sync.aligned.u32 216;");
    // ---- softmax + output: thread = one query row of tile t ----
    const int t = warp >> 2;
    const int quarter = warp & 3;                 // the TMEM lanes this warp may touch
    const int r = quarter * 32 + lane;
    const uint32_t lane_off = uint32_t(quarter * 32) << 16;
    const uint32_t s_addr = tmem_base + lane_off + t * KT;
    const uint32_t o_addr = tmem_base + lane_off + 256 + t * 128;
    if (t < ntiles) {
      float m_run = -INFINITY, l_run = 0.f;
      bool ok = true;
      for (int j = 0; j < T; ++j) {
        if (!mbar_wait(&s_full[t], j & 1)) { report(p.status, DEV_TIMEOUT_SOFTMAX); ok = false; break; }
        tc_fence_after();
        const int valid = p.kv_len - j * KT;  // >= 1
        float sc[KT];
        if (valid < KT) tile_load_scores<true>(s_addr, valid, sc);
        else tile_load_scores<false>(s_addr, valid, sc);
        float mx0 = sc[0], mx1 = sc[1], mx2 = sc[2], mx3 = sc[3];
#pragma unroll
        for (int i = 4; i < KT; i += 4) {
          mx0 = fmaxf(mx0, sc[i]); mx1 = fmaxf(mx1, sc[i + 1]); mx2 = fmaxf(mx2, sc[i + 2]); mx3 = fmaxf(mx3, sc[i + 3]);
        }
        const float mx = fmaxf(fmaxf(mx0, mx1), fmaxf(mx2, mx3)) * p.scale_log2;
        // Raise the running maximum only when it would grow by more than the threshold: probabilities
        // may then exceed 1 (by at most 2^threshold), which fp32 sums and bf16 P hold without loss.
        float alpha = 1.f;
        if (mx > m_run + kRescaleThreshold) {
          alpha = fast_exp2(m_run - mx);  // 0 on the first tile (m_run = -inf)
          m_run = mx;
        }
        // S_t of tile j was issued after P V of tile j-1, so O_t is at rest here.
        if (j > 0 && __any_sync(0xffffffffu, alpha != 1.f)) {
#pragma unroll
          for (int c = 0; c < HD / 32; ++c) {
            uint32_t o[32];
            tmem_ld32(o_addr + c * 32, o);
            tmem_wait_ld();
#pragma unroll
            for (int i = 0; i < 32; ++i) o[i] = __float_as_uint(__uint_as_float(o[i]) * alpha);
            tmem_st32(o_addr + c * 32, o);
          }
        }
        const float rs = tile_exp_store(sc, s_addr, p.scale_log2, m_run);
        l_run = fmaf(l_run, alpha, rs);
        tmem_wait_st();
        tc_fence_before();
        mbar_arrive(&p_full[t]);
      }
      if (ok && !mbar_wait(&o_done[t], (T - 1) & 1)) { report(p.status, DEV_TIMEOUT_SOFTMAX); ok = false; }
      tc_fence_after();
      if (ok) {
        const float inv_l = 1.f / l_run;
        const int row = q0 + t * QT + r;
        __nv_bfloat16* dst = p.out + ((size_t)img * p.rows + row) * p.C + head * HD;
#pragma unroll
        for (int c = 0; c < HD / 32; ++c) {
          uint32_t o[32];
          tmem_ld32(o_addr + c * 32, o);
          tmem_wait_ld();
          if (row < p.rows) {
#pragma unroll
            for (int g = 0; g < 4; ++g) {
              uint4 v;
              v.x = pack_bf16x2(__uint_as_float(o[8 * g + 0]) * inv_l, __uint_as_float(o[8 * g + 1]) * inv_l);
              v.y = pack_bf16x2(__uint_as_float(o[8 * g + 2]) * inv_l, __uint_as_float(o[8 * g + 3]) * inv_l);
              v.z = pack_bf16x2(__uint_as_float(o[8 * g + 4]) * inv_l, __uint_as_float(o[8 * g + 5]) * inv_l);
              v.w = pack_bf16x2(__uint_as_float(o[8 * g + 6]) * inv_l, __uint_as_float(o[8 * g + 7]) * inv_l);
              reinterpret_cast<uint4*>(dst + c * 32)[g] = v;
            }
          }
        }
      }
    }
  }
  tc_fence_before();
  __syncthreads();
  if (warp == 9) {
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
  dim3 grid((a.rows + 2 * QT - 1) / (2 * QT), a.H, a.B);
  LaunchScope scope(KC_ATTENTION, 1, 4.0 * a.B * (double)a.rows * a.kv_len * a.C,
                    2.0 * a.B * a.C * (2.0 * a.rows + 2.0 * a.kv_len), st);  // Q in, O out, K and V^T once
  return launch_pdl(attention_kernel<HD>, grid, dim3(kAttnThreads), AttnCfg<HD>::kSmemBytes, st, tmQ, tmK, tmV, p) == cudaSuccess
             ? FV_OK : FV_ERR_CUDA;
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
