// tcgen05 GEMM on CTA pairs (cta_group::2) for the large projections of the pruned scale steps
// (Fig. 3b: "Attention or FFN layers using FastVAR"): out = epilogue(A[M,K] * W[N,K]^T + bias).
//
// A single CTA feeding 128 x 256 MMAs has to pull (128 + 256) x 64 bf16 per k-block through its own
// L2 port, which is what bounds the one-CTA kernel.  Here two CTAs of a cluster share one 256 x BN output
// tile: each loads ITS 128 rows of A and ITS BN/2 rows of W, and the leader's MMA reads both halves of W
// from the two shared memories.  Per CTA that is (128 + BN/2) x 64 elements per k-block for the same
// MMA time -- a third less operand traffic at BN = 256.  No TMA multicast is used.
//   warp 0 (both CTAs): TMA producer of its own halves; the bytes of both CTAs complete on the LEADER's
//             full barrier.
//   warp 1 (leader)   : one lane issues tcgen05.mma.cta_group::2 (M = 256); tcgen05.commit multicasts to
//             the stage's empty barrier and the tile's accumulator barrier of both CTAs.
//   warps 2-5 (both)  : epilogue on the CTA's own 128 accumulator rows; the accumulator buffer is handed
//             back by arriving on the leader's barrier (256 arrivals).
// Persistent over tiles, two accumulator buffers in TMEM, every mbarrier wait bounded.
#include <cuda.h>
#include <cuda_bf16.h>

#include "gemm_epilogue.cuh"
#include "internal.h"
#include "sm100.cuh"

namespace fv {

using namespace gemm_detail;

namespace {

constexpr int BM = 128;   // rows of A per CTA (256 per pair)
constexpr int BK = 64;
constexpr int kThreads = 192;
constexpr int kATileBytes = BM * BK * 2;  // 16 KB

template <int BN> struct PairCfg {
  static constexpr int kKps = 2;                                // k-blocks per pipeline stage (one barrier round trip for both)
  static constexpr int kBHalfBytes = (BN / 2) * BK * 2;
  static constexpr int kSubBytes = kATileBytes + kBHalfBytes;   // one k-block: this CTA's A tile, then its half of the W tile
  static constexpr int kStageBytes = kKps * kSubBytes;
  static constexpr int kStages = (BN == 256) ? 3 : 4;
  static constexpr int kTmemCols = 512;    // two accumulators, 256 columns apart
  static constexpr int kAccStride = 256;
  // operand stages | per-warp bias slices | barriers | (residual-epilogue kernels only) one turning tile per warp
  static constexpr int smem_bytes(bool resid) {
    return kStages * kStageBytes + kBiasSmemBytes + 256 /*barriers*/ + (resid ? kResidSmemBytes : 0) + 1024 /*alignment slack*/;
  }
};

// RESID: the instantiation launched for the residual epilogue (a kernel of its own: it needs far more registers).
template <int BN, bool RESID>
__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(kThreads, 1)
gemm_pair_kernel(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmB, const GemmDev p) {
  using Cfg = PairCfg<BN>;
  constexpr int STAGES = Cfg::kStages;
  constexpr int KPS = Cfg::kKps;
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  uint4* bias_s = reinterpret_cast<uint4*>(smem + STAGES * Cfg::kStageBytes);   // per-warp bias slice of the tile
  float* resid_s = reinterpret_cast<float*>(smem + STAGES * Cfg::kStageBytes + kBiasSmemBytes + 256);   // RESID: one tile per warp
  uint64_t* full_bar = reinterpret_cast<uint64_t*>(smem + STAGES * Cfg::kStageBytes + kBiasSmemBytes);  // used in the leader
  uint64_t* empty_bar = full_bar + STAGES;   // one per CTA, completed by the leader's commits
  uint64_t* acc_full = empty_bar + STAGES;   // [2] one per CTA
  uint64_t* acc_empty = acc_full + 2;        // [2] used in the leader: 256 arrivals
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(acc_empty + 2);

  pdl_trigger();
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const uint32_t rank = cluster_ctarank();
  const int pair = blockIdx.x >> 1, npairs = gridDim.x >> 1;
  const int tiles_m = (p.M + 2 * BM - 1) / (2 * BM);
  const int tiles_n = (p.N + BN - 1) / BN;
  const int total_tiles = tiles_m * tiles_n;
  const int num_kb = (p.K + BK - 1) / BK;

  if (threadIdx.x == 0) {
    for (int s = 0; s < STAGES; ++s) { mbar_init(&full_bar[s], 1); mbar_init(&empty_bar[s], 1); }
    for (int s = 0; s < 2; ++s) { mbar_init(&acc_full[s], 1); mbar_init(&acc_empty[s], 256); }
    mbar_fence_init();
    tma_prefetch_desc(&tmA);
    tma_prefetch_desc(&tmB);
  }
  cluster_sync_all();  // the peer's barriers exist before anything is signalled across the pair
  if (warp == 1) { tmem_alloc_pair(tmem_slot, Cfg::kTmemCols); tmem_relinquish_pair(); }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;
  // Set-up above overlaps the previous kernel.  Activations and outputs are touched only after
  // pdl_wait(); the weight tiles (never written by a kernel of the step) are requested before it.

  if (warp == 0) {
    if (lane == 0) {
      uint32_t it = 0;
      bool ok = true;
      int pre = 0;  // stages of the first tile whose W half-tile is already on its way
      if (pair < total_tiles) {
        const int n0 = (pair / tiles_m) * BN + (int)rank * (BN / 2);
        pre = min(STAGES, (num_kb + KPS - 1) / KPS);
        for (int i = 0; i < pre; ++i) {
          if (rank == 0) mbar_expect_tx(&full_bar[i], 2 * Cfg::kStageBytes);
          for (int u = 0; u < KPS; ++u)   // (a k-block beyond K reads zeros)
            tma_load_2d_pair(smem + i * Cfg::kStageBytes + u * Cfg::kSubBytes + kATileBytes, &tmB, (KPS * i + u) * BK, n0, &full_bar[i]);
        }
      }
      pdl_wait();
      for (int tile = pair; ok && tile < total_tiles; tile += npairs) {
        const int m0 = (tile % tiles_m) * (2 * BM) + (int)rank * BM;
        const int n0 = (tile / tiles_m) * BN + (int)rank * (BN / 2);
        for (int kb = 0; kb < num_kb; kb += KPS, ++it) {
          const int s = it % STAGES;
          uint8_t* a_s = smem + s * Cfg::kStageBytes;
          if ((int)it < pre) {  // W half-tiles requested before the wait: only the activations are missing
            for (int u = 0; u < KPS; ++u) tma_load_2d_pair(a_s + u * Cfg::kSubBytes, &tmA, (kb + u) * BK, m0, &full_bar[s]);
            continue;
          }
          const uint32_t ph = (it / STAGES) & 1;
          if (!mbar_wait(&empty_bar[s], ph ^ 1)) { report(p.status, DEV_TIMEOUT_TMA); ok = false; break; }
          if (rank == 0) mbar_expect_tx(&full_bar[s], 2 * Cfg::kStageBytes);
          for (int u = 0; u < KPS; ++u) {
            tma_load_2d_pair(a_s + u * Cfg::kSubBytes, &tmA, (kb + u) * BK, m0, &full_bar[s]);
            tma_load_2d_pair(a_s + u * Cfg::kSubBytes + kATileBytes, &tmB, (kb + u) * BK, n0, &full_bar[s]);
          }
        }
      }
    }
  } else if (warp == 1) {
    pdl_wait();
    if (rank == 0 && lane == 0) {
      constexpr uint32_t idesc = umma_idesc_bf16(2 * BM, BN);
      uint32_t it = 0, lt = 0;
      bool ok = true;
      for (int tile = pair; ok && tile < total_tiles; tile += npairs, ++lt) {
        const uint32_t buf = lt & 1;
        if (!mbar_wait(&acc_empty[buf], ((lt >> 1) & 1) ^ 1)) { report(p.status, DEV_TIMEOUT_MMA); ok = false; break; }
        tc_fence_after();
        const uint32_t d = tmem_base + buf * Cfg::kAccStride;
        for (int kb = 0; kb < num_kb; kb += KPS, ++it) {
          const int s = it % STAGES;
          const uint32_t ph = (it / STAGES) & 1;
          if (!mbar_wait(&full_bar[s], ph)) { report(p.status, DEV_TIMEOUT_MMA); ok = false; break; }
          tc_fence_after();
          const uint32_t a_addr = smem_u32(smem + s * Cfg::kStageBytes);
#pragma unroll
          for (int u = 0; u < KPS; ++u) {
            const uint64_t adesc = umma_desc_k_sw128(a_addr + u * Cfg::kSubBytes);
            const uint64_t bdesc = umma_desc_k_sw128(a_addr + u * Cfg::kSubBytes + kATileBytes);
#pragma unroll
            for (int kk = 0; kk < BK / 16; ++kk)
              umma_bf16_pair(d, adesc + 2 * kk, bdesc + 2 * kk, idesc, (kb | u | kk) != 0);
          }
          umma_commit_pair(&empty_bar[s]);
        }
        if (ok) umma_commit_pair(&acc_full[buf]);
      }
    }
  } else {
    // ---- epilogue: thread = one of this CTA's 128 accumulator rows, 32 fp32 columns per tcgen05.ld ----
    pdl_wait();
    const int quarter = warp & 3;
    const uint32_t lane_off = uint32_t(quarter * 32) << 16;
    uint32_t lt = 0;
    for (int tile = pair; tile < total_tiles; tile += npairs, ++lt) {
      const uint32_t buf = lt & 1;
      const int m0 = (tile % tiles_m) * (2 * BM) + (int)rank * BM, n0 = (tile / tiles_m) * BN;
      const int row = m0 + quarter * 32 + lane;
      const bool row_ok = row < p.M;
      uint4* bias_w = bias_s + quarter * 32;
      stage_bias(p, bias_w, lane, n0, BN);
      // residual epilogue (images of fewer than 32 rows take the row-per-thread path below): the first chunk
      // of `out` is on its way while the accumulator is computed
      const bool resid = RESID && (p.rows_per_image >= 32 || p.epilogue == EPI_F32);
      ResidRows rr;
      float4 xa[8], xb[8];
      if (resid) {
        rr = resid_rows(p, lane, m0 + quarter * 32);
        residual_load_x(p, rr, xa, lane, n0);
      }
      if (!mbar_wait(&acc_full[buf], (lt >> 1) & 1)) { report(p.status, DEV_TIMEOUT_EPI); break; }
      tc_fence_after();
      const int img = row_ok ? row / p.rows_per_image : 0;
      const int jrow = row_ok ? row - img * p.rows_per_image : 0;
      const uint32_t t0 = tmem_base + lane_off + buf * Cfg::kAccStride;
      if (resid) {   // whole warp: rows are re-distributed over the lanes
        float* tile_s = resid_s + quarter * (32 * kResidTilePitch);
#pragma unroll 1
        for (int ch = 0; ch < BN / 32; ++ch) {   // rolled: the code of one chunk is fetched once and then reused
          uint32_t r0[32];
          tmem_ld32(t0 + 32 * ch, r0);
          if (ch + 1 < BN / 32) residual_load_x(p, rr, xb, lane, n0 + 32 * (ch + 1));
          tmem_wait_ld();
          if (ch == BN / 32 - 1) {  // accumulator fully in registers: hand the buffer back to the MMA warp
            tc_fence_before();
            mbar_arrive_cluster(&acc_empty[buf], 0);
          }
          if (n0 + 32 * ch < p.N) residual_chunk(p, rr, r0, xa, tile_s, lane, n0 + 32 * ch, bias_w + 4 * ch);
#pragma unroll
          for (int i = 0; i < 8; ++i) xa[i] = xb[i];
        }
      } else {
#pragma unroll 1
        for (int c0 = 0; c0 < BN; c0 += 64) {
          uint32_t r0[32], r1[32];
          tmem_ld32(t0 + c0, r0);
          tmem_ld32(t0 + c0 + 32, r1);
          tmem_wait_ld();
          if (c0 + 64 >= BN) {  // accumulator fully in registers: hand the buffer back to the leader's MMA warp
            tc_fence_before();
            mbar_arrive_cluster(&acc_empty[buf], 0);
          }
          const int col = n0 + c0;
          if (row_ok && col < p.N) epilogue_chunk(p, r0, row, img, jrow, col, bias_w + c0 / 8);
          if (row_ok && col + 32 < p.N) epilogue_chunk(p, r1, row, img, jrow, col + 32, bias_w + c0 / 8 + 4);
        }
      }
    }
  }
  // Neither CTA may leave (or free tensor memory) while the other can still signal it or read its operands.
  tc_fence_before();
  cluster_sync_all();
  if (warp == 1) {
    __syncwarp();
    tmem_dealloc_pair(tmem_base, Cfg::kTmemCols);
  }
}

int g_pair_sms = 148;

}  // namespace

template <int BN, bool RESID> static cudaError_t set_pair_attr() {
  return cudaFuncSetAttribute(gemm_pair_kernel<BN, RESID>, cudaFuncAttributeMaxDynamicSharedMemorySize, PairCfg<BN>::smem_bytes(RESID));
}

cudaError_t gemm_pair_init() {
  cudaError_t e = set_pair_attr<256, false>();
  if (e == cudaSuccess) e = set_pair_attr<128, false>();
  if (e == cudaSuccess) e = set_pair_attr<256, true>();
  if (e == cudaSuccess) e = set_pair_attr<128, true>();
  if (e != cudaSuccess) return e;
  int dev = 0;
  e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return e;
  return cudaDeviceGetAttribute(&g_pair_sms, cudaDevAttrMultiProcessorCount, dev);
}

cudaError_t launch_gemm_pair(const GemmArgs& g, const GemmDev& p, int bn, cudaStream_t st) {
  alignas(64) CUtensorMap tmA, tmB;
  if (!make_tmap_bf16_2d(&tmA, g.a, g.M, g.K, BM)) return cudaErrorInvalidValue;
  if (!make_tmap_bf16_2d(&tmB, g.w, g.N, g.K, bn / 2)) return cudaErrorInvalidValue;
  const long tiles = (long)((g.M + 2 * BM - 1) / (2 * BM)) * ((g.N + bn - 1) / bn);
  const int max_pairs = g_pair_sms / 2;
  const int pairs = (int)(tiles < max_pairs ? tiles : max_pairs);
  const bool resid = p.epilogue == EPI_RESIDUAL || p.epilogue == EPI_F32;
  if (bn == 256 && resid) return launch_pdl(gemm_pair_kernel<256, true>, dim3(2 * pairs), dim3(kThreads), PairCfg<256>::smem_bytes(true), st, tmA, tmB, p);
  if (bn == 128 && resid) return launch_pdl(gemm_pair_kernel<128, true>, dim3(2 * pairs), dim3(kThreads), PairCfg<128>::smem_bytes(true), st, tmA, tmB, p);
  if (bn == 256) return launch_pdl(gemm_pair_kernel<256, false>, dim3(2 * pairs), dim3(kThreads), PairCfg<256>::smem_bytes(false), st, tmA, tmB, p);
  if (bn == 128) return launch_pdl(gemm_pair_kernel<128, false>, dim3(2 * pairs), dim3(kThreads), PairCfg<128>::smem_bytes(false), st, tmA, tmB, p);
  return cudaErrorInvalidValue;
}

}  // namespace fv
