// K split inside a thread-block cluster: the GEMMs of the small scale steps (few rows against a large weight
// matrix) have too few output tiles to occupy the GPU, so S CTAs of one cluster share a tile and each takes
// 1/S of its k-blocks.  The partial accumulators never go through global memory: every CTA writes the rows
// that another CTA owns straight into that CTA's shared memory (distributed shared memory), one cluster
// barrier later every CTA adds the S partials of its own 128/S rows in rank order and runs the epilogue for
// them -- a reduce-scatter, so the work after the barrier shrinks with S instead of growing, and the result
// does not depend on timing.  No scratch buffer, no arrival counters.
//
// One tile per cluster, one accumulator of BN columns in TMEM per CTA; warp roles as in gemm.cu (warp 0 TMA
// producer, warp 1 MMA issuer, warps 2-5 accumulator readers / epilogue).  Every mbarrier wait is bounded; a
// CTA whose wait expires reports it and still takes part in the cluster barrier, so the others never hang.
#include <cuda.h>
#include <cuda_bf16.h>

#include "gemm_epilogue.cuh"
#include "internal.h"
#include "sm100.cuh"

namespace fv {

using namespace gemm_detail;

namespace {

constexpr int BM = 128;
constexpr int BK = 64;
constexpr int kThreads = 192;

// AROWS: rows of A that are actually loaded per k-block (32 when the GEMM has at most 32 rows, else 128).  The
// MMA always reads a 128-row A tile from shared memory; with AROWS = 32 the rows beyond the 4 KB that were
// loaded are whatever follows in shared memory (the stage's own W tile, the next stage, the buffers behind the
// ring -- all inside the allocation).  They only feed accumulator rows >= 32, which belong to no row of the
// output and are neither reduced nor stored.  The 12 KB saved per k-block buy a deeper ring.
//
// kKps: k-blocks per pipeline stage.  The thread that issues the MMAs is a chain of dependent instructions: per stage
// it spends about 0.16 us between its commit and seeing the next full barrier, 0.06 us on the commit and 0.03 us per
// MMA, so with one k-block per stage a k-block costs 0.34 us whatever its bytes (measured with device timestamps: no
// change without the A loads, with one MMA of four, with the weights resident in L2, with another weight pitch).
// Two k-blocks behind one barrier halve the per-stage part: 0.24 us per k-block.  Where the ring would shrink to two
// stages (128 rows of A against 128-wide tiles) one k-block per stage stays.
template <int BN, int AROWS> struct ClusterCfg {
  static constexpr int kKps = (AROWS == 128 && BN == 128) ? 1 : 2;
  static constexpr int kATile = AROWS * BK * 2;
  static constexpr int kBTileBytes = BN * BK * 2;
  static constexpr int kSubBytes = kATile + kBTileBytes;       // one k-block: A tile, then W tile
  static constexpr int kStageBytes = kKps * kSubBytes;
  static constexpr int kStages = AROWS == 32 ? ((BN == 128) ? 3 : 5) : ((BN == 128) ? 4 : 3);
  static constexpr int kTmemCols = BN;                      // one accumulator (64 or 128: powers of two)
  static constexpr int kRedPitch = BN + 4;                  // floats per row of the reduce buffer (bank spread)
  static constexpr int kRedBytes = BM * kRedPitch * 4;      // [S sources][128/S rows][pitch] = 128 rows in all
  // operand stages | per-warp bias slices | barriers | reduce buffer
  static constexpr int kSmemBytes = kStages * kStageBytes + kBiasSmemBytes + 256 + kRedBytes + 1024 /*alignment slack*/;
};

__device__ __forceinline__ uint32_t map_to_cta(const void* p, uint32_t cta) {
  uint32_t remote;
  asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(remote) : "r"(smem_u32(p)), "r"(cta));
  return remote;
}
__device__ __forceinline__ void st_cluster_f4(uint32_t addr, uint32_t a, uint32_t b, uint32_t c, uint32_t d) {
  asm volatile("st.shared::cluster.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(addr), "r"(a), "r"(b), "r"(c), "r"(d) : "memory");
}

template <int BN, int S, int AROWS>
__global__ void __launch_bounds__(kThreads, 1)
gemm_cluster_kernel(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmB, const GemmDev p) {
  using Cfg = ClusterCfg<BN, AROWS>;
  constexpr int kATileBytes = Cfg::kATile;
  constexpr int STAGES = Cfg::kStages;
  constexpr int KPS = Cfg::kKps;
  constexpr int ROWS_PER = BM / S;        // rows of the tile each CTA finishes
  constexpr int CHUNKS = BN / 32;         // 32-column chunks per row
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  uint4* bias_s = reinterpret_cast<uint4*>(smem + STAGES * Cfg::kStageBytes);
  uint64_t* full_bar = reinterpret_cast<uint64_t*>(smem + STAGES * Cfg::kStageBytes + kBiasSmemBytes);
  uint64_t* empty_bar = full_bar + STAGES;
  uint64_t* acc_full = empty_bar + STAGES;
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(acc_full + 1);
  float* red = reinterpret_cast<float*>(smem + STAGES * Cfg::kStageBytes + kBiasSmemBytes + 256);   // [S][ROWS_PER][pitch]

  pdl_trigger();
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const uint32_t rank = cluster_ctarank();
  const int tile = blockIdx.x / S;
  const int tiles_m = (p.M + BM - 1) / BM;
  const int m0 = (tile % tiles_m) * BM, n0 = (tile / tiles_m) * BN;
  const int num_kb = (p.K + BK - 1) / BK;
  const int kb0 = min(num_kb, (int)rank * p.kb_per_split), kb1 = min(num_kb, kb0 + p.kb_per_split);

  if (threadIdx.x == 0) {
    for (int s = 0; s < STAGES; ++s) { mbar_init(&full_bar[s], 1); mbar_init(&empty_bar[s], 1); }
    mbar_init(acc_full, 1);
    mbar_fence_init();
    tma_prefetch_desc(&tmA);
    tma_prefetch_desc(&tmB);
  }
  if (warp == 1) { tmem_alloc(tmem_slot, Cfg::kTmemCols); tmem_relinquish(); }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;
  // first half of the "every CTA of the cluster has started" barrier; the second half precedes the first
  // store into another CTA's shared memory (a rank with an empty K slice gets there almost at once)
  cluster_arrive_relaxed();

  if (warp == 0) {
    if (lane == 0) {
      // the weight tiles (never written by a kernel of the step) are requested before the dependency wait
      const int nst = (kb1 - kb0 + KPS - 1) / KPS;    // stages of KPS k-blocks; a k-block beyond K reads zeros
      const int pre = min(STAGES, nst);
      for (int i = 0; i < pre; ++i) {
        mbar_expect_tx(&full_bar[i], Cfg::kStageBytes);
        for (int u = 0; u < KPS; ++u)
          tma_load_2d(smem + i * Cfg::kStageBytes + u * Cfg::kSubBytes + kATileBytes, &tmB, (kb0 + KPS * i + u) * BK, n0, &full_bar[i]);
      }
      pdl_wait();
      for (int it = 0; it < nst; ++it) {
        const int s = it % STAGES;
        const int kb = kb0 + KPS * it;
        uint8_t* a_s = smem + s * Cfg::kStageBytes;
        if (it < pre) {
          for (int u = 0; u < KPS; ++u) tma_load_2d(a_s + u * Cfg::kSubBytes, &tmA, (kb + u) * BK, m0, &full_bar[s]);
          continue;
        }
        const uint32_t ph = (it / STAGES) & 1;
        if (!mbar_wait(&empty_bar[s], ph ^ 1)) { report(p.status, DEV_TIMEOUT_TMA); break; }
        mbar_expect_tx(&full_bar[s], Cfg::kStageBytes);
        for (int u = 0; u < KPS; ++u) {
          tma_load_2d(a_s + u * Cfg::kSubBytes, &tmA, (kb + u) * BK, m0, &full_bar[s]);
          tma_load_2d(a_s + u * Cfg::kSubBytes + kATileBytes, &tmB, (kb + u) * BK, n0, &full_bar[s]);
        }
      }
    }
  } else if (warp == 1) {
    pdl_wait();
    if (lane == 0) {
      constexpr uint32_t idesc = umma_idesc_bf16(BM, BN);
      bool ok = true;
      const int nst = (kb1 - kb0 + KPS - 1) / KPS;
      for (int it = 0; it < nst; ++it) {
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
            umma_bf16(tmem_base, adesc + 2 * kk, bdesc + 2 * kk, idesc, (it | u | kk) != 0);
        }
        umma_commit(&empty_bar[s]);
      }
      if (ok && kb1 > kb0) umma_commit(acc_full);
    }
  } else {
    // ---- accumulator readers: thread = one accumulator row; its partial goes to the CTA that owns the row ----
    pdl_wait();
    const int quarter = warp & 3;
    const int trow = quarter * 32 + lane;                 // row inside the tile
    const uint32_t owner = (uint32_t)(trow / ROWS_PER);
    const int lrow = trow - (int)owner * ROWS_PER;
    stage_bias(p, bias_s + quarter * 32, lane, n0, BN);
    bool have = kb1 > kb0;
    if (have && !mbar_wait(acc_full, 0)) { report(p.status, DEV_TIMEOUT_EPI); have = false; }
    have = __all_sync(0xffffffffu, have);   // the TMEM loads below are warp-wide
    tc_fence_after();
    cluster_wait();                         // every CTA of the cluster is running: its shared memory may be written
    const uint32_t dst = map_to_cta(red + ((size_t)rank * ROWS_PER + lrow) * Cfg::kRedPitch, owner);
    const uint32_t t0 = tmem_base + (uint32_t(quarter * 32) << 16);
#pragma unroll 1
    for (int c0 = 0; c0 < BN; c0 += 32) {
      uint32_t r[32];
      if (have) {            // uniform over the warp
        tmem_ld32(t0 + c0, r);
        tmem_wait_ld();
      } else {
#pragma unroll
        for (int i = 0; i < 32; ++i) r[i] = 0u;   // a slice without k-blocks (or an expired wait) adds nothing
      }
      if (m0 + trow < p.M) {
#pragma unroll
        for (int g = 0; g < 8; ++g) st_cluster_f4(dst + (c0 + 4 * g) * 4, r[4 * g], r[4 * g + 1], r[4 * g + 2], r[4 * g + 3]);
      }
    }
    tc_fence_before();
  }
  // Every thread of every CTA of the cluster: the partials are in place after this barrier, and no CTA is
  // written to afterwards (so each may finish and exit on its own).
  __syncwarp();
  if (warp < 2) cluster_wait();             // completes these warps' half of the start-up barrier
  cluster_sync_all();
  if (warp >= 2) {
    const int e = threadIdx.x - 64;                        // 0..127
    const uint4* bias_w = bias_s + (warp & 3) * 32;
    for (int ci = e; ci < ROWS_PER * CHUNKS; ci += 128) {
      const int lrow = ci / CHUNKS, ch = ci - lrow * CHUNKS;
      const int row = m0 + (int)rank * ROWS_PER + lrow;
      const int col = n0 + 32 * ch;
      if (row >= p.M || col >= p.N) continue;
      float acc[32];
      const float* src = red + (size_t)lrow * Cfg::kRedPitch + 32 * ch;
#pragma unroll
      for (int g = 0; g < 8; ++g) {
        const float4 v = *reinterpret_cast<const float4*>(src + 4 * g);
        acc[4 * g] = v.x; acc[4 * g + 1] = v.y; acc[4 * g + 2] = v.z; acc[4 * g + 3] = v.w;
      }
#pragma unroll
      for (int s = 1; s < S; ++s) {                        // rank order: the sum does not depend on timing
        const float* ss = src + (size_t)s * ROWS_PER * Cfg::kRedPitch;
#pragma unroll
        for (int g = 0; g < 8; ++g) {
          const float4 v = *reinterpret_cast<const float4*>(ss + 4 * g);
          acc[4 * g] += v.x; acc[4 * g + 1] += v.y; acc[4 * g + 2] += v.z; acc[4 * g + 3] += v.w;
        }
      }
      uint32_t r[32];
#pragma unroll
      for (int i = 0; i < 32; ++i) r[i] = __float_as_uint(acc[i]);
      const int img = row / p.rows_per_image;
      epilogue_chunk(p, r, row, img, row - img * p.rows_per_image, col, bias_w + 4 * ch);
    }
  }
  __syncthreads();
  if (warp == 1) {
    __syncwarp();
    tmem_dealloc(tmem_base, Cfg::kTmemCols);
  }
}

template <int BN, int S, int AROWS> cudaError_t set_attr() {
  return cudaFuncSetAttribute(gemm_cluster_kernel<BN, S, AROWS>, cudaFuncAttributeMaxDynamicSharedMemorySize, ClusterCfg<BN, AROWS>::kSmemBytes);
}

template <int BN, int S, int AROWS>
cudaError_t launch(const GemmArgs& g, const GemmDev& p, long tiles, cudaStream_t st) {
  alignas(64) CUtensorMap tmA, tmB;
  if (!make_tmap_bf16_2d(&tmA, g.a, g.M, g.K, AROWS)) return cudaErrorInvalidValue;
  if (!make_tmap_bf16_2d(&tmB, g.w, g.N, g.K, BN)) return cudaErrorInvalidValue;
  cudaLaunchConfig_t cfg{};
  cfg.gridDim = dim3((unsigned)(tiles * S)); cfg.blockDim = dim3(kThreads); cfg.dynamicSmemBytes = ClusterCfg<BN, AROWS>::kSmemBytes; cfg.stream = st;
  cudaLaunchAttribute at[2];
  at[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  at[0].val.programmaticStreamSerializationAllowed = 1;
  at[1].id = cudaLaunchAttributeClusterDimension;
  at[1].val.clusterDim.x = S; at[1].val.clusterDim.y = 1; at[1].val.clusterDim.z = 1;
  cfg.attrs = at; cfg.numAttrs = 2;
  return cudaLaunchKernelEx(&cfg, gemm_cluster_kernel<BN, S, AROWS>, tmA, tmB, p);
}

}  // namespace

cudaError_t gemm_cluster_init() {
  cudaError_t e = set_attr<128, 2, 128>();
  if (e == cudaSuccess) e = set_attr<128, 4, 128>();
  if (e == cudaSuccess) e = set_attr<64, 2, 128>();
  if (e == cudaSuccess) e = set_attr<64, 4, 128>();
  if (e == cudaSuccess) e = set_attr<128, 2, 32>();
  if (e == cudaSuccess) e = set_attr<128, 4, 32>();
  if (e == cudaSuccess) e = set_attr<64, 2, 32>();
  if (e == cudaSuccess) e = set_attr<64, 4, 32>();
  return e;
}

// bn in {64, 128}, slices in {2, 4}; p.kb_per_split k-blocks per CTA.
cudaError_t launch_gemm_cluster(const GemmArgs& g, const GemmDev& p, int bn, int slices, cudaStream_t st) {
  const long tiles = (long)((g.M + BM - 1) / BM) * ((g.N + bn - 1) / bn);
  if (g.M <= 32) {   // at most 32 rows: short A tiles, deeper ring
    if (bn == 128 && slices == 2) return launch<128, 2, 32>(g, p, tiles, st);
    if (bn == 128 && slices == 4) return launch<128, 4, 32>(g, p, tiles, st);
    if (bn == 64 && slices == 2) return launch<64, 2, 32>(g, p, tiles, st);
    if (bn == 64 && slices == 4) return launch<64, 4, 32>(g, p, tiles, st);
  }
  if (bn == 128 && slices == 2) return launch<128, 2, 128>(g, p, tiles, st);
  if (bn == 128 && slices == 4) return launch<128, 4, 128>(g, p, tiles, st);
  if (bn == 64 && slices == 2) return launch<64, 2, 128>(g, p, tiles, st);
  if (bn == 64 && slices == 4) return launch<64, 4, 128>(g, p, tiles, st);
  return cudaErrorInvalidValue;
}

}  // namespace fv
