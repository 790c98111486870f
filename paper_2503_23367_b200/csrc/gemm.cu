// tcgen05 GEMM for the transformer sublayers run on the kept rows (Fig. 3b: "Attention or FFN layers
// using FastVAR"): out = epilogue(A[M,K] * W[N,K]^T + bias), bf16 operands, fp32 accumulation in TMEM.
//
// Persistent kernel: one CTA per SM walks over 128 x BN output tiles (tile t = blockIdx.x + i*gridDim.x,
// m fastest so that the CTAs running together share W tiles in L2).  Warp roles:
//   warp 0   : TMA producer -- streams 128x64 A tiles and BNx64 W tiles (128-byte swizzle) through a
//              ring of shared-memory stages guarded by full/empty mbarriers; the ring runs across tiles.
//   warp 1   : allocates TMEM (two accumulators of BN columns), and one lane issues tcgen05.mma
//              (M=128, N=BN, K=16) four times per stage; tcgen05.commit releases the stage and, after
//              the last k-block of a tile, signals that tile's accumulator.
//   warps 2-5: epilogue -- tcgen05.ld the accumulator (thread = row, 32 columns at a time), fuse bias /
//              GELU / gate+residual / the Q | K-cache | V^T-cache split, and store; the accumulator is
//              handed back as soon as it is in registers, so the epilogue of tile i runs under the
//              MMAs of tile i+1.
// BN (128 / 192 / 256) is picked per shape on the host to minimise rounds x tile width on the SM count.
// Shapes with too few tiles to occupy the GPU (the small scale steps, where the GEMM is a stream of
// weights) are split along K: work item = (tile, K slice), every slice leaves its fp32 partial rows in
// a scratch buffer, and the last slice of a tile to arrive adds them in slice order and runs the
// epilogue, so the result does not depend on arrival order.  A K-split launch has one work item per CTA.
// Every wait is bounded; on expiry a code is written to the status word and the CTA unwinds normally.
#include <cuda.h>
#include <cuda_bf16.h>

#include <mutex>

#include "gemm_epilogue.cuh"
#include "internal.h"
#include "sm100.cuh"

namespace fv {

using namespace gemm_detail;

namespace {

constexpr int BM = 128;
constexpr int BK = 64;
constexpr int kGemmThreads = 192;
constexpr int kATileBytes = BM * BK * 2;  // 16 KB

// kKps: k-blocks per pipeline stage.  The MMA-issuing thread pays a fixed price per stage (the wait on the full barrier
// and the commit that frees the stage: about 0.2 us of dependent instructions), which for tiles of up to 128 columns
// exceeds the time of the stage's MMAs; with two k-blocks behind one barrier it is paid half as often.  The wider
// tiles keep one k-block per stage: their MMAs take that long anyway, and two k-blocks would leave two stages.
template <int BN> struct GemmCfg {
  static constexpr int kKps = (BN <= 128) ? 2 : 1;
  static constexpr int kBTileBytes = BN * BK * 2;
  static constexpr int kSubBytes = kATileBytes + kBTileBytes;   // one k-block: A tile, then W tile
  static constexpr int kStageBytes = kKps * kSubBytes;
  static constexpr int kStages = (BN == 256) ? 4 : (BN == 192 ? 5 : (BN == 128 ? 3 : 4));
  static constexpr int kTmemCols = (BN <= 64) ? 128 : ((BN == 128) ? 256 : 512);  // two accumulators, power of two
  static constexpr int kAccStride = (BN <= 64) ? 64 : ((BN == 128) ? 128 : 256);  // column offset of the second accumulator
  // operand stages | per-warp bias slices | barriers | (residual-epilogue kernels only) one turning tile per warp
  static constexpr int smem_bytes(bool resid) {
    return kStages * kStageBytes + kBiasSmemBytes + 256 /*barriers*/ + (resid ? kResidSmemBytes : 0) + 1024 /*alignment slack*/;
  }
};

// KIND 1 (RESID): the instantiation launched for the residual epilogue.  It is a kernel of its own because that epilogue
// needs ~90 more registers per thread; the others stay small enough for a bandwidth-bound kernel of another
// stream (the restoration of the rows that were not kept) to share the SMs with them.
template <int BN, bool SPLIT, int KIND>
__global__ void __launch_bounds__(kGemmThreads, 1)
gemm_bf16_kernel(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmB, const GemmDev p) {
  using Cfg = GemmCfg<BN>;
  constexpr int STAGES = Cfg::kStages;
  constexpr int KPS = Cfg::kKps;
  constexpr bool RESID = KIND == 1;   // KIND 2: the QKV projection with cosine attention / rotary positions on Q and K
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  uint4* bias_s = reinterpret_cast<uint4*>(smem + STAGES * Cfg::kStageBytes);   // per-warp bias slice of the tile
  uint64_t* full_bar = reinterpret_cast<uint64_t*>(smem + STAGES * Cfg::kStageBytes + kBiasSmemBytes);
  float* resid_s = reinterpret_cast<float*>(smem + STAGES * Cfg::kStageBytes + kBiasSmemBytes + 256);   // RESID: one tile per warp
  uint64_t* empty_bar = full_bar + STAGES;
  uint64_t* acc_full = empty_bar + STAGES;   // [2]
  uint64_t* acc_empty = acc_full + 2;        // [2]
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(acc_empty + 2);
  volatile int* sk_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);
  uint64_t* fix_bar = reinterpret_cast<uint64_t*>(tmem_slot + 2);  // K-split: arrival of the slices' partials

  pdl_trigger();
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int tiles_m = (p.M + BM - 1) / BM;
  const int tiles_n = (p.N + BN - 1) / BN;
  const int splits = SPLIT ? p.splits : 1;
  const int total_tiles = tiles_m * tiles_n * splits;   // work items: (tile, K slice), slice fastest
  const int num_kb = (p.K + BK - 1) / BK;

  if (threadIdx.x == 0) {
    for (int s = 0; s < STAGES; ++s) { mbar_init(&full_bar[s], 1); mbar_init(&empty_bar[s], 1); }
    for (int s = 0; s < 2; ++s) { mbar_init(&acc_full[s], 1); mbar_init(&acc_empty[s], 128); }
    if (SPLIT) mbar_init(fix_bar, 1);
    mbar_fence_init();
    tma_prefetch_desc(&tmA);
    tma_prefetch_desc(&tmB);
  }
  if (warp == 1) { tmem_alloc(tmem_slot, Cfg::kTmemCols); tmem_relinquish(); }
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
      int pre = 0;  // stages of the first work item whose W tile is already on its way
      if ((int)blockIdx.x < total_tiles) {
        const int tile = (int)blockIdx.x / splits, slice = (int)blockIdx.x - tile * splits;
        const int n0 = (tile / tiles_m) * BN;
        const int kb0 = slice * p.kb_per_split, kb1 = min(num_kb, kb0 + p.kb_per_split);
        pre = min(STAGES, (kb1 - kb0 + KPS - 1) / KPS);
        for (int i = 0; i < pre; ++i) {
          mbar_expect_tx(&full_bar[i], Cfg::kStageBytes);
          for (int u = 0; u < KPS; ++u)   // (a k-block beyond K reads zeros)
            tma_load_2d(smem + i * Cfg::kStageBytes + u * Cfg::kSubBytes + kATileBytes, &tmB, (kb0 + KPS * i + u) * BK, n0, &full_bar[i]);
        }
      }
      pdl_wait();
      for (int item = blockIdx.x; ok && item < total_tiles; item += gridDim.x) {
        const int tile = item / splits, slice = item - tile * splits;
        const int m0 = (tile % tiles_m) * BM, n0 = (tile / tiles_m) * BN;
        const int kb0 = slice * p.kb_per_split, kb1 = min(num_kb, kb0 + p.kb_per_split);
        for (int kb = kb0; kb < kb1; kb += KPS, ++it) {   // one stage: KPS k-blocks of this work item
          const int s = it % STAGES;
          uint8_t* a_s = smem + s * Cfg::kStageBytes;
          if ((int)it < pre) {  // W tiles requested before the wait: only the activations are missing
            for (int u = 0; u < KPS; ++u) tma_load_2d(a_s + u * Cfg::kSubBytes, &tmA, (kb + u) * BK, m0, &full_bar[s]);
            continue;
          }
          const uint32_t ph = (it / STAGES) & 1;
          if (!mbar_wait(&empty_bar[s], ph ^ 1)) { report(p.status, DEV_TIMEOUT_TMA); ok = false; break; }
          mbar_expect_tx(&full_bar[s], Cfg::kStageBytes);
          for (int u = 0; u < KPS; ++u) {
            tma_load_2d(a_s + u * Cfg::kSubBytes, &tmA, (kb + u) * BK, m0, &full_bar[s]);
            tma_load_2d(a_s + u * Cfg::kSubBytes + kATileBytes, &tmB, (kb + u) * BK, n0, &full_bar[s]);
          }
        }
      }
    }
  } else if (warp == 1) {
    pdl_wait();
    if (lane == 0) {
      constexpr uint32_t idesc = umma_idesc_bf16(BM, BN);
      uint32_t it = 0, lt = 0;
      bool ok = true;
      for (int item = blockIdx.x; ok && item < total_tiles; item += gridDim.x, ++lt) {
        const uint32_t buf = lt & 1;
        if (!mbar_wait(&acc_empty[buf], ((lt >> 1) & 1) ^ 1)) { report(p.status, DEV_TIMEOUT_MMA); ok = false; break; }
        tc_fence_after();
        const uint32_t d = tmem_base + buf * Cfg::kAccStride;
        const int slice = item % splits;
        const int kb0 = slice * p.kb_per_split, kb1 = min(num_kb, kb0 + p.kb_per_split);
        for (int kb = kb0; kb < kb1; kb += KPS, ++it) {
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
              umma_bf16(d, adesc + 2 * kk, bdesc + 2 * kk, idesc, (kb > kb0) || (u | kk) != 0);
          }
          umma_commit(&empty_bar[s]);
        }
        if (ok) umma_commit(&acc_full[buf]);
      }
    }
  } else {
    // ---- epilogue: thread = one accumulator row, 32 fp32 columns per tcgen05.ld ----
    pdl_wait();
    const int quarter = warp & 3;
    const uint32_t lane_off = uint32_t(quarter * 32) << 16;
    uint32_t lt = 0;
    for (int item = blockIdx.x; item < total_tiles; item += gridDim.x, ++lt) {
      const uint32_t buf = lt & 1;
      const int tile = item / splits, slice = item - tile * splits;
      const int m0 = (tile % tiles_m) * BM, n0 = (tile / tiles_m) * BN;
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
            mbar_arrive(&acc_empty[buf]);
          }
          if (n0 + 32 * ch < p.N) residual_chunk(p, rr, r0, xa, tile_s, lane, n0 + 32 * ch, bias_w + 4 * ch);
#pragma unroll
          for (int i = 0; i < 8; ++i) xa[i] = xb[i];
        }
      } else if (KIND == 2) {
        qkv_extras_tile<BN>(p, t0, row, row_ok, img, jrow, n0, bias_w);
        tc_fence_before();
        mbar_arrive(&acc_empty[buf]);
      } else if (!SPLIT) {
#pragma unroll 1
        for (int c0 = 0; c0 < BN; c0 += 64) {
          // two chunks in flight: the second load overlaps the first chunk's stores
          uint32_t r0[32], r1[32];
          tmem_ld32(t0 + c0, r0);
          tmem_ld32(t0 + c0 + 32, r1);
          tmem_wait_ld();
          if (c0 + 64 >= BN) {  // accumulator fully in registers: hand the buffer back to the MMA warp
            tc_fence_before();
            mbar_arrive(&acc_empty[buf]);
          }
          const int col = n0 + c0;
          if (row_ok && col < p.N) epilogue_chunk(p, r0, row, img, jrow, col, bias_w + c0 / 8);
          if (row_ok && col + 32 < p.N) epilogue_chunk(p, r1, row, img, jrow, col + 32, bias_w + c0 / 8 + 4);
        }
      } else {
        // ---- K-split: park this slice's partial rows, then the last slice to arrive finishes the tile
        float* mine = p.sk_partial + ((size_t)item * BM + (quarter * 32 + lane)) * BN;
#pragma unroll 1
        for (int c0 = 0; c0 < BN; c0 += 32) {
          uint32_t r0[32];
          tmem_ld32(t0 + c0, r0);
          tmem_wait_ld();
          if (row_ok && n0 + c0 < p.N) {
#pragma unroll
            for (int g = 0; g < 8; ++g)
              __stcg(reinterpret_cast<uint4*>(mine + c0) + g, make_uint4(r0[4 * g], r0[4 * g + 1], r0[4 * g + 2], r0[4 * g + 3]));
          }
        }
        tc_fence_before();
        mbar_arrive(&acc_empty[buf]);
        __threadfence();
        asm volatile("bar.sync 1, 128;" ::: "memory");
        if (threadIdx.x == 64) {
          const unsigned int prev = atomicAdd(p.sk_tickets + tile, 1u);
          const int last = (prev == (unsigned int)(p.splits - 1));
          if (last) p.sk_tickets[tile] = 0u;
          *sk_flag = last;
        }
        asm volatile("bar.sync 1, 128;" ::: "memory");
        const int last = *sk_flag;
        asm volatile("bar.sync 1, 128;" ::: "memory");  // flag consumed before the next item may rewrite it
        if (last) {
          // The slices' partial rows are pulled into the (now idle) operand stages with bulk copies --
          // one CTA cannot keep enough ordinary loads in flight to fetch them quickly -- and added
          // there in slice order, the running sum living in slot 0; then every thread takes its row.
          __threadfence();
          const int et = threadIdx.x - 64;                       // 0..127 among the epilogue threads
          const int rows_valid = min(BM, p.M - m0);
          const uint32_t slice_bytes = (uint32_t)rows_valid * BN * 4;
          const int max_slots = (STAGES * Cfg::kStageBytes) / (int)slice_bytes;   // >= 3
          const float* src0 = p.sk_partial + (size_t)tile * p.splits * BM * BN;
          float4* slot0 = reinterpret_cast<float4*>(smem);
          const int nf4 = rows_valid * (BN / 4);
          int done = 0;
          uint32_t phase = 0;
          bool ok = true;
          while (done < p.splits) {
            const int first_slot = done == 0 ? 0 : 1;
            const int cnt = min(max_slots - first_slot, p.splits - done);
            if (cnt <= 0) { report(p.status, DEV_TIMEOUT_EPI); ok = false; break; }   // cannot happen while a slice fits the stages twice over
            if (et == 0) {
              fence_proxy_async_all();   // earlier generic accesses to these slots / partials before the copies
              mbar_expect_tx(fix_bar, (uint32_t)cnt * slice_bytes);
              for (int i = 0; i < cnt; ++i)
                bulk_load_1d(smem + (size_t)(first_slot + i) * slice_bytes, src0 + (size_t)(done + i) * BM * BN, slice_bytes, fix_bar);
            }
            if (!mbar_wait(fix_bar, phase)) { report(p.status, DEV_TIMEOUT_EPI); ok = false; break; }
            phase ^= 1;
            const int last_slot = first_slot + cnt - 1;
            for (int f = et; f < nf4; f += 128) {
              float4 acc = slot0[f];
              for (int i = 1; i <= last_slot; ++i) {
                const float4 v = reinterpret_cast<const float4*>(smem + (size_t)i * slice_bytes)[f];
                acc.x += v.x; acc.y += v.y; acc.z += v.z; acc.w += v.w;
              }
              slot0[f] = acc;
            }
            done += cnt;
            asm volatile("bar.sync 1, 128;" ::: "memory");
          }
          if (ok && row_ok) {
            const float4* mysum = slot0 + (size_t)(quarter * 32 + lane) * (BN / 4);
#pragma unroll 1
            for (int c0 = 0; c0 < BN; c0 += 32) {
              const int col = n0 + c0;
              if (col >= p.N) break;
              uint32_t r0[32];
#pragma unroll
              for (int g = 0; g < 8; ++g) {
                const float4 v = mysum[c0 / 4 + g];
                r0[4 * g] = __float_as_uint(v.x); r0[4 * g + 1] = __float_as_uint(v.y);
                r0[4 * g + 2] = __float_as_uint(v.z); r0[4 * g + 3] = __float_as_uint(v.w);
              }
              epilogue_chunk(p, r0, row, img, jrow, col, bias_w + c0 / 8);
            }
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

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*, const cuuint64_t*,
                                  const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                                  CUtensorMapL2promotion, CUtensorMapFloatOOBfill);
EncodeTiledFn g_encode = nullptr;
int g_num_sms = 148;
std::once_flag g_encode_once;

void load_encode() {
  void* fn = nullptr;
  cudaDriverEntryPointQueryResult qres;
  if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &qres) == cudaSuccess &&
      qres == cudaDriverEntryPointSuccess)
    g_encode = reinterpret_cast<EncodeTiledFn>(fn);
}

template <int BN, bool SPLIT, int KIND> cudaError_t set_attr() {
  return cudaFuncSetAttribute(gemm_bf16_kernel<BN, SPLIT, KIND>, cudaFuncAttributeMaxDynamicSharedMemorySize, GemmCfg<BN>::smem_bytes(KIND == 1));
}

}  // namespace

bool make_tmap_bf16_2d(void* tmap_out, const void* base, uint64_t rows, uint64_t cols, uint32_t box_rows) {
  std::call_once(g_encode_once, load_encode);
  if (!g_encode) return false;
  cuuint64_t dims[2] = {cols, rows};
  cuuint64_t strides[1] = {cols * 2};
  cuuint32_t box[2] = {64, box_rows};
  cuuint32_t estr[2] = {1, 1};
  CUresult r = g_encode(static_cast<CUtensorMap*>(tmap_out), CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(base), dims,
                        strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                        CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  return r == CUDA_SUCCESS;
}

cudaError_t gemm_init() {
  cudaError_t e = set_attr<128, false, 0>();
  if (e == cudaSuccess) e = set_attr<128, true, 0>();
  if (e == cudaSuccess) e = set_attr<192, false, 0>();
  if (e == cudaSuccess) e = set_attr<256, false, 0>();
  if (e == cudaSuccess) e = set_attr<128, false, 1>();
  if (e == cudaSuccess) e = set_attr<192, false, 1>();
  if (e == cudaSuccess) e = set_attr<256, false, 1>();
  if (e == cudaSuccess) e = set_attr<64, false, 0>();
  if (e == cudaSuccess) e = set_attr<64, true, 0>();
  if (e == cudaSuccess) e = set_attr<64, false, 1>();
  if (e == cudaSuccess) e = set_attr<128, false, 2>();
  if (e == cudaSuccess) e = set_attr<192, false, 2>();
  if (e == cudaSuccess) e = set_attr<256, false, 2>();
  if (e == cudaSuccess) e = gemm_pair_init();
  if (e == cudaSuccess) e = gemm_cluster_init();
  if (e != cudaSuccess) return e;
  int dev = 0;
  e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return e;
  return cudaDeviceGetAttribute(&g_num_sms, cudaDevAttrMultiProcessorCount, dev);
}

// Kernel and tile width for a shape.  Measured on B200 (launches replayed from a CUDA graph, so that the host does
// not pace them), one launch costs about
//     fixed + rounds x (per_round + k-blocks x per_kblock)
// where rounds = ceil(tiles / resident CTAs or pairs).  A k-block of a 128-wide tile is paced by the thread that
// issues its MMAs (two k-blocks per pipeline stage there), the wider tiles by the MMAs themselves and the operand
// loads; wider tiles and CTA pairs win by needing fewer rounds and less L2 traffic per flop.
struct TileChoice { int bn; bool pair; };
static TileChoice pick_tile(int M, int N, int K, int sms) {
  const int num_kb = (K + BK - 1) / BK;
  struct Cand { int bn; bool pair; double fixed_us, round_us, kb_us; };
  // least-squares fit over M 256 ... 3277 x the four projection shapes of a 2048-wide block, every candidate forced
  const Cand cand[5] = {{128, false, 2.23, 0.98, 0.235}, {192, false, 2.16, 2.19, 0.292}, {256, false, 1.17, 3.01, 0.349},
                        {256, true, 3.99, 2.30, 0.316}, {64, false, 2.9, 0.5, 0.21}};
  TileChoice best{128, false};
  double best_cost = 1e30;
  for (const Cand& c : cand) {
    if (c.pair && M <= 256) continue;
    const int rows = c.pair ? 256 : 128;
    const int slots = c.pair ? sms / 2 : sms;
    const long tiles = (long)((M + rows - 1) / rows) * ((N + c.bn - 1) / c.bn);
    const long rounds = (tiles + slots - 1) / slots;
    const double cost = c.fixed_us + (double)rounds * (c.round_us + num_kb * c.kb_us);
    if (cost < best_cost - 1e-9) { best_cost = cost; best = TileChoice{c.bn, c.pair}; }
  }
  return best;
}

// K-split scratch: room for two work items per SM of the widest tile, after 4 KB of arrival counters.
constexpr size_t kSplitTicketBytes = 4096;
constexpr int kSplitMaxItems = 2 * 148;
size_t gemm_splitk_ticket_bytes() { return kSplitTicketBytes; }
size_t gemm_splitk_ws_bytes() { return kSplitTicketBytes + (size_t)kSplitMaxItems * BM * 128 * sizeof(float); }

// How many K slices for a shape that leaves SMs idle.  A CTA's operand pipeline is bound by load latency
// (a k-block every ~0.3 us whatever the tile), so spreading a tile's k-blocks over idle CTAs pays --
// until the last arriver's work, pulling slices x rows x 512 bytes back in, outweighs it.  Measured:
// long K (>= 64 k-blocks) gains at any row count with >= 16 k-blocks per slice; short K only gains
// while rows x slices stays small (<= 256) and there are at least 4 slices of >= 4 k-blocks.
static int pick_splits(long tiles, int M, int num_kb, int sms) {
  if (tiles * 2 > sms || num_kb < 16) return 1;
  int s = (int)(sms / tiles);
  if (num_kb >= 64) {
    const int rows = M < 128 ? M : 128;
    if (s > num_kb / 16) s = num_kb / 16;
    if (s > 512 / rows) s = 512 / rows;
    if (s < 2) return 1;
  } else {
    const int rows = M < 128 ? M : 128;
    if (s > num_kb / 4) s = num_kb / 4;
    if (s > 256 / rows) s = 256 / rows;
    if (s < 4) return 1;
  }
  const int per = (num_kb + s - 1) / s;
  return (num_kb + per - 1) / per;  // no empty slice
}

template <int BN>
static cudaError_t launch_bn(const GemmArgs& g, const GemmDev& p, int tiles_m, cudaStream_t st) {
  alignas(64) CUtensorMap tmA, tmB;
  if (!make_tmap_bf16_2d(&tmA, g.a, g.M, g.K, BM)) return cudaErrorInvalidValue;
  if (!make_tmap_bf16_2d(&tmB, g.w, g.N, g.K, BN)) return cudaErrorInvalidValue;
  const long tiles = (long)tiles_m * ((g.N + BN - 1) / BN) * p.splits;
  const int grid = (int)(tiles < g_num_sms ? tiles : g_num_sms);
  if (p.splits > 1) {
    if constexpr (BN <= 128) return launch_pdl(gemm_bf16_kernel<BN, true, 0>, dim3(grid), dim3(kGemmThreads), GemmCfg<BN>::smem_bytes(false), st, tmA, tmB, p);
    else return cudaErrorInvalidValue;
  } else {
    if (p.epilogue == EPI_RESIDUAL || p.epilogue == EPI_F32)
      return launch_pdl(gemm_bf16_kernel<BN, false, 1>, dim3(grid), dim3(kGemmThreads), GemmCfg<BN>::smem_bytes(true), st, tmA, tmB, p);
    if constexpr (BN < 128)
      if (p.epilogue == EPI_QKV_SPLIT && (p.qk_scale || p.rope_table)) return cudaErrorInvalidValue;   // never chosen for them
    if constexpr (BN >= 128)
      if (p.epilogue == EPI_QKV_SPLIT && (p.qk_scale || p.rope_table))
        return launch_pdl(gemm_bf16_kernel<BN, false, 2>, dim3(grid), dim3(kGemmThreads), GemmCfg<BN>::smem_bytes(false), st, tmA, tmB, p);
    return launch_pdl(gemm_bf16_kernel<BN, false, 0>, dim3(grid), dim3(kGemmThreads), GemmCfg<BN>::smem_bytes(false), st, tmA, tmB, p);
  }
}

static int g_force_path = 0;
void gemm_force_path(int path) { g_force_path = path; }

fv_status launch_gemm(const GemmArgs& g, cudaStream_t st) {
  if (g.M <= 0 || g.N <= 0 || g.K <= 0 || (g.K % 8) || (g.N % 8) || !g.a || !g.w) return FV_ERR_INVALID_ARG;
  if (g.rows_per_image <= 0) return FV_ERR_INVALID_ARG;
  if (g.epilogue == EPI_QKV_SPLIT && (g.C % 128 || g.q_cols % 128)) return FV_ERR_UNSUPPORTED;
  const int tiles_m = (g.M + BM - 1) / BM;
  TileChoice tc = pick_tile(g.M, g.N, g.K, g_num_sms);
  // Few rows against a narrow output (the out-projections and the second MLP GEMM of the small scale steps):
  // 64-wide tiles double the CTAs that stream the weight matrix.  Measured (M <= 128, N = 2048): 9.7 us instead
  // of 11.4 at M = 32, K = 2048; 20.6 instead of 30.1 at M = 128, K = 8192; wider outputs and more rows lose.
  if (g.M <= 128 && g.N <= 2048 && g.N > 64) tc = TileChoice{64, false};
  if (g_force_path == 1 && tc.pair) tc = TileChoice{256, false};
  if (g_force_path == 2) tc = TileChoice{256, true};
  if (g_force_path == 3) tc = TileChoice{128, true};
  if (g_force_path >= 4 && g_force_path <= 6) tc = TileChoice{128 + 64 * (g_force_path - 4), false};
  if (g_force_path == 7) tc = TileChoice{64, false};
  // Q / K extras (cosine attention, rotary positions): one-CTA tiles that hold whole heads, no K split
  const bool qk_extras = g.epilogue == EPI_QKV_SPLIT && (g.qk_scale || g.rope_table);
  if (qk_extras) {
    if (g.head_dim != 64 && g.head_dim != 128) return FV_ERR_UNSUPPORTED;
    if (tc.pair) tc = TileChoice{256, false};
    if (tc.bn < 128) tc.bn = 128;            // the extras exist for tiles of at least 128 columns
    if (tc.bn % g.head_dim) tc.bn = 256;
  }
  int bn = tc.bn;
  GemmDev p;
  p.splits = 1; p.kb_per_split = (g.K + BK - 1) / BK; p.sk_partial = nullptr; p.sk_tickets = nullptr;
  if (g.splitk_ws && !qk_extras) {
    const int num_kb = (g.K + BK - 1) / BK;
    const int bn_split = tc.bn == 64 ? 64 : 128;
    const long tiles128 = (long)tiles_m * ((g.N + bn_split - 1) / bn_split);
    const int sp = pick_splits(tiles128, g.M, num_kb, g_num_sms);
    if (sp > 1 && tiles128 * sp <= g_num_sms && tiles128 * sp <= kSplitMaxItems && tiles128 * sizeof(unsigned int) <= kSplitTicketBytes) {
      bn = bn_split;
      p.kb_per_split = (num_kb + sp - 1) / sp;
      p.kb_per_split += p.kb_per_split & 1;   // even: a pipeline stage may hold two k-blocks of ONE slice
      p.splits = (num_kb + p.kb_per_split - 1) / p.kb_per_split;   // no empty slice
      p.sk_tickets = static_cast<unsigned int*>(g.splitk_ws);
      p.sk_partial = reinterpret_cast<float*>(static_cast<char*>(g.splitk_ws) + kSplitTicketBytes);
    }
  }
  p.bias = static_cast<const __nv_bfloat16*>(g.bias);
  p.M = g.M; p.N = g.N; p.K = g.K; p.epilogue = g.epilogue; p.out = g.out; p.aux = g.aux; p.gamma = g.gamma;
  if (g.epilogue == EPI_F32) { p.aux = nullptr; p.gamma = nullptr; }
  p.mod_stride = g.mod_stride; p.rows_per_image = g.rows_per_image; p.q_cols = g.q_cols; p.C = g.C;
  p.k_cache = static_cast<__nv_bfloat16*>(g.k_cache); p.vt_cache = static_cast<__nv_bfloat16*>(g.vt_cache);
  p.kv_capacity = g.kv_capacity; p.kv_offset = g.kv_offset; p.status = g.status;
  p.qk_scale = qk_extras ? g.qk_scale : nullptr;
  p.rope_table = qk_extras ? reinterpret_cast<const float2*>(g.rope_table) : nullptr;
  p.rope_idx = qk_extras ? g.rope_idx : nullptr;
  p.head_dim = g.head_dim;
  // Few tiles against a long K (every GEMM of the small scale steps): split K over the CTAs of a cluster, the
  // partials reduced through distributed shared memory.  Measured back to back on B200 (us, against the best
  // of the other paths): N 2048 K 2048: 6.6 / 7.4 / 8.0 / 12.0 / 12.4 at M = 2 / 32 / 128 / 288 / 512 (9.7 /
  // 9.7 / 12.7 / 13.7 / 14.0); N 2048 K 8192: 14.9 / 15.0 / 15.9 / 26.9 / 27.5 (14.9 / 15.9 / 20.8 / 29.5 /
  // 35.6); N 6144 K 2048 at M <= 128: 13.2 / 11.4 / 13.8 (14.4 / 14.1 / 14.3); N 8192: 13.6 / 12.0 / 14.3
  // (17.7 / 14.6 / 15.1).  Which of the three shapes wins follows the tile counts:
  int cluster_slices = 0, cluster_bn = 0;
  if (g_force_path == 0 && !qk_extras) {
    const int num_kb = (g.K + BK - 1) / BK;
    const long t128 = (long)tiles_m * ((g.N + 127) / 128), t64 = (long)tiles_m * ((g.N + 63) / 64);
    // (re-measured GPU-bound after the narrow tiles took two k-blocks per pipeline stage: with more than 32 rows the
    // 128-wide x 2 cluster, whose ring has no room for that, only wins on a long K; 64-wide x 2 wins on a short one)
    if (num_kb >= 8) {
      if (g.M > 16 && t64 * 4 <= g_num_sms) { cluster_bn = 64; cluster_slices = 4; }
      else if (g.M > 16 && t64 * 2 <= g_num_sms && num_kb < 64) { cluster_bn = 64; cluster_slices = 2; }
      else if (t128 * 4 <= g_num_sms) { cluster_bn = 128; cluster_slices = 4; }
      else if (t128 * 2 <= g_num_sms && (g.M <= 32 || num_kb >= 64)) { cluster_bn = 128; cluster_slices = 2; }
    }
  }
  if (g_force_path >= 8 && g_force_path <= 11 && !qk_extras) {   // 8: 128 wide x 4 slices, 9: 128 x 2, 10: 64 x 4, 11: 64 x 2
    cluster_bn = g_force_path <= 9 ? 128 : 64;
    cluster_slices = (g_force_path & 1) ? 2 : 4;
  }
  if (cluster_slices) {
    const int num_kb = (g.K + BK - 1) / BK;
    p.splits = 1; p.sk_partial = nullptr; p.sk_tickets = nullptr;
    p.kb_per_split = (num_kb + cluster_slices - 1) / cluster_slices;
    p.kb_per_split += p.kb_per_split & 1;   // even: a pipeline stage of the cluster kernel may hold two k-blocks of ONE slice
  }
  LaunchScope scope(KC_GEMM, 1, 2.0 * g.M * (double)g.N * g.K, 2.0 * ((double)g.M * g.K + (double)g.N * g.K + (double)g.M * g.N), st);
  if (cluster_slices) return launch_gemm_cluster(g, p, cluster_bn, cluster_slices, st) == cudaSuccess ? FV_OK : FV_ERR_CUDA;
  if (p.splits == 1 && tc.pair) {
    cudaError_t e2 = launch_gemm_pair(g, p, bn, st);
    return e2 == cudaSuccess ? FV_OK : FV_ERR_CUDA;
  }
  cudaError_t e = bn == 256 ? launch_bn<256>(g, p, tiles_m, st)
                : (bn == 192 ? launch_bn<192>(g, p, tiles_m, st) : (bn == 64 ? launch_bn<64>(g, p, tiles_m, st) : launch_bn<128>(g, p, tiles_m, st)));
  return e == cudaSuccess ? FV_OK : FV_ERR_CUDA;
}

}  // namespace fv
