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
// Every wait is bounded; on expiry a code is written to the status word and the CTA unwinds normally.
#include <cuda.h>
#include <cuda_bf16.h>

#include <mutex>

#include "internal.h"
#include "sm100.cuh"

namespace fv {

namespace {

constexpr int BM = 128;
constexpr int BK = 64;
constexpr int kGemmThreads = 192;
constexpr int kATileBytes = BM * BK * 2;  // 16 KB

template <int BN> struct GemmCfg {
  static constexpr int kBTileBytes = BN * BK * 2;
  static constexpr int kStageBytes = kATileBytes + kBTileBytes;
  static constexpr int kStages = (BN == 256) ? 4 : (BN == 192 ? 5 : 6);
  static constexpr int kTmemCols = (BN == 128) ? 256 : 512;  // two accumulators, power of two
  static constexpr int kAccStride = (BN == 128) ? 128 : 256;  // column offset of the second accumulator
  static constexpr int kSmemBytes = kStages * kStageBytes + 1024 /*alignment slack*/ + 256 /*barriers*/;
};

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

template <int BN>
__global__ void __launch_bounds__(kGemmThreads, 1)
gemm_bf16_kernel(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmB, const GemmDev p) {
  using Cfg = GemmCfg<BN>;
  constexpr int STAGES = Cfg::kStages;
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  uint64_t* full_bar = reinterpret_cast<uint64_t*>(smem + STAGES * Cfg::kStageBytes);
  uint64_t* empty_bar = full_bar + STAGES;
  uint64_t* acc_full = empty_bar + STAGES;   // [2]
  uint64_t* acc_empty = acc_full + 2;        // [2]
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(acc_empty + 2);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int tiles_m = (p.M + BM - 1) / BM;
  const int tiles_n = (p.N + BN - 1) / BN;
  const int total_tiles = tiles_m * tiles_n;
  const int num_kb = (p.K + BK - 1) / BK;

  if (threadIdx.x == 0) {
    for (int s = 0; s < STAGES; ++s) { mbar_init(&full_bar[s], 1); mbar_init(&empty_bar[s], 1); }
    for (int s = 0; s < 2; ++s) { mbar_init(&acc_full[s], 1); mbar_init(&acc_empty[s], 128); }
    mbar_fence_init();
    tma_prefetch_desc(&tmA);
    tma_prefetch_desc(&tmB);
  }
  if (warp == 1) { tmem_alloc(tmem_slot, Cfg::kTmemCols); tmem_relinquish(); }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;

  if (warp == 0) {
    if (lane == 0) {
      uint32_t it = 0;
      bool ok = true;
      for (int tile = blockIdx.x; ok && tile < total_tiles; tile += gridDim.x) {
        const int m0 = (tile % tiles_m) * BM, n0 = (tile / tiles_m) * BN;
        for (int kb = 0; kb < num_kb; ++kb, ++it) {
          const int s = it % STAGES;
          const uint32_t ph = (it / STAGES) & 1;
          if (!mbar_wait(&empty_bar[s], ph ^ 1)) { report(p.status, DEV_TIMEOUT_TMA); ok = false; break; }
          mbar_expect_tx(&full_bar[s], Cfg::kStageBytes);
          uint8_t* a_s = smem + s * Cfg::kStageBytes;
          tma_load_2d(a_s, &tmA, kb * BK, m0, &full_bar[s]);
          tma_load_2d(a_s + kATileBytes, &tmB, kb * BK, n0, &full_bar[s]);
        }
      }
    }
  } else if (warp == 1) {
    if (lane == 0) {
      constexpr uint32_t idesc = umma_idesc_bf16(BM, BN);
      uint32_t it = 0, lt = 0;
      bool ok = true;
      for (int tile = blockIdx.x; ok && tile < total_tiles; tile += gridDim.x, ++lt) {
        const uint32_t buf = lt & 1;
        if (!mbar_wait(&acc_empty[buf], ((lt >> 1) & 1) ^ 1)) { report(p.status, DEV_TIMEOUT_MMA); ok = false; break; }
        tc_fence_after();
        const uint32_t d = tmem_base + buf * Cfg::kAccStride;
        for (int kb = 0; kb < num_kb; ++kb, ++it) {
          const int s = it % STAGES;
          const uint32_t ph = (it / STAGES) & 1;
          if (!mbar_wait(&full_bar[s], ph)) { report(p.status, DEV_TIMEOUT_MMA); ok = false; break; }
          tc_fence_after();
          const uint32_t a_addr = smem_u32(smem + s * Cfg::kStageBytes);
          const uint64_t adesc = umma_desc_k_sw128(a_addr);
          const uint64_t bdesc = umma_desc_k_sw128(a_addr + kATileBytes);
#pragma unroll
          for (int kk = 0; kk < BK / 16; ++kk)
            umma_bf16(d, adesc + 2 * kk, bdesc + 2 * kk, idesc, (kb | kk) != 0);
          umma_commit(&empty_bar[s]);
        }
        if (ok) umma_commit(&acc_full[buf]);
      }
    }
  } else {
    // ---- epilogue: thread = one accumulator row, 32 fp32 columns per tcgen05.ld ----
    const int quarter = warp & 3;
    const uint32_t lane_off = uint32_t(quarter * 32) << 16;
    uint32_t lt = 0;
    for (int tile = blockIdx.x; tile < total_tiles; tile += gridDim.x, ++lt) {
      const uint32_t buf = lt & 1;
      const int m0 = (tile % tiles_m) * BM, n0 = (tile / tiles_m) * BN;
      const int row = m0 + quarter * 32 + lane;
      const bool row_ok = row < p.M;
      if (!mbar_wait(&acc_full[buf], (lt >> 1) & 1)) { report(p.status, DEV_TIMEOUT_EPI); break; }
      tc_fence_after();
      const int img = row_ok ? row / p.rows_per_image : 0;
      const int jrow = row_ok ? row - img * p.rows_per_image : 0;
      const uint32_t t0 = tmem_base + lane_off + buf * Cfg::kAccStride;
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
        if (row_ok && col < p.N) epilogue_chunk(p, r0, row, img, jrow, col);
        if (row_ok && col + 32 < p.N) epilogue_chunk(p, r1, row, img, jrow, col + 32);
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

template <int BN> cudaError_t set_attr() {
  return cudaFuncSetAttribute(gemm_bf16_kernel<BN>, cudaFuncAttributeMaxDynamicSharedMemorySize, GemmCfg<BN>::kSmemBytes);
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
  cudaError_t e = set_attr<128>();
  if (e == cudaSuccess) e = set_attr<192>();
  if (e == cudaSuccess) e = set_attr<256>();
  if (e != cudaSuccess) return e;
  int dev = 0;
  e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return e;
  return cudaDeviceGetAttribute(&g_num_sms, cudaDevAttrMultiProcessorCount, dev);
}

// Tile width for a shape: the persistent grid runs ceil(tiles / SMs) rounds of BN-wide tiles, so pick
// the BN with the smallest rounds x BN (128-wide tiles pay ~10 % for their shared-memory read rate).
static int pick_bn(int tiles_m, int N, int sms) {
  const int cand[3] = {256, 192, 128};
  int best = 128;
  double best_cost = 1e30;
  for (int bn : cand) {
    const long tiles = (long)tiles_m * ((N + bn - 1) / bn);
    const long rounds = (tiles + sms - 1) / sms;
    const double cost = (double)rounds * bn * (bn == 128 ? 1.1 : 1.0);
    if (cost < best_cost - 1e-9) { best_cost = cost; best = bn; }
  }
  return best;
}

template <int BN>
static cudaError_t launch_bn(const GemmArgs& g, const GemmDev& p, int tiles_m, cudaStream_t st) {
  alignas(64) CUtensorMap tmA, tmB;
  if (!make_tmap_bf16_2d(&tmA, g.a, g.M, g.K, BM)) return cudaErrorInvalidValue;
  if (!make_tmap_bf16_2d(&tmB, g.w, g.N, g.K, BN)) return cudaErrorInvalidValue;
  const long tiles = (long)tiles_m * ((g.N + BN - 1) / BN);
  const int grid = (int)(tiles < g_num_sms ? tiles : g_num_sms);
  gemm_bf16_kernel<BN><<<grid, kGemmThreads, GemmCfg<BN>::kSmemBytes, st>>>(tmA, tmB, p);
  return cudaGetLastError();
}

fv_status launch_gemm(const GemmArgs& g, cudaStream_t st) {
  if (g.M <= 0 || g.N <= 0 || g.K <= 0 || (g.K % 8) || (g.N % 8) || !g.a || !g.w) return FV_ERR_INVALID_ARG;
  if (g.rows_per_image <= 0) return FV_ERR_INVALID_ARG;
  if (g.epilogue == EPI_QKV_SPLIT && (g.C % 128 || g.q_cols % 128)) return FV_ERR_UNSUPPORTED;
  const int tiles_m = (g.M + BM - 1) / BM;
  const int bn = pick_bn(tiles_m, g.N, g_num_sms);
  GemmDev p;
  p.bias = static_cast<const __nv_bfloat16*>(g.bias);
  p.M = g.M; p.N = g.N; p.K = g.K; p.epilogue = g.epilogue; p.out = g.out; p.aux = g.aux; p.gamma = g.gamma;
  p.mod_stride = g.mod_stride; p.rows_per_image = g.rows_per_image; p.q_cols = g.q_cols; p.C = g.C;
  p.k_cache = static_cast<__nv_bfloat16*>(g.k_cache); p.vt_cache = static_cast<__nv_bfloat16*>(g.vt_cache);
  p.kv_capacity = g.kv_capacity; p.kv_offset = g.kv_offset; p.status = g.status;
  LaunchScope scope(KC_GEMM, 1, 2.0 * g.M * (double)g.N * g.K, st);
  cudaError_t e = bn == 256 ? launch_bn<256>(g, p, tiles_m, st) : (bn == 192 ? launch_bn<192>(g, p, tiles_m, st) : launch_bn<128>(g, p, tiles_m, st));
  return e == cudaSuccess ? FV_OK : FV_ERR_CUDA;
}

}  // namespace fv
