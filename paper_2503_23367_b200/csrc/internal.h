// Host-side launch functions shared between the translation units of libfastvar.
#pragma once
#include <cuda_runtime.h>
#include <stddef.h>
#include <stdint.h>

#include "../../include/fastvar.h"

namespace fv {

inline size_t align_up(size_t v, size_t a) { return (v + a - 1) / a * a; }

// Launch with programmatic stream serialization: the grid may start (and run up to its
// griddepcontrol.wait) while the kernel before it in the stream is still finishing, which hides launch
// latency and per-CTA set-up between the many short dependent kernels of a scale step.  Every kernel
// launched this way executes pdl_wait() before its first access to global memory that an earlier
// kernel may write or read.
#ifdef __CUDACC__
}  // namespace fv
#include <cuda_bf16.h>
namespace fv {
// Four / eight consecutive elements of the residual stream, fp32 or bf16, as floats.  NC: read-only path, else through L2.
template <bool NC> __device__ __forceinline__ float4 x_load4(const float* p) {
  return NC ? __ldg(reinterpret_cast<const float4*>(p)) : __ldcg(reinterpret_cast<const float4*>(p));
}
template <bool NC> __device__ __forceinline__ float4 x_load4(const __nv_bfloat16* p) {
  const uint2 u = NC ? __ldg(reinterpret_cast<const uint2*>(p)) : __ldcg(reinterpret_cast<const uint2*>(p));
  return make_float4(__uint_as_float(u.x << 16), __uint_as_float(u.x & 0xFFFF0000u), __uint_as_float(u.y << 16), __uint_as_float(u.y & 0xFFFF0000u));
}
__device__ __forceinline__ void x_load8(const float* p, float (&f)[8]) {
  const float4 a = reinterpret_cast<const float4*>(p)[0], b = reinterpret_cast<const float4*>(p)[1];
  f[0] = a.x; f[1] = a.y; f[2] = a.z; f[3] = a.w; f[4] = b.x; f[5] = b.y; f[6] = b.z; f[7] = b.w;
}
__device__ __forceinline__ void x_load8(const __nv_bfloat16* p, float (&f)[8]) {
  const uint4 v = *reinterpret_cast<const uint4*>(p);
  const uint32_t u[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
  for (int i = 0; i < 4; ++i) { f[2 * i] = __uint_as_float(u[i] << 16); f[2 * i + 1] = __uint_as_float(u[i] & 0xFFFF0000u); }
}
__device__ __forceinline__ void x_store8(float* p, const float (&f)[8]) {
  reinterpret_cast<float4*>(p)[0] = make_float4(f[0], f[1], f[2], f[3]);
  reinterpret_cast<float4*>(p)[1] = make_float4(f[4], f[5], f[6], f[7]);
}
// bf16 stream: the updated values are rounded to nearest even once, and those rounded values are what is stored,
// summed and scored from then on (f is overwritten with them).
__device__ __forceinline__ void x_store8(__nv_bfloat16* p, float (&f)[8]) {
  uint32_t u[4];
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    const __nv_bfloat162 v = __floats2bfloat162_rn(f[2 * i], f[2 * i + 1]);
    u[i] = *reinterpret_cast<const uint32_t*>(&v);
    f[2 * i] = __uint_as_float(u[i] << 16); f[2 * i + 1] = __uint_as_float(u[i] & 0xFFFF0000u);
  }
  *reinterpret_cast<uint4*>(p) = make_uint4(u[0], u[1], u[2], u[3]);
}
__device__ __forceinline__ void pdl_trigger() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }
__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
template <typename... KArgs, typename... Args>
inline cudaError_t launch_pdl(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t st, Args&&... args) {
  cudaLaunchConfig_t cfg{};
  cfg.gridDim = grid; cfg.blockDim = block; cfg.dynamicSmemBytes = smem; cfg.stream = st;
  cudaLaunchAttribute at[1];
  at[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  at[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = at; cfg.numAttrs = 1;
  return cudaLaunchKernelEx(&cfg, kernel, static_cast<KArgs>(args)...);
}
#endif

// ---- prof.cu : launch counting and optional per-kernel-class timing (CUDA events on the stream) ---
enum KernelClass : int { KC_SELECT = 0, KC_GATHER_LN = 1, KC_GEMM = 2, KC_ATTENTION = 3, KC_RESTORE = 4, KC_COUNT = 5 };
// Brackets the launches of one kernel class: counts `kernels` launches, adds `work` (algorithmic bytes
// for the HBM-bound classes, flops for GEMM / attention) and `dram_bytes` (the bytes the launch has to
// move to and from HBM once: its operands and results; checked against ncu's DRAM counters) and, when
// timing is enabled, records an event pair around them on `st`.
struct LaunchScope {
  LaunchScope(KernelClass c, int kernels, double work, double dram_bytes, cudaStream_t st);
  ~LaunchScope();
  int slot;
  cudaStream_t st;
};

// ---- select.cu : Pivotal Token Selection (Eq. 4-5, Algorithm 1) ---------------------------------
constexpr int kColsumRows = 32;        // token rows folded into one chunk partial of the column sums
constexpr int kMaxGroups = 16;         // chunk partials are folded again into at most this many group partials
constexpr int kTopkMaxTokens = 49152;  // scores of one image must fit the top-k CTA's shared memory
// Scratch of the selection, carved out of one caller buffer.  Column sums of the token map are kept at
// two levels: one partial per chunk of kColsumRows tokens, folded (by the last CTA of each group to
// finish) into <= kMaxGroups group partials per image, which the scoring kernel adds up itself.
struct SelectWs {
  unsigned int* tickets;  // [B, kMaxGroups] group arrival counters, [B] image counters, [B, 2] score range words; zero between launches
  float* chunk_partial;   // [B, nchunks, C]
  float* group_partial;   // [B, ngroups, C]
  float* score;           // [B, n]
  int nchunks, group, ngroups;
};
size_t select_workspace_bytes(int B, int n, int C);
size_t select_ticket_bytes(int B);  // leading bytes of the workspace that must be zero before first use
SelectWs select_ws_carve(void* workspace, int B, int n, int C);
// Scores [B,n] (fp32), then exact per-image top-k -> idx [B,k] ascending, inv [B,n].  have_partials:
// the group partials in the workspace already hold the column sums of x (left there by
// launch_restore_residual), so the column-sum pass is skipped.
// x_bf16 (select, gather, restore launchers): the residual stream is bf16 instead of fp32 (fv_config.resid_dtype).
cudaError_t launch_select(const void* x, int B, int n, int C, int k, int32_t* idx, int32_t* inv, float* score,
                          int32_t* near_tie, void* workspace, bool have_partials, cudaStream_t st, bool x_bf16 = false);
// The selection of a wrapped sublayer inside a scale step, in one launch with what surrounds it on the kept rows:
// the previous sublayer's kept-row restoration before it (y != null) and the gather + LayerNorm + modulation of the
// newly kept rows after it.  sel_ws holds the column sums of the rows the kernel does not update itself (left there
// by the restoration of the rows that were not kept, or by launch_colsum for a map nothing has restored yet).
struct FusedSelect {
  float* x; int B, n, C, k;
  const void* y; const int32_t* idx_prev; const float* gamma_prev; int mod_stride;   // y null: no kept rows to restore
  void* sel_ws; void* fused_ws;
  int32_t* idx; int32_t* inv;
  const float* sigma; const float* beta; void* a_out;
  int32_t* status;
  unsigned int* done_total; unsigned int* epoch;   // host counters of the context: what the kernel's waits compare against
};
size_t select_fused_ws_bytes(int B, int C);
size_t select_fused_sync_bytes(int B);            // leading bytes of fused_ws that must be zero before first use
bool select_fused_supported(int B, int n, int C);
cudaError_t launch_select_fused(const FusedSelect& f, cudaStream_t st);
cudaError_t launch_colsum(const float* x, int B, int n, int C, void* workspace, cudaStream_t st);   // column sums of a map -> sel_ws
cudaError_t launch_inv_from_idx(const int32_t* idx, int B, int k, int n, int32_t* inv, cudaStream_t st);
cudaError_t launch_inv_fill(int B, int n, int32_t* inv, cudaStream_t st);  // every token unkept (-1)
cudaError_t select_init();  // one-time function attributes

// ---- rows.cu : gather + LayerNorm + modulate, restore (+ gate and residual) ----------------------
// status (all gathers): device status word that receives DEV_BAD_ROW_INDEX when an index lies outside [0, n) (the
// index is clamped, so the read stays inside the map), or null.
cudaError_t launch_gather_ln(const void* x, const int32_t* idx, int B, int n, int k, int C, const float* sigma,
                             const float* beta, int mod_stride, void* a_out, int32_t* status, cudaStream_t st, bool x_bf16 = false);
// A wait nobody ends: one warp waits on an mbarrier without arrivals for limit_ns, then writes DEV_TIMEOUT_SELFTEST.
cudaError_t launch_expired_wait(int32_t* status, unsigned long long limit_ns, cudaStream_t st);
// colsum_ws: null, or the selection workspace that receives the column sums of the updated x.
// part: 0 = every row; 1 = the rows that were not kept; 2 = the kept rows (and the fold of the column sums);
// 3 = the rows that were not kept, their column sums folded (the kept rows are left to the next fused selection).
// interp_mode (all restore launchers): 0 nearest, 1 bilinear with half-pixel centres.
cudaError_t launch_restore_residual(void* x, const void* y, const void* cache, const int32_t* inv,
                                    const float* gamma, int mod_stride, int B, int k, int h, int w, int hc, int wc,
                                    int C, void* colsum_ws, int part, int interp_mode, cudaStream_t st, bool x_bf16 = false);
cudaError_t rows_init();               // one-time function attributes
void restore_force_fold(int mode);     // test hook: 0 by shape, 1 fold through global memory, 2 fold inside clusters
// Per-step granularity: fp32 gather of the kept rows, and fp32 restoration of the step's output map.
cudaError_t launch_gather_rows(const float* x, const int32_t* idx, int B, int n, int k, int C, float* out, int32_t* status, cudaStream_t st);
cudaError_t launch_restore_rows_f32(const float* cache, int hc, int wc, const float* pivots, const int32_t* inv, int B, int k,
                                    int h, int w, int C, float* out, int interp_mode, cudaStream_t st);
cudaError_t launch_restore_bf16(const void* cache, int hc, int wc, const void* pivots, const int32_t* inv, int B,
                                int k, int h, int w, int C, void* out, int interp_mode, cudaStream_t st);

// ---- gemm.cu : tcgen05 GEMM with fused epilogues -----------------------------------------------
enum GemmEpilogue : int { EPI_BF16 = 0, EPI_GELU_BF16 = 1, EPI_RESIDUAL = 2, EPI_QKV_SPLIT = 3, EPI_F32 = 4,
                          EPI_RESIDUAL_XBF16 = 5 /* as EPI_RESIDUAL with a bf16 residual stream: out bf16 [M,N] in place */ };
struct GemmArgs {
  const void* a;     // [M,K] bf16
  const void* w;     // [N,K] bf16
  const void* bias;  // [N] bf16 or null
  int M, N, K;
  int epilogue;
  void* out;           // EPI_BF16/GELU: bf16 [M,N]; EPI_RESIDUAL: fp32 [M,N] in place; EPI_F32: fp32 [M,N] written; EPI_QKV_SPLIT: Q bf16 [M,q_cols]
  void* aux;           // EPI_RESIDUAL: optional bf16 [M,N] copy of acc+bias
  const float* gamma;  // EPI_RESIDUAL: per-image gate or null
  int mod_stride;      // floats between images in gamma
  int rows_per_image;  // rows of A that belong to one image
  // EPI_QKV_SPLIT: columns [0,q_cols) -> out; [q_cols, q_cols+C) -> K rows; the rest -> V^T.
  int q_cols, C;
  void* k_cache;       // [B, kv_capacity, C] bf16
  void* vt_cache;      // [B, C, kv_capacity] bf16
  int kv_capacity, kv_offset;
  int32_t* status;     // device status word or null
  void* splitk_ws;     // scratch for K-split partials (gemm_splitk_ws_bytes(), tickets at its head zero) or null
  // EPI_QKV_SPLIT extras on the Q and K columns (all null = none):
  const float* qk_scale;      // [H] fp32: cosine attention (q, k divided by their per-head norm, q times this)
  const float* rope_table;    // [tokens of the scale][head_dim/2][2] fp32 (cos, sin) of the rotary angles
  const int32_t* rope_idx;    // [B, rows_per_image] original token of every row, or null (row j is token j)
  int head_dim;               // 64 or 128 (needed with either extra)
};
// (cos, sin) of the 2-D rotary angles of every token of an (h, w) map placed in the (h_last, w_last) frame:
// first head_dim/4 pairs turn with the row coordinate y * h_last / h, the rest with x * w_last / w, pair j of
// either group at frequency base^(-j / (head_dim/4)).  table: [h*w][head_dim/2][2] fp32.
cudaError_t launch_rope_table(float* table, int h, int w, int h_last, int w_last, int head_dim, float base, cudaStream_t st);
cudaError_t gemm_init();
// Test / profiling hook: 0 = choose per shape, 1 = one-CTA kernel, 2 = CTA-pair kernel 256x256, 3 = CTA-pair 256x128.
void gemm_force_path(int path);
size_t gemm_splitk_ws_bytes();      // size of the K-split scratch
size_t gemm_splitk_ticket_bytes();  // its leading bytes that must be zero before first use
fv_status launch_gemm(const GemmArgs& g, cudaStream_t st);

// ---- attention.cu : flash-style attention over the KV cache ------------------------------------
struct AttnArgs {
  const void* q;   // [B*rows, C] bf16
  const void* k;   // [B, kv_capacity, C] bf16
  const void* vt;  // [B, C, kv_capacity] bf16
  void* out;       // [B*rows, C] bf16
  int B, rows, H, C, kv_len, kv_capacity;
  int32_t* status;
  void* workspace;   // null (one work item per CTA), or attention_ws_bytes() of scratch whose leading attention_ws_ticket_bytes() are zero
};
cudaError_t attention_init();
size_t attention_ws_bytes();
size_t attention_ws_ticket_bytes();
void attention_force_ctas(int ctas);   // test hook: CTAs of a split launch (0 = one per SM)
fv_status launch_attention(const AttnArgs& a, cudaStream_t st);

// ---- tensor maps (gemm.cu) ------------------------------------------------------------------------
// 2-D bf16 row-major tensor [rows, cols] -> TMA descriptor with a (box_rows x 64) box and 128-byte swizzle.
bool make_tmap_bf16_2d(void* tmap_out, const void* base, uint64_t rows, uint64_t cols, uint32_t box_rows);

// generate.cu reads the step sizes of a context (api.cu owns the context's layout)
}  // namespace fv
struct fv_ctx;
namespace fv {
const fv_config* ctx_config(const fv_ctx* ctx);
int32_t* ctx_status_word(const fv_ctx* ctx);   // the device status word in the context's workspace
}  // namespace fv
