// C ABI of libfastvar: argument checking, the context (host metadata only), and the per-step
// orchestration of the pruned scale step (Sec. 3.3 "Overview" / "Implementation", Fig. 3).
#include <cuda_runtime.h>

#include <cmath>
#include <cstring>
#include <mutex>
#include <new>
#include <vector>

#include "internal.h"

using namespace fv;

struct fv_ctx {
  fv_config cfg;
  std::vector<int32_t> h, w;
  // borrowed device pointers, per block
  std::vector<const void*> w_qkv, b_qkv, w_o, b_o, w_fc1, b_fc1, w_fc2, b_fc2, w_q_x, w_kv_x, w_o_x;
  const float* mod = nullptr;
  const void* text = nullptr;
  char* kv = nullptr;
  char* cache = nullptr;
  char* ws = nullptr;
  int n_sub = 2, n_cache = 0, n_max = 0;
  int next_step = 0, kv_len = 0;
  bool text_ready = false;
  // workspace carve-up
  int32_t* status = nullptr;
  char *a_buf = nullptr, *q_buf = nullptr, *o_buf = nullptr, *y_buf = nullptr, *h_buf = nullptr;
  int32_t *idx = nullptr, *inv = nullptr;
  int32_t *idx2 = nullptr, *inv2 = nullptr;   // second set: the fused selection reads the previous sublayer's indices while it writes the next
  void* sel_ws = nullptr;
  void* fsel_ws = nullptr;                    // scratch of the fused selection (arrival counts, kept-row partial sums)
  unsigned int fsel_done = 0, fsel_epoch = 0; // what its grid-wide waits compare against (grow with every launch)
  void* splitk_ws = nullptr;
  void* attn_ws = nullptr;
  cudaStream_t side = nullptr;           // the unkept rows of a restoration run here, beside the sublayer's branch
  cudaEvent_t ev_fork = nullptr, ev_join = nullptr;
  float* step_cache = nullptr;  // fp32 output map of the caching step [B_max, n_cache, C] (skipped steps; granularity 1)
  float* xc = nullptr;  // granularity 1: compact fp32 residual stream of a pruned step [B*k, C]
  // fv_var_step_host: copy streams and the events that order two staging buffers per direction
  cudaStream_t io_in = nullptr, io_out = nullptr;
  cudaEvent_t ev_in[2] = {nullptr, nullptr}, ev_used[2] = {nullptr, nullptr}, ev_out[2] = {nullptr, nullptr}, ev_copied[2] = {nullptr, nullptr};
  bool used_rec[2] = {false, false}, copied_rec[2] = {false, false};
  unsigned io_count = 0;
  const float* qk_scale = nullptr;      // [L, H] or null
  std::vector<float*> rope_tab;         // per scale step: (cos, sin) table [h*w][hd/2][2], empty = no rotary positions
  size_t kv_block_bytes = 0, k_bytes = 0, text_k_bytes = 0, text_block_bytes = 0, cache_sub_bytes = 0;
};

namespace fv {
const fv_config* ctx_config(const fv_ctx* ctx) { return &ctx->cfg; }
int32_t* ctx_status_word(const fv_ctx* ctx) { return ctx->status; }
}  // namespace fv

namespace {

// Test / profiling hook.  true: a free-running selection is one launch that also restores the previous sublayer's kept
// rows and gathers the new ones (select_fused_kernel).  Measured on B200 it does not pay: with programmatic dependent
// launch the separate kernels already overlap their launch gaps, while the fused kernel runs one CTA per SM and waits
// twice grid-wide (pruned steps of the 1024-pixel workload 3 % slower, of the 2K workload equal), so it is off.
bool g_step_fused = false;

std::once_flag g_init_once;
cudaError_t g_init_err = cudaSuccess;

cudaError_t ensure_init() {
  std::call_once(g_init_once, [] {
    g_init_err = select_init();
    if (g_init_err == cudaSuccess) g_init_err = rows_init();
    if (g_init_err == cudaSuccess) g_init_err = gemm_init();
    if (g_init_err == cudaSuccess) g_init_err = attention_init();
  });
  return g_init_err;
}

bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

struct Layout {
  size_t status, a, q, o, y, hbuf, idx, inv, idx2, inv2, sel, fsel, splitk, attn, xc, rope, total;
};

int max_tokens(const fv_config* c) {
  int n = 0;
  for (int i = 0; i < c->n_steps; ++i) n = std::max(n, c->h[i] * c->w[i]);
  return n;
}

bool config_ok(const fv_config* c) {
  if (!c || c->L <= 0 || c->C <= 0 || c->H <= 0 || c->mlp_ratio <= 0 || c->B_max <= 0 || c->n_steps <= 0) return false;
  if (!c->h || !c->w || c->cross_len < 0 || c->kv_capacity <= 0) return false;
  for (int i = 0; i < c->n_steps; ++i)
    if (c->h[i] <= 0 || c->w[i] <= 0) return false;
  if (c->cache_step >= c->n_steps) return false;
  if (c->granularity != 0 && c->granularity != 1) return false;
  if (c->interp_mode < 0 || c->interp_mode > 2) return false;
  if (c->resid_dtype != 0 && c->resid_dtype != 1) return false;
  if (!(c->rope_base >= 0.f)) return false;
  return true;
}

Layout workspace_layout(const fv_config* c) {
  Layout l;
  const size_t M = (size_t)c->B_max * max_tokens(c);
  const size_t C = c->C, F = (size_t)c->C * c->mlp_ratio;
  size_t off = 0;
  auto take = [&](size_t bytes) { size_t o = off; off += align_up(bytes, 1024); return o; };
  l.status = take(256);
  l.a = take(M * C * 2);
  l.q = take(M * C * 2);
  l.o = take(M * C * 2);
  l.y = take(M * C * 2);
  l.hbuf = take(M * F * 2);
  l.idx = take(M * 4);
  l.inv = take(M * 4);
  l.idx2 = take(M * 4);
  l.inv2 = take(M * 4);
  l.sel = take(select_workspace_bytes(c->B_max, max_tokens(c), c->C));
  l.fsel = take(select_fused_ws_bytes(c->B_max, c->C));
  l.splitk = take(gemm_splitk_ws_bytes());
  l.attn = take(attention_ws_bytes());
  l.xc = take(c->granularity == 1 ? M * C * 4 : 0);
  size_t rope_bytes = 0;
  if (c->rope_base > 0.f)
    for (int i = 0; i < c->n_steps; ++i) rope_bytes += align_up((size_t)c->h[i] * c->w[i] * (c->C / c->H / 2) * 8, 1024);
  l.rope = take(rope_bytes);
  l.total = off;
  return l;
}

fv_status cuda_status(cudaError_t e) { return e == cudaSuccess ? FV_OK : FV_ERR_CUDA; }

}  // namespace

extern "C" {

const char* fv_status_string(fv_status s) {
  switch (s) {
    case FV_OK: return "ok";
    case FV_ERR_INVALID_ARG: return "invalid argument";
    case FV_ERR_BAD_STATE: return "bad state";
    case FV_ERR_CAPACITY: return "capacity exceeded";
    case FV_ERR_UNSUPPORTED: return "unsupported shape";
    case FV_ERR_CUDA: return "CUDA error";
    case FV_ERR_TIMEOUT: return "device-side wait expired";
    case FV_ERR_DEVICE_DATA: return "a kernel met an index outside its range";
  }
  return "unknown";
}

int32_t fv_k_for(double keep_ratio, int32_t h, int32_t w) {
  const long n = (long)h * w;
  long k = (long)std::ceil(keep_ratio * (double)n - 1e-9);
  if (k < 1) k = 1;
  if (k > n) k = n;
  return (int32_t)k;
}

size_t fv_prune_select_workspace_bytes(int32_t B, int32_t n_tokens, int32_t C) {
  if (B <= 0 || n_tokens <= 0 || C <= 0) return 0;
  return select_workspace_bytes(B, n_tokens, C);
}

fv_status fv_prune_select(const float* x_dev, int32_t B, int32_t h, int32_t w, int32_t C, double keep_ratio,
                          int32_t* idx_out_dev, int32_t* inv_out_dev, float* score_out_dev, int32_t* near_tie_dev,
                          int32_t* k_out_host, void* workspace_dev, size_t workspace_bytes, void* stream) {
  if (!x_dev || !idx_out_dev || !workspace_dev || B <= 0 || h <= 0 || w <= 0 || C <= 0) return FV_ERR_INVALID_ARG;
  if (!(keep_ratio > 0.0) || keep_ratio > 1.0 || (C % 4) || !aligned16(x_dev) || !aligned16(workspace_dev)) return FV_ERR_INVALID_ARG;
  const long n = (long)h * w;
  if (n > kTopkMaxTokens || C > kTopkMaxTokens) return FV_ERR_UNSUPPORTED;
  if (workspace_bytes < select_workspace_bytes(B, (int)n, C)) return FV_ERR_CAPACITY;
  if (ensure_init() != cudaSuccess) return FV_ERR_CUDA;
  const int k = fv_k_for(keep_ratio, h, w);
  if (k_out_host) *k_out_host = k;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  // the arrival counters at the head of the workspace must start at zero
  if (cudaMemsetAsync(workspace_dev, 0, select_ticket_bytes(B), st) != cudaSuccess) return FV_ERR_CUDA;
  return cuda_status(launch_select(x_dev, B, (int)n, C, k, idx_out_dev, inv_out_dev, score_out_dev, near_tie_dev,
                                   workspace_dev, false, st));
}

fv_status fv_restore(const void* cache_prev_dev, int32_t hc, int32_t wc, const void* pivots_dev, const int32_t* idx_dev,
                     int32_t B, int32_t k, int32_t h, int32_t w, int32_t C, void* out_dev, int32_t* inv_scratch_dev,
                     int32_t interp_mode, void* stream) {
  if (!cache_prev_dev || !pivots_dev || !idx_dev || !out_dev || !inv_scratch_dev) return FV_ERR_INVALID_ARG;
  if (interp_mode < 0 || interp_mode > 2) return FV_ERR_INVALID_ARG;
  if (B <= 0 || k <= 0 || h <= 0 || w <= 0 || hc <= 0 || wc <= 0 || C <= 0 || (C % 8) || k > h * w) return FV_ERR_INVALID_ARG;
  if (!aligned16(cache_prev_dev) || !aligned16(pivots_dev) || !aligned16(out_dev)) return FV_ERR_INVALID_ARG;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  cudaError_t e = launch_inv_from_idx(idx_dev, B, k, h * w, inv_scratch_dev, st);
  if (e != cudaSuccess) return FV_ERR_CUDA;
  return cuda_status(launch_restore_bf16(cache_prev_dev, hc, wc, pivots_dev, inv_scratch_dev, B, k, h, w, C, out_dev, interp_mode, st));
}

fv_status fv_gather_ln(const float* x_dev, const int32_t* idx_dev, int32_t B, int32_t n_tokens, int32_t k, int32_t C,
                       const float* sigma_dev, const float* beta_dev, int32_t mod_stride, void* a_out_dev, int32_t* status_dev,
                       void* stream) {
  if (!x_dev || !a_out_dev || B <= 0 || n_tokens <= 0 || k <= 0 || k > n_tokens || C <= 0 || (C % 4)) return FV_ERR_INVALID_ARG;
  if ((sigma_dev == nullptr) != (beta_dev == nullptr)) return FV_ERR_INVALID_ARG;
  if (C > 2048) return FV_ERR_UNSUPPORTED;
  if (!idx_dev && k != n_tokens) return FV_ERR_INVALID_ARG;
  return cuda_status(launch_gather_ln(x_dev, idx_dev, B, n_tokens, k, C, sigma_dev, beta_dev, mod_stride, a_out_dev, status_dev,
                                      static_cast<cudaStream_t>(stream)));
}

fv_status fv_restore_residual(float* x_dev, const void* y_dev, const void* cache_dev, const int32_t* inv_dev,
                              const float* gamma_dev, int32_t mod_stride, int32_t B, int32_t k, int32_t h, int32_t w,
                              int32_t hc, int32_t wc, int32_t C, int32_t interp_mode, void* colsum_ws_dev, size_t colsum_ws_bytes,
                              int32_t part, void* stream) {
  if (interp_mode < 0 || interp_mode > 2 || part < 0 || part > 2) return FV_ERR_INVALID_ARG;
  if (!x_dev || !y_dev || !cache_dev || !inv_dev || B <= 0 || k <= 0 || h <= 0 || w <= 0 || hc <= 0 || wc <= 0) return FV_ERR_INVALID_ARG;
  if (C <= 0 || (C % 8)) return FV_ERR_INVALID_ARG;
  if (ensure_init() != cudaSuccess) return FV_ERR_CUDA;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  if (colsum_ws_dev) {
    if (!aligned16(colsum_ws_dev)) return FV_ERR_INVALID_ARG;
    if ((long)h * w > kTopkMaxTokens) return FV_ERR_UNSUPPORTED;
    if (colsum_ws_bytes < select_workspace_bytes(B, h * w, C)) return FV_ERR_CAPACITY;
    // the arrival counters at the head of the workspace start at zero (the kernels leave them at zero)
    if (part != 2 && cudaMemsetAsync(colsum_ws_dev, 0, select_ticket_bytes(B), st) != cudaSuccess) return FV_ERR_CUDA;
  }
  return cuda_status(launch_restore_residual(x_dev, y_dev, cache_dev, inv_dev, gamma_dev, mod_stride, B, k, h, w, hc, wc, C,
                                             colsum_ws_dev, part, interp_mode, st));
}

fv_status fv_prune_select_after_restore(const float* x_dev, int32_t B, int32_t h, int32_t w, int32_t C, double keep_ratio,
                                        int32_t* idx_out_dev, int32_t* inv_out_dev, float* score_out_dev, int32_t* near_tie_dev,
                                        int32_t* k_out_host, void* workspace_dev, size_t workspace_bytes, void* stream) {
  if (!x_dev || !idx_out_dev || !workspace_dev || B <= 0 || h <= 0 || w <= 0 || C <= 0) return FV_ERR_INVALID_ARG;
  if (!(keep_ratio > 0.0) || keep_ratio > 1.0 || (C % 4) || !aligned16(x_dev) || !aligned16(workspace_dev)) return FV_ERR_INVALID_ARG;
  const long n = (long)h * w;
  if (n > kTopkMaxTokens || C > kTopkMaxTokens) return FV_ERR_UNSUPPORTED;
  if (workspace_bytes < select_workspace_bytes(B, (int)n, C)) return FV_ERR_CAPACITY;
  if (ensure_init() != cudaSuccess) return FV_ERR_CUDA;
  const int k = fv_k_for(keep_ratio, h, w);
  if (k_out_host) *k_out_host = k;
  return cuda_status(launch_select(x_dev, B, (int)n, C, k, idx_out_dev, inv_out_dev, score_out_dev, near_tie_dev, workspace_dev, true,
                                   static_cast<cudaStream_t>(stream)));
}

fv_status fv_prune_select_workspace_layout(int32_t B, int32_t n_tokens, int32_t C, size_t* offset_host, int32_t* n_partials_host) {
  if (B <= 0 || n_tokens <= 0 || C <= 0 || !offset_host || !n_partials_host) return FV_ERR_INVALID_ARG;
  static char origin[1];     // carve relative to any address; only the offset is reported
  const SelectWs w = select_ws_carve(origin, B, n_tokens, C);
  *offset_host = (size_t)(reinterpret_cast<char*>(w.group_partial) - origin);
  *n_partials_host = w.ngroups;
  return FV_OK;
}

fv_status fv_step_fused_selection(int32_t on) {
  g_step_fused = on != 0;
  return FV_OK;
}

fv_status fv_restore_force_fold(int32_t mode) {
  if (mode < 0 || mode > 2) return FV_ERR_INVALID_ARG;
  restore_force_fold(mode);
  return FV_OK;
}

fv_status fv_gemm_bf16(const void* a_dev, const void* w_dev, const void* bias_dev, int32_t M, int32_t N, int32_t K,
                       int32_t epilogue, void* out_dev, void* aux_dev, const float* gamma_dev, int32_t mod_stride,
                       int32_t rows_per_image, int32_t* status_dev, void* splitk_ws_dev, size_t splitk_ws_bytes, void* stream) {
  if (!a_dev || !w_dev || !out_dev || epilogue < 0 || epilogue > 5 || epilogue == EPI_QKV_SPLIT) return FV_ERR_INVALID_ARG;
  if (splitk_ws_dev && (splitk_ws_bytes < gemm_splitk_ws_bytes() || !aligned16(splitk_ws_dev))) return FV_ERR_CAPACITY;
  if (!aligned16(a_dev) || !aligned16(w_dev) || !aligned16(out_dev) || (bias_dev && !aligned16(bias_dev))) return FV_ERR_INVALID_ARG;
  if (ensure_init() != cudaSuccess) return FV_ERR_CUDA;
  GemmArgs g{};
  g.a = a_dev; g.w = w_dev; g.bias = bias_dev; g.M = M; g.N = N; g.K = K; g.epilogue = epilogue; g.out = out_dev;
  g.aux = aux_dev; g.gamma = gamma_dev; g.mod_stride = mod_stride; g.rows_per_image = rows_per_image > 0 ? rows_per_image : M;
  g.status = status_dev;
  g.splitk_ws = splitk_ws_dev;
  return launch_gemm(g, static_cast<cudaStream_t>(stream));
}

size_t fv_attention_workspace_bytes(void) { return attention_ws_bytes(); }

fv_status fv_attention_force_ctas(int32_t ctas) {
  if (ctas < -1) return FV_ERR_INVALID_ARG;
  attention_force_ctas(ctas);
  return FV_OK;
}

fv_status fv_attention(const void* q_dev, const void* k_dev, const void* vt_dev, int32_t B, int32_t rows, int32_t H,
                       int32_t C, int32_t kv_len, int32_t kv_capacity, void* out_dev, int32_t* status_dev, void* workspace_dev,
                       size_t workspace_bytes, void* stream) {
  if (ensure_init() != cudaSuccess) return FV_ERR_CUDA;
  if (!aligned16(q_dev) || !aligned16(k_dev) || !aligned16(vt_dev) || !aligned16(out_dev)) return FV_ERR_INVALID_ARG;
  if (workspace_dev && (!aligned16(workspace_dev) || workspace_bytes < attention_ws_bytes())) return FV_ERR_CAPACITY;
  AttnArgs a{};
  a.workspace = workspace_dev;
  a.q = q_dev; a.k = k_dev; a.vt = vt_dev; a.out = out_dev; a.B = B; a.rows = rows; a.H = H; a.C = C; a.kv_len = kv_len;
  a.kv_capacity = kv_capacity; a.status = status_dev;
  return launch_attention(a, static_cast<cudaStream_t>(stream));
}

// ------------------------------------------------------------------------------------------------ context

size_t fv_gemm_splitk_workspace_bytes(void) { return gemm_splitk_ws_bytes(); }

fv_status fv_gemm_force_path(int32_t path) {
  if (path < 0 || path > 11) return FV_ERR_INVALID_ARG;
  gemm_force_path(path);
  return FV_OK;
}

size_t fv_workspace_bytes(const fv_config* cfg) { return config_ok(cfg) ? workspace_layout(cfg).total : 0; }

size_t fv_kv_bytes(const fv_config* cfg) {
  if (!config_ok(cfg)) return 0;
  const size_t per_block = 2 * align_up((size_t)cfg->B_max * cfg->kv_capacity * cfg->C * 2, 1024);
  const size_t text_block = 2 * align_up((size_t)cfg->B_max * cfg->cross_len * cfg->C * 2, 1024);
  return (size_t)cfg->L * (per_block + text_block);
}

size_t fv_cache_bytes(const fv_config* cfg) {
  if (!config_ok(cfg) || cfg->cache_step < 0) return 0;
  const size_t n_cache = (size_t)cfg->h[cfg->cache_step] * cfg->w[cfg->cache_step];
  // the fp32 output map of the caching step comes first (restored by skipped steps and by granularity 1) ...
  const size_t step_bytes = align_up((size_t)cfg->B_max * n_cache * cfg->C * 4, 1024);
  if (cfg->granularity == 1) return step_bytes;
  // ... then, for the paper's granularity, one bf16 cache per wrapped sublayer
  const int n_sub = cfg->cross_len ? 3 : 2;
  return step_bytes + (size_t)cfg->L * n_sub * align_up((size_t)cfg->B_max * n_cache * cfg->C * 2, 1024);
}

fv_status fv_create(const fv_config* cfg, const fv_weights* wts, void* kv_dev, void* cache_dev, void* workspace_dev,
                    fv_ctx** out) {
  if (!out) return FV_ERR_INVALID_ARG;
  *out = nullptr;
  if (!config_ok(cfg) || !wts || !kv_dev || !workspace_dev) return FV_ERR_INVALID_ARG;
  if (cfg->cache_step >= 0 && !cache_dev) return FV_ERR_INVALID_ARG;
  if ((reinterpret_cast<uintptr_t>(kv_dev) | reinterpret_cast<uintptr_t>(workspace_dev) | reinterpret_cast<uintptr_t>(cache_dev)) & 1023u)
    return FV_ERR_INVALID_ARG;
  if (cfg->C % cfg->H || cfg->kv_capacity % 8 || cfg->cross_len % 8) return FV_ERR_INVALID_ARG;
  const int hd = cfg->C / cfg->H;
  if ((hd != 64 && hd != 128) || cfg->C > 2048 || cfg->C % 128) return FV_ERR_UNSUPPORTED;
  if (max_tokens(cfg) > kTopkMaxTokens) return FV_ERR_UNSUPPORTED;
  if (cfg->resid_dtype == 1 && (cfg->granularity != 0 || cfg->interp_mode != 0)) return FV_ERR_UNSUPPORTED;
  if (!wts->w_qkv || !wts->b_qkv || !wts->w_o || !wts->b_o || !wts->w_fc1 || !wts->b_fc1 || !wts->w_fc2 || !wts->b_fc2 || !wts->mod_dev)
    return FV_ERR_INVALID_ARG;
  if (cfg->cross_len && (!wts->w_q_x || !wts->w_kv_x || !wts->w_o_x || !wts->text_dev)) return FV_ERR_INVALID_ARG;
  if (ensure_init() != cudaSuccess) return FV_ERR_CUDA;

  fv_ctx* c = new (std::nothrow) fv_ctx();
  if (!c) return FV_ERR_INVALID_ARG;
  c->cfg = *cfg;
  c->h.assign(cfg->h, cfg->h + cfg->n_steps);
  c->w.assign(cfg->w, cfg->w + cfg->n_steps);
  c->cfg.h = c->h.data();
  c->cfg.w = c->w.data();
  auto copy = [&](std::vector<const void*>& dst, const void* const* src) { if (src) dst.assign(src, src + cfg->L); };
  copy(c->w_qkv, wts->w_qkv); copy(c->b_qkv, wts->b_qkv); copy(c->w_o, wts->w_o); copy(c->b_o, wts->b_o);
  copy(c->w_fc1, wts->w_fc1); copy(c->b_fc1, wts->b_fc1); copy(c->w_fc2, wts->w_fc2); copy(c->b_fc2, wts->b_fc2);
  if (cfg->cross_len) { copy(c->w_q_x, wts->w_q_x); copy(c->w_kv_x, wts->w_kv_x); copy(c->w_o_x, wts->w_o_x); }
  for (int l = 0; l < cfg->L; ++l) {
    const void* must[] = {c->w_qkv[l], c->b_qkv[l], c->w_o[l], c->b_o[l], c->w_fc1[l], c->b_fc1[l], c->w_fc2[l], c->b_fc2[l]};
    for (const void* p : must)
      if (!p || !aligned16(p)) { delete c; return FV_ERR_INVALID_ARG; }
    if (cfg->cross_len && (!c->w_q_x[l] || !c->w_kv_x[l] || !c->w_o_x[l])) { delete c; return FV_ERR_INVALID_ARG; }
  }
  c->mod = wts->mod_dev;
  c->text = wts->text_dev;
  c->kv = static_cast<char*>(kv_dev);
  c->step_cache = static_cast<float*>(cache_dev);
  c->cache = (cache_dev && cfg->cache_step >= 0) ? static_cast<char*>(cache_dev) +
                             align_up((size_t)cfg->B_max * cfg->h[cfg->cache_step] * cfg->w[cfg->cache_step] * cfg->C * 4, 1024)
                       : nullptr;
  c->ws = static_cast<char*>(workspace_dev);
  c->n_sub = cfg->cross_len ? 3 : 2;
  c->n_max = max_tokens(cfg);
  c->n_cache = cfg->cache_step >= 0 ? cfg->h[cfg->cache_step] * cfg->w[cfg->cache_step] : 0;
  c->k_bytes = align_up((size_t)cfg->B_max * cfg->kv_capacity * cfg->C * 2, 1024);
  c->kv_block_bytes = 2 * c->k_bytes;
  c->text_k_bytes = align_up((size_t)cfg->B_max * cfg->cross_len * cfg->C * 2, 1024);
  c->text_block_bytes = 2 * c->text_k_bytes;
  c->cache_sub_bytes = align_up((size_t)cfg->B_max * c->n_cache * cfg->C * 2, 1024);
  const Layout lay = workspace_layout(cfg);
  c->status = reinterpret_cast<int32_t*>(c->ws + lay.status);
  c->a_buf = c->ws + lay.a; c->q_buf = c->ws + lay.q; c->o_buf = c->ws + lay.o; c->y_buf = c->ws + lay.y;
  c->h_buf = c->ws + lay.hbuf;
  c->idx = reinterpret_cast<int32_t*>(c->ws + lay.idx);
  c->inv = reinterpret_cast<int32_t*>(c->ws + lay.inv);
  c->idx2 = reinterpret_cast<int32_t*>(c->ws + lay.idx2);
  c->inv2 = reinterpret_cast<int32_t*>(c->ws + lay.inv2);
  c->sel_ws = c->ws + lay.sel;
  c->fsel_ws = c->ws + lay.fsel;
  c->splitk_ws = c->ws + lay.splitk;
  c->attn_ws = c->ws + lay.attn;
  c->xc = reinterpret_cast<float*>(c->ws + lay.xc);
  c->qk_scale = wts->qk_scale_dev;
  bool rope_ok = true;
  if (cfg->rope_base > 0.f) {
    char* t = c->ws + lay.rope;
    for (int i = 0; i < cfg->n_steps; ++i) {
      c->rope_tab.push_back(reinterpret_cast<float*>(t));
      rope_ok = rope_ok && launch_rope_table(c->rope_tab.back(), cfg->h[i], cfg->w[i], cfg->h[cfg->n_steps - 1], cfg->w[cfg->n_steps - 1], hd,
                                             cfg->rope_base, nullptr) == cudaSuccess;
      t += align_up((size_t)cfg->h[i] * cfg->w[i] * (hd / 2) * 8, 1024);
    }
  }
  // Never-written KV rows must read as zeros (they meet zero probabilities in P*V).
  if (!rope_ok || cudaMemset(kv_dev, 0, fv_kv_bytes(cfg)) != cudaSuccess || cudaMemset(c->status, 0, 256) != cudaSuccess ||
      cudaMemset(c->sel_ws, 0, select_ticket_bytes(cfg->B_max)) != cudaSuccess ||
      cudaMemset(c->fsel_ws, 0, select_fused_sync_bytes(cfg->B_max)) != cudaSuccess ||
      cudaMemset(c->splitk_ws, 0, gemm_splitk_ticket_bytes()) != cudaSuccess ||
      cudaMemset(c->attn_ws, 0, attention_ws_ticket_bytes()) != cudaSuccess ||
      cudaStreamCreateWithFlags(&c->side, cudaStreamNonBlocking) != cudaSuccess ||
      cudaEventCreateWithFlags(&c->ev_fork, cudaEventDisableTiming) != cudaSuccess ||
      cudaEventCreateWithFlags(&c->ev_join, cudaEventDisableTiming) != cudaSuccess ||
      cudaDeviceSynchronize() != cudaSuccess) {
    fv_destroy(c);
    return FV_ERR_CUDA;
  }
  *out = c;
  return FV_OK;
}

void fv_destroy(fv_ctx* ctx) {
  if (!ctx) return;
  if (ctx->side) { cudaStreamSynchronize(ctx->side); cudaStreamDestroy(ctx->side); }
  if (ctx->ev_fork) cudaEventDestroy(ctx->ev_fork);
  if (ctx->ev_join) cudaEventDestroy(ctx->ev_join);
  if (ctx->io_in) { cudaStreamSynchronize(ctx->io_in); cudaStreamDestroy(ctx->io_in); }
  if (ctx->io_out) { cudaStreamSynchronize(ctx->io_out); cudaStreamDestroy(ctx->io_out); }
  for (int i = 0; i < 2; ++i)
    for (cudaEvent_t e : {ctx->ev_in[i], ctx->ev_used[i], ctx->ev_out[i], ctx->ev_copied[i]})
      if (e) cudaEventDestroy(e);
  delete ctx;
}

fv_status fv_reset(fv_ctx* ctx) {
  if (!ctx) return FV_ERR_INVALID_ARG;
  ctx->next_step = 0;
  ctx->kv_len = 0;
  return FV_OK;
}

fv_status fv_get_state(const fv_ctx* ctx, int32_t* next_step_host, int32_t* kv_len_host) {
  if (!ctx) return FV_ERR_INVALID_ARG;
  if (next_step_host) *next_step_host = ctx->next_step;
  if (kv_len_host) *kv_len_host = ctx->kv_len;
  return FV_OK;
}

fv_status fv_set_state(fv_ctx* ctx, int32_t next_step, int32_t kv_len) {
  if (!ctx || next_step < 0 || next_step > ctx->cfg.n_steps || kv_len < 0 || kv_len > ctx->cfg.kv_capacity) return FV_ERR_INVALID_ARG;
  ctx->next_step = next_step;
  ctx->kv_len = kv_len;
  return FV_OK;
}

fv_status fv_kv_pointers(const fv_ctx* ctx, int32_t block, void** k_dev, void** vt_dev) {
  if (!ctx || block < 0 || block >= ctx->cfg.L) return FV_ERR_INVALID_ARG;
  char* base = ctx->kv + (size_t)block * ctx->kv_block_bytes;
  if (k_dev) *k_dev = base;
  if (vt_dev) *vt_dev = base + ctx->k_bytes;
  return FV_OK;
}

fv_status fv_cache_pointer(const fv_ctx* ctx, int32_t block, int32_t sublayer, void** cache_dev) {
  if (!ctx || !cache_dev || block < 0 || block >= ctx->cfg.L || sublayer < 0 || sublayer >= ctx->n_sub || !ctx->cache) return FV_ERR_INVALID_ARG;
  if (ctx->cfg.granularity == 1) {  // one step-level cache
    if (block != 0 || sublayer != 0) return FV_ERR_INVALID_ARG;
    *cache_dev = ctx->step_cache;
    return FV_OK;
  }
  *cache_dev = ctx->cache + ((size_t)block * ctx->n_sub + sublayer) * ctx->cache_sub_bytes;
  return FV_OK;
}

static char* text_k(const fv_ctx* c, int l) { return c->kv + (size_t)c->cfg.L * c->kv_block_bytes + (size_t)l * c->text_block_bytes; }

fv_status fv_prepare_text(fv_ctx* ctx, int32_t B, void* stream) {
  if (!ctx || B <= 0 || B > ctx->cfg.B_max) return FV_ERR_INVALID_ARG;
  if (!ctx->cfg.cross_len) return FV_OK;
  const fv_config& c = ctx->cfg;
  for (int l = 0; l < c.L; ++l) {
    GemmArgs g{};
    g.a = ctx->text; g.w = ctx->w_kv_x[l]; g.bias = nullptr; g.M = B * c.cross_len; g.N = 2 * c.C; g.K = c.C;
    g.epilogue = EPI_QKV_SPLIT; g.out = nullptr; g.q_cols = 0; g.C = c.C; g.rows_per_image = c.cross_len;
    g.k_cache = text_k(ctx, l); g.vt_cache = text_k(ctx, l) + ctx->text_k_bytes; g.kv_capacity = c.cross_len; g.kv_offset = 0;
    g.status = ctx->status; g.splitk_ws = ctx->splitk_ws;
    fv_status s = launch_gemm(g, static_cast<cudaStream_t>(stream));
    if (s != FV_OK) return s;
  }
  ctx->text_ready = true;
  return FV_OK;
}

fv_status fv_device_status(fv_ctx* ctx, int32_t* code_host, void* stream) {
  if (!ctx) return FV_ERR_INVALID_ARG;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  int32_t code = 0;
  if (cudaMemcpyAsync(&code, ctx->status, 4, cudaMemcpyDeviceToHost, st) != cudaSuccess) return FV_ERR_CUDA;
  if (cudaStreamSynchronize(st) != cudaSuccess) return FV_ERR_CUDA;
  if (code_host) *code_host = code;
  if (code != 0) {
    cudaMemsetAsync(ctx->status, 0, 4, st);
    // a kernel that gave up may have left arrival counts half-way: every counter starts afresh
    cudaMemsetAsync(ctx->sel_ws, 0, select_ticket_bytes(ctx->cfg.B_max), st);
    cudaMemsetAsync(ctx->fsel_ws, 0, select_fused_sync_bytes(ctx->cfg.B_max), st);
    cudaMemsetAsync(ctx->splitk_ws, 0, gemm_splitk_ticket_bytes(), st);
    cudaMemsetAsync(ctx->attn_ws, 0, attention_ws_ticket_bytes(), st);
    ctx->fsel_done = 0; ctx->fsel_epoch = 0;
    cudaStreamSynchronize(st);
    return code >= 100 ? FV_ERR_TIMEOUT : FV_ERR_DEVICE_DATA;
  }
  return FV_OK;
}

fv_status fv_selftest_expired_wait(fv_ctx* ctx, uint64_t limit_ns, void* stream) {
  if (!ctx || limit_ns == 0 || limit_ns > 1000000000ull) return FV_ERR_INVALID_ARG;
  return cuda_status(launch_expired_wait(ctx->status, limit_ns, static_cast<cudaStream_t>(stream)));
}

fv_status fv_var_step(fv_ctx* ctx, const void* tokens_dev, int32_t B, int32_t scale_idx, double keep_ratio, void* out_dev,
                      const int32_t* forced_idx_dev, int32_t* idx_trace_dev, void* stream) {
  if (!ctx || !tokens_dev || !out_dev || B <= 0 || B > ctx->cfg.B_max) return FV_ERR_INVALID_ARG;
  if (!(keep_ratio >= 0.0) || keep_ratio > 1.0 || !aligned16(tokens_dev) || !aligned16(out_dev)) return FV_ERR_INVALID_ARG;
  const fv_config& c = ctx->cfg;
  if (scale_idx < 0 || scale_idx >= c.n_steps) return FV_ERR_INVALID_ARG;
  if (scale_idx != ctx->next_step) return FV_ERR_BAD_STATE;
  const bool xb = c.resid_dtype == 1;          // bf16 residual stream
  const size_t xes = xb ? 2 : 4;
  if (keep_ratio == 0.0) {
    if (xb) return FV_ERR_UNSUPPORTED;
    // Skipped step (the paper's 100 % pruning ratio, Sec. 4.1): no token is forwarded, nothing enters the
    // KV cache; the output is the caching step's output map interpolated to this scale.
    if (c.cache_step < 0 || scale_idx <= c.cache_step) return FV_ERR_BAD_STATE;
    if (forced_idx_dev || idx_trace_dev) return FV_ERR_INVALID_ARG;
    cudaStream_t st0 = static_cast<cudaStream_t>(stream);
    const int h0 = c.h[scale_idx], w0 = c.w[scale_idx];
    if (launch_inv_fill(B, h0 * w0, ctx->inv, st0) != cudaSuccess) return FV_ERR_CUDA;
    if (launch_restore_rows_f32(ctx->step_cache, c.h[c.cache_step], c.w[c.cache_step], ctx->step_cache, ctx->inv, B, 0, h0, w0, c.C,
                                static_cast<float*>(out_dev), c.interp_mode, st0) != cudaSuccess)
      return FV_ERR_CUDA;
    ctx->next_step += 1;
    return FV_OK;
  }
  const bool pruned = keep_ratio < 1.0;
  if (pruned && (c.cache_step < 0 || scale_idx <= c.cache_step)) return FV_ERR_BAD_STATE;
  if (!pruned && (forced_idx_dev || idx_trace_dev)) return FV_ERR_INVALID_ARG;
  const int h = c.h[scale_idx], w = c.w[scale_idx], n = h * w, C = c.C, F = c.C * c.mlp_ratio;
  const int k = pruned ? fv_k_for(keep_ratio, h, w) : n;
  const int M = B * k;
  if (ctx->kv_len + k > c.kv_capacity) return FV_ERR_CAPACITY;
  if (c.cross_len && scale_idx > 0 && !ctx->text_ready) return FV_ERR_BAD_STATE;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  void* x = out_dev;
  // (per-step granularity, pruned step: the output map is written whole by the final restoration)
  if (out_dev != tokens_dev && !(pruned && c.granularity == 1) &&
      cudaMemcpyAsync(out_dev, tokens_dev, (size_t)B * n * C * xes, cudaMemcpyDeviceToDevice, st) != cudaSuccess)
    return FV_ERR_CUDA;
  if (c.cross_len && scale_idx == 0) {
    fv_status s = fv_prepare_text(ctx, B, stream);
    if (s != FV_OK) return s;
  }
  const bool write_cache = (scale_idx == c.cache_step);
  const int hc = c.cache_step >= 0 ? c.h[c.cache_step] : 1, wc = c.cache_step >= 0 ? c.w[c.cache_step] : 1;
  const int mod_stride = 6 * C;
  fv_status s = FV_OK;
  cudaError_t e = cudaSuccess;
  const bool whole_step = c.granularity == 1;
  // Per sublayer (the paper): every sublayer selects from the full map x and restores into it.
  // Per step: one selection here, the blocks then run on the compact rows xr = ctx->xc as if unpruned.
  const bool sub_pruned = pruned && !whole_step;
  void* xr = x;         // residual stream the blocks update
  int nr = n;           // its rows per image
  const int32_t* step_idx = nullptr;   // per-step granularity: the kept indices of the whole step
  if (pruned && whole_step) {
    const int32_t* idx = forced_idx_dev;
    if (forced_idx_dev) {
      e = launch_inv_from_idx(forced_idx_dev, B, k, n, ctx->inv, st);
    } else {
      idx = ctx->idx;
      if (cudaMemsetAsync(ctx->sel_ws, 0, select_ticket_bytes(B), st) != cudaSuccess) return FV_ERR_CUDA;
      e = launch_select(tokens_dev, B, n, C, k, ctx->idx, ctx->inv, nullptr, nullptr, ctx->sel_ws, false, st);
    }
    if (e != cudaSuccess) return FV_ERR_CUDA;
    if (idx_trace_dev && cudaMemcpyAsync(idx_trace_dev, idx, (size_t)B * k * 4, cudaMemcpyDeviceToDevice, st) != cudaSuccess) return FV_ERR_CUDA;
    if (launch_gather_rows(static_cast<const float*>(tokens_dev), idx, B, n, k, C, ctx->xc, ctx->status, st) != cudaSuccess) return FV_ERR_CUDA;
    xr = ctx->xc;
    nr = k;
    step_idx = idx;
  }
  // Column sums of x (Eq. 4) for the next selection are left in the selection scratch by the restore
  // kernel of the sublayer before it; only the first sublayer of a step has to sum the map itself.
  bool have_partials = false;
  const bool selecting = sub_pruned && !forced_idx_dev;
  if (selecting && cudaMemsetAsync(ctx->sel_ws, 0, select_ticket_bytes(B), st) != cudaSuccess) return FV_ERR_CUDA;
  // Optional (fv_step_fused_selection): free-running selections take one launch each -- the previous sublayer's
  // kept-row restoration, the selection and the gather + LayerNorm of the newly kept rows (select_fused_kernel).  The
  // kept rows of a sublayer are then restored by the NEXT sublayer's launch; only the last sublayer of the step
  // restores its own.
  const bool fused = selecting && g_step_fused && !xb && select_fused_supported(B, n, C);
  bool pending = false;                 // a kept-row restoration waits for the next fused selection
  const float* pending_gamma = nullptr;
  int flip = 0;

  // A failed launch between the fork to the side stream and the join must not leave the side stream's part of the
  // restoration unordered against whatever the caller does next with x, the selection scratch or the context.
  bool forked = false;
  struct JoinGuard {
    cudaStream_t st; cudaEvent_t ev; const bool& forked;
    ~JoinGuard() { if (forked) cudaStreamWaitEvent(st, ev, 0); }
  } join_guard{st, ctx->ev_join, forked};

  for (int l = 0; l < c.L && s == FV_OK; ++l) {
    const float* mod = ctx->mod + (size_t)l * c.B_max * 6 * C;
    char* kbase = ctx->kv + (size_t)l * ctx->kv_block_bytes;
    for (int sub = 0; sub < ctx->n_sub && s == FV_OK; ++sub) {
      const int kind = (ctx->n_sub == 3) ? sub : (sub == 0 ? 0 : 2);  // 0 self-attention, 1 cross-attention, 2 FFN
      char* cache_sub = (ctx->cache && !whole_step) ? ctx->cache + ((size_t)l * ctx->n_sub + sub) * ctx->cache_sub_bytes : nullptr;
      const size_t trace_off = ((size_t)l * ctx->n_sub + sub) * (size_t)B * k;
      // ---- Pivotal Token Selection
      const int32_t* idx = nullptr;
      if (sub_pruned) {
        if (forced_idx_dev) {
          idx = forced_idx_dev + trace_off;
          e = launch_inv_from_idx(idx, B, k, n, ctx->inv, st);
        } else if (!fused) {
          idx = ctx->idx;
          e = launch_select(x, B, n, C, k, ctx->idx, ctx->inv, nullptr, nullptr, ctx->sel_ws, have_partials, st, xb);
        }
        if (e != cudaSuccess) { s = FV_ERR_CUDA; break; }
        if (!fused && idx_trace_dev && cudaMemcpyAsync(idx_trace_dev + trace_off, idx, (size_t)B * k * 4, cudaMemcpyDeviceToDevice, st) != cudaSuccess) {
          s = FV_ERR_CUDA; break;
        }
      }
      // ---- gather + LayerNorm (+ AdaLN modulation)
      const float* sigma = kind == 0 ? mod : (kind == 2 ? mod + 3 * C : nullptr);
      const float* beta = kind == 0 ? mod + C : (kind == 2 ? mod + 4 * C : nullptr);
      const float* gamma = kind == 0 ? mod + 2 * C : (kind == 2 ? mod + 5 * C : nullptr);
      const bool more = selecting && !(l == c.L - 1 && sub == ctx->n_sub - 1);
      int32_t* inv_cur = ctx->inv;
      if (fused) {
        int32_t* idx_cur = flip ? ctx->idx2 : ctx->idx;
        inv_cur = flip ? ctx->inv2 : ctx->inv;
        FusedSelect f{};
        f.x = static_cast<float*>(x); f.B = B; f.n = n; f.C = C; f.k = k; f.mod_stride = mod_stride;
        f.sel_ws = ctx->sel_ws; f.fused_ws = ctx->fsel_ws; f.idx = idx_cur; f.inv = inv_cur;
        f.sigma = sigma; f.beta = beta; f.a_out = ctx->a_buf; f.status = ctx->status;
        f.done_total = &ctx->fsel_done; f.epoch = &ctx->fsel_epoch;
        if (pending) {
          // the rows of the previous sublayer that were not kept (side stream) must be in x, and their sums folded
          if (cudaStreamWaitEvent(st, ctx->ev_join, 0) != cudaSuccess) { s = FV_ERR_CUDA; break; }
          forked = false;
          f.y = ctx->y_buf; f.idx_prev = flip ? ctx->idx : ctx->idx2; f.gamma_prev = pending_gamma;
        } else if (launch_colsum(static_cast<const float*>(x), B, n, C, ctx->sel_ws, st) != cudaSuccess) {   // first sublayer of the step: sum the map itself
          s = FV_ERR_CUDA; break;
        }
        if (launch_select_fused(f, st) != cudaSuccess) { s = FV_ERR_CUDA; break; }
        pending = false;
        idx = idx_cur;
        flip ^= 1;
        if (idx_trace_dev && cudaMemcpyAsync(idx_trace_dev + trace_off, idx, (size_t)B * k * 4, cudaMemcpyDeviceToDevice, st) != cudaSuccess) {
          s = FV_ERR_CUDA; break;
        }
      }
      if (sub_pruned) {
        // Cached Token Restoration of the rows that were NOT kept needs only the selection and the cache:
        // it runs on the side stream while the gather and the branch below work on the kept rows (the two
        // touch disjoint rows of x).
        if (cudaEventRecord(ctx->ev_fork, st) != cudaSuccess || cudaStreamWaitEvent(ctx->side, ctx->ev_fork, 0) != cudaSuccess) { s = FV_ERR_CUDA; break; }
        e = launch_restore_residual(x, ctx->y_buf, cache_sub, inv_cur, gamma, mod_stride, B, k, h, w, hc, wc, C,
                                    more ? ctx->sel_ws : nullptr, (fused && more) ? 3 : 1, c.interp_mode, ctx->side, xb);
        const cudaError_t e_join = cudaEventRecord(ctx->ev_join, ctx->side);   // recorded even if the launch failed
        forked = e_join == cudaSuccess;
        if (e != cudaSuccess || e_join != cudaSuccess) { s = FV_ERR_CUDA; break; }
      }
      if (!fused) {
        e = launch_gather_ln(xr, idx, B, nr, k, C, sigma, beta, mod_stride, ctx->a_buf, ctx->status, st, xb);
        if (e != cudaSuccess) { s = FV_ERR_CUDA; break; }
      }
      // ---- branch on the compact rows
      GemmArgs g{};
      g.status = ctx->status; g.rows_per_image = k; g.mod_stride = mod_stride; g.splitk_ws = ctx->splitk_ws;
      const void* last_in = nullptr; const void* last_w = nullptr; const void* last_b = nullptr; int last_K = C;
      if (kind == 0) {
        g.a = ctx->a_buf; g.w = ctx->w_qkv[l]; g.bias = ctx->b_qkv[l]; g.M = M; g.N = 3 * C; g.K = C;
        g.epilogue = EPI_QKV_SPLIT; g.out = ctx->q_buf; g.q_cols = C; g.C = C;
        g.k_cache = kbase; g.vt_cache = kbase + ctx->k_bytes; g.kv_capacity = c.kv_capacity; g.kv_offset = ctx->kv_len;
        // optional: cosine attention and rotary positions on q and k; a kept row's angle is that of its original slot
        g.qk_scale = ctx->qk_scale ? ctx->qk_scale + (size_t)l * c.H : nullptr;
        g.rope_table = ctx->rope_tab.empty() ? nullptr : ctx->rope_tab[scale_idx];
        g.rope_idx = sub_pruned ? idx : step_idx;
        g.head_dim = C / c.H;
        s = launch_gemm(g, st);
        if (s != FV_OK) break;
        AttnArgs a{};
        a.q = ctx->q_buf; a.k = kbase; a.vt = kbase + ctx->k_bytes; a.out = ctx->o_buf; a.B = B; a.rows = k; a.H = c.H; a.C = C;
        a.kv_len = ctx->kv_len + k; a.kv_capacity = c.kv_capacity; a.status = ctx->status; a.workspace = ctx->attn_ws;
        s = launch_attention(a, st);
        if (s != FV_OK) break;
        last_in = ctx->o_buf; last_w = ctx->w_o[l]; last_b = ctx->b_o[l];
      } else if (kind == 1) {
        g.a = ctx->a_buf; g.w = ctx->w_q_x[l]; g.bias = nullptr; g.M = M; g.N = C; g.K = C; g.epilogue = EPI_BF16; g.out = ctx->q_buf;
        s = launch_gemm(g, st);
        if (s != FV_OK) break;
        AttnArgs a{};
        a.q = ctx->q_buf; a.k = text_k(ctx, l); a.vt = text_k(ctx, l) + ctx->text_k_bytes; a.out = ctx->o_buf; a.B = B; a.rows = k;
        a.H = c.H; a.C = C; a.kv_len = c.cross_len; a.kv_capacity = c.cross_len; a.status = ctx->status; a.workspace = ctx->attn_ws;
        s = launch_attention(a, st);
        if (s != FV_OK) break;
        last_in = ctx->o_buf; last_w = ctx->w_o_x[l]; last_b = nullptr;
      } else {
        g.a = ctx->a_buf; g.w = ctx->w_fc1[l]; g.bias = ctx->b_fc1[l]; g.M = M; g.N = F; g.K = C; g.epilogue = EPI_GELU_BF16;
        g.out = ctx->h_buf;
        s = launch_gemm(g, st);
        if (s != FV_OK) break;
        last_in = ctx->h_buf; last_w = ctx->w_fc2[l]; last_b = ctx->b_fc2[l]; last_K = F;
      }
      // ---- last projection, then Cached Token Restoration + gate + residual
      GemmArgs o{};
      o.status = ctx->status; o.rows_per_image = k; o.mod_stride = mod_stride; o.splitk_ws = ctx->splitk_ws;
      o.a = last_in; o.w = last_w; o.bias = last_b; o.M = M; o.N = C; o.K = last_K;
      if (sub_pruned) {
        o.epilogue = EPI_BF16; o.out = ctx->y_buf;
        s = launch_gemm(o, st);
        if (s != FV_OK) break;
        if (fused && more) {     // the next sublayer's launch restores these kept rows
          pending = true;
          pending_gamma = gamma;
          continue;
        }
        if (cudaStreamWaitEvent(st, ctx->ev_join, 0) != cudaSuccess) { s = FV_ERR_CUDA; break; }
        forked = false;
        e = launch_restore_residual(x, ctx->y_buf, cache_sub, inv_cur, gamma, mod_stride, B, k, h, w, hc, wc, C,
                                    more ? ctx->sel_ws : nullptr, 2, c.interp_mode, st, xb);
        if (e != cudaSuccess) { s = FV_ERR_CUDA; break; }
        have_partials = more;
      } else {
        o.epilogue = xb ? EPI_RESIDUAL_XBF16 : EPI_RESIDUAL; o.out = xr; o.gamma = gamma; o.aux = (write_cache && !whole_step) ? cache_sub : nullptr;
        s = launch_gemm(o, st);
        if (s != FV_OK) break;
      }
    }
  }
  if (s != FV_OK) return s;
  if (write_cache && !xb &&   // (a bf16 stream has no skipped steps and no per-step granularity: nothing reads this copy)
      cudaMemcpyAsync(ctx->step_cache, x, (size_t)B * n * C * sizeof(float), cudaMemcpyDeviceToDevice, st) != cudaSuccess)
    return FV_ERR_CUDA;  // the step-level cache: this step's output map (image stride n*C == n_cache*C here)
  if (whole_step && pruned &&
      launch_restore_rows_f32(ctx->step_cache, hc, wc, ctx->xc, ctx->inv, B, k, h, w, C, static_cast<float*>(out_dev), c.interp_mode, st) != cudaSuccess)
    return FV_ERR_CUDA;
  if (s != FV_OK) return s;
  ctx->kv_len += k;
  ctx->next_step += 1;
  return FV_OK;
}

// fv_var_step for callers whose token maps live in host memory.  The copies run on two streams of the context
// (one per direction) over two staging buffers per direction, ordered against the caller's stream by events:
// the input of call i+1 travels while call i computes, and the result of call i travels while call i+1 computes.
size_t fv_var_step_host_staging_bytes(const fv_config* cfg) {
  if (!config_ok(cfg)) return 0;
  return 4 * align_up((size_t)cfg->B_max * max_tokens(cfg) * cfg->C * (cfg->resid_dtype == 1 ? 2 : 4), 1024);
}

fv_status fv_var_step_host(fv_ctx* ctx, const void* tokens_host, int32_t B, int32_t scale_idx, double keep_ratio, void* out_host,
                           void* staging_dev, size_t staging_bytes, void* stream) {
  if (!ctx || !tokens_host || !out_host || !staging_dev || B <= 0 || B > ctx->cfg.B_max) return FV_ERR_INVALID_ARG;
  if (scale_idx < 0 || scale_idx >= ctx->cfg.n_steps || (reinterpret_cast<uintptr_t>(staging_dev) & 1023u)) return FV_ERR_INVALID_ARG;
  if (staging_bytes < fv_var_step_host_staging_bytes(&ctx->cfg)) return FV_ERR_CAPACITY;
  if (!ctx->io_in) {
    bool ok = cudaStreamCreateWithFlags(&ctx->io_in, cudaStreamNonBlocking) == cudaSuccess &&
              cudaStreamCreateWithFlags(&ctx->io_out, cudaStreamNonBlocking) == cudaSuccess;
    for (int i = 0; i < 2 && ok; ++i)
      for (cudaEvent_t* e : {&ctx->ev_in[i], &ctx->ev_used[i], &ctx->ev_out[i], &ctx->ev_copied[i]})
        ok = ok && cudaEventCreateWithFlags(e, cudaEventDisableTiming) == cudaSuccess;
    if (!ok) return FV_ERR_CUDA;
  }
  const fv_config& c = ctx->cfg;
  const size_t half = fv_var_step_host_staging_bytes(&c) / 4;
  const size_t bytes = (size_t)B * c.h[scale_idx] * c.w[scale_idx] * c.C * (c.resid_dtype == 1 ? 2 : 4);
  const int p = (int)(ctx->io_count & 1u);
  void* in_dev = static_cast<char*>(staging_dev) + (size_t)p * half;
  void* out_dev = static_cast<char*>(staging_dev) + (size_t)(2 + p) * half;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  // in: this buffer's previous reader (the step two calls ago) must be done
  if (ctx->used_rec[p] && cudaStreamWaitEvent(ctx->io_in, ctx->ev_used[p], 0) != cudaSuccess) return FV_ERR_CUDA;
  if (cudaMemcpyAsync(in_dev, tokens_host, bytes, cudaMemcpyHostToDevice, ctx->io_in) != cudaSuccess ||
      cudaEventRecord(ctx->ev_in[p], ctx->io_in) != cudaSuccess || cudaStreamWaitEvent(st, ctx->ev_in[p], 0) != cudaSuccess)
    return FV_ERR_CUDA;
  // out: this buffer's previous copy to the host must be done before the step overwrites it
  if (ctx->copied_rec[p] && cudaStreamWaitEvent(st, ctx->ev_copied[p], 0) != cudaSuccess) return FV_ERR_CUDA;
  const fv_status s = fv_var_step(ctx, in_dev, B, scale_idx, keep_ratio, out_dev, nullptr, nullptr, stream);
  if (s != FV_OK) return s;
  if (cudaEventRecord(ctx->ev_used[p], st) != cudaSuccess || cudaEventRecord(ctx->ev_out[p], st) != cudaSuccess) return FV_ERR_CUDA;
  ctx->used_rec[p] = true;
  if (cudaStreamWaitEvent(ctx->io_out, ctx->ev_out[p], 0) != cudaSuccess ||
      cudaMemcpyAsync(out_host, out_dev, bytes, cudaMemcpyDeviceToHost, ctx->io_out) != cudaSuccess ||
      cudaEventRecord(ctx->ev_copied[p], ctx->io_out) != cudaSuccess)
    return FV_ERR_CUDA;
  ctx->copied_rec[p] = true;
  ctx->io_count += 1;
  return FV_OK;
}

// Makes `stream` wait for every result copy fv_var_step_host has enqueued: once the stream has run, they have landed.
fv_status fv_host_io_flush(fv_ctx* ctx, void* stream) {
  if (!ctx) return FV_ERR_INVALID_ARG;
  for (int p = 0; p < 2; ++p)
    if (ctx->copied_rec[p] && cudaStreamWaitEvent(static_cast<cudaStream_t>(stream), ctx->ev_copied[p], 0) != cudaSuccess) return FV_ERR_CUDA;
  return FV_OK;
}

void fv_struct_sizes(size_t* sizes3_host) {
  if (!sizes3_host) return;
  sizes3_host[0] = sizeof(fv_config); sizes3_host[1] = sizeof(fv_weights); sizes3_host[2] = sizeof(fv_generator);
}

}  // extern "C"
