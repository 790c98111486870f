/* fastvar.h -- C ABI of the B200 (sm_100a) hot path of FastVAR's cached token pruning:
 * the pruned large-scale next-scale-prediction step of a VAR transformer.
 *
 * Conventions (all entry points)
 *   - Pointers named *_dev are DEVICE pointers, *_host are HOST pointers.  Every device buffer is
 *     allocated and owned by the caller; the library allocates no device memory, keeps no copy of
 *     weights and only borrows the pointers it is given (they must stay valid while used).
 *   - `stream` is a cudaStream_t passed as void* (NULL = the legacy default stream).  All device
 *     work is enqueued on it; no entry point synchronises with the device unless it says so.
 *   - bf16 = bfloat16, row-major.  "Token map" layout is [B, h*w, C], tokens row-major over (y, x).
 *   - Linear weights are stored [out_features, in_features] (y = a * W^T + b).
 *   - Every call returns fv_status; argument and state errors are detected on the host BEFORE any
 *     launch.  Device-side trouble (a bounded wait that expired) is recorded in a status word in the
 *     workspace and reported by fv_device_status(); kernels never trap and never wait unboundedly.
 *   - Results are deterministic: the same inputs give bit-identical outputs run to run.
 */
#ifndef FASTVAR_H_
#define FASTVAR_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct fv_ctx fv_ctx; /* opaque; host-side metadata only */

typedef enum {
  FV_OK = 0,
  FV_ERR_INVALID_ARG = 1, /* NULL pointer, non-positive size, ratio outside (0,1], bad alignment   */
  FV_ERR_BAD_STATE = 2,   /* scale step taken out of order, missing cache, ...                       */
  FV_ERR_CAPACITY = 3,    /* KV cache or workspace too small for this call                           */
  FV_ERR_UNSUPPORTED = 4, /* shape outside what the kernels cover (stated per call)                  */
  FV_ERR_CUDA = 5,        /* a CUDA runtime / driver call failed (launch error, descriptor encoding) */
  FV_ERR_TIMEOUT = 6,     /* a bounded device-side wait expired (see fv_device_status)               */
  FV_ERR_DEVICE_DATA = 7  /* a kernel met an index outside its range and clamped it (fv_device_status) */
} fv_status;

const char *fv_status_string(fv_status s);

/* Kept-token count of Pivotal Token Selection (Sec. 3.3): k = ceil(keep_ratio * h * w), clamped to
 * [1, h*w]; keep_ratio = 1 - the paper's pruning ratio (Sec. 4.1).  Pure host function. */
int32_t fv_k_for(double keep_ratio, int32_t h, int32_t w);

/* ------------------------------------------------------------------------------------------------
 * (1) Pivotal Token Selection -- Sec. 3.3 "Pivotal Token Selection", Eq. 4-5, Algorithm 1 (first
 *     routine).  Per image: mean token over the h*w tokens (Eq. 4), score of every token = sum over
 *     channels of the squared deviation from that mean (Algorithm 1; the square of Eq. 5's norm, same
 *     ranking), exact top-k with ties going to the LOWEST token index, kept indices emitted in
 *     ASCENDING order.
 *   x_dev        [B, h*w, C] fp32 token map (the residual stream entering a sublayer).  C % 4 == 0.
 *   keep_ratio   in (0, 1]; k = fv_k_for(keep_ratio, h, w) is also written to *k_out_host if non-NULL.
 *   idx_out_dev  [B, k] int32, ascending per image.
 *   inv_out_dev  [B, h*w] int32 or NULL: position j of token t in idx, or -1 if pruned.
 *   score_out_dev[B, h*w] fp32 or NULL: the scores.
 *   near_tie_dev [B] int32 or NULL: number of tokens whose score is within 1e-5 (relative) of the
 *                k-th largest score (>= 1; values > 1 mean the kept set is decided by a near-tie).
 *   workspace_dev scratch of at least fv_prune_select_workspace_bytes(B, h*w, C) bytes, 16-byte aligned.
 * Errors: INVALID_ARG (NULLs, sizes, ratio, alignment), CAPACITY (workspace too small),
 *         UNSUPPORTED (h*w > 49152), CUDA (launch failed).  */
size_t fv_prune_select_workspace_bytes(int32_t B, int32_t n_tokens, int32_t C);
fv_status fv_prune_select(const float *x_dev, int32_t B, int32_t h, int32_t w, int32_t C,
                          double keep_ratio, int32_t *idx_out_dev, int32_t *inv_out_dev,
                          float *score_out_dev, int32_t *near_tie_dev, int32_t *k_out_host,
                          void *workspace_dev, size_t workspace_bytes, void *stream);

/* Same selection, for callers that cannot allocate.  (The paper has no counterpart of this call; it
 * exists for the deployment reason below.)  Some hosts of this library may not call cudaMalloc: a
 * serving process that split all device memory into fixed pools at start-up, or a plug-in that must
 * not touch the allocator because allocation synchronises the device under its pipeline.  They
 * cannot provide `workspace_dev`, so this variant keeps the scratch (arrival counters, partial column
 * sums, scores) in a fixed array inside the library's device image: fv_prune_select_static_capacity()
 * bytes (8 MiB), held by every GPU that loads the library until the process exits.
 *   - Inputs and outputs are still the caller's; arguments as in fv_prune_select, minus the workspace.
 *   - It allocates nothing: no cudaMalloc / cudaFree, no allocating library routine.  Shapes whose
 *     scratch need, fv_prune_select_workspace_bytes(B, h*w, C), exceeds the capacity are refused with
 *     FV_ERR_CAPACITY (e.g. B = 2, 64x64 tokens, C = 2048 needs 2.3 MiB; B = 1, 128x128, C = 2048 needs
 *     4.2 MiB; B = 4 at 128x128, C = 2048 does not fit).
 *   - The first call on each device looks up the array's device address (with that device current);
 *     make that first call outside any stream capture.
 *   - All calls on a device share the one array and it keeps the previous call's contents; every
 *     call first clears the few counters that must start at zero (every other word it reads it has
 *     written itself), so leftovers are harmless, but two calls whose
 *     kernels overlap on the GPU (different streams, no ordering between them) race on it: order them.
 * Errors: INVALID_ARG, UNSUPPORTED (h*w > 49152), CAPACITY, CUDA. */
size_t fv_prune_select_static_capacity(void);
fv_status fv_prune_select_static(const float *x_dev, int32_t B, int32_t h, int32_t w, int32_t C,
                                 double keep_ratio, int32_t *idx_out_dev, int32_t *inv_out_dev,
                                 float *score_out_dev, int32_t *near_tie_dev, int32_t *k_out_host,
                                 void *stream);

/* ------------------------------------------------------------------------------------------------
 * (3) Cached Token Restoration -- Sec. 3.3 "Cached Token Restoration", Eq. 6, Algorithm 1 (second
 *     routine).  out[b,t,:] = pivots[b,j,:] if t == idx[b,j], else cache_prev[b, src(t), :] where
 *     src is the nearest-neighbour source of token t when the (hc,wc) map is interpolated to (h,w):
 *     src = floor(y*hc/h)*wc + floor(x*wc/w).  Exact (a copy): bit-identical to the inputs.
 *   cache_prev_dev [B, hc*wc, C] bf16 : the cached sublayer output y_{K-N}.
 *   pivots_dev     [B, k, C] bf16     : the forwarded rows.
 *   idx_dev        [B, k] int32       : their token indices (any order, no duplicates, in [0,h*w)).
 *   out_dev        [B, h*w, C] bf16.   C % 8 == 0.
 *   inv_scratch_dev[B, h*w] int32 scratch (overwritten).
 *   interp_mode    0: nearest, as above (the default reading of the paper's mode-less interpolate).
 *                  1: bilinear with half-pixel centres (source coordinate (dst+0.5)*in/out - 0.5 per axis,
 *                     clamped): an unkept token is the fp32 blend of four cached rows, rounded to bf16 once.
 *                  2: bicubic at the same coordinates (cubic convolution with a = -0.75 over 4 x 4 cached
 *                     tokens, tap indices clamped to the map), blended in fp32, rounded once.
 * Errors: INVALID_ARG, CUDA. */
fv_status fv_restore(const void *cache_prev_dev, int32_t hc, int32_t wc, const void *pivots_dev,
                     const int32_t *idx_dev, int32_t B, int32_t k, int32_t h, int32_t w, int32_t C,
                     void *out_dev, int32_t *inv_scratch_dev, int32_t interp_mode, void *stream);

/* ------------------------------------------------------------------------------------------------
 * (2) The pruned scale step -- Sec. 3.3 "Overview" and "Implementation", Fig. 3: at the pruned steps
 *     PTS runs before and CTR after EVERY attention and FFN layer; the per-layer outputs of the last
 *     unpruned step (K-N) are the cache; only the kept rows' K/V enter the KV cache.
 *
 * Model (the paper leaves the backbone block open; this is the block both this library and its CPU
 * oracle define): per block, for sublayer in (self-attention, [cross-attention], FFN):
 *     I = PTS(x)  (keep_ratio < 1)             a = LayerNorm(x[I]) (eps 1e-6, no affine)
 *     self-attn : a = a*(1+sigma1)+beta1; [q,k,v] = a*Wqkv^T+b; append k,v to the KV cache;
 *                 o = softmax(q K^T / sqrt(hd)) V over all cached keys + the rows just appended;
 *                 y = o*Wo^T+bo;  x += gamma1 * CTR(y)
 *     cross-attn: q = a*Wq^T; K,V = text*Wkv^T; y = softmax(q K^T/sqrt(hd)) V * Wo^T;  x += CTR(y)
 *     FFN       : a = a*(1+sigma2)+beta2; y = gelu_tanh(a*W1^T+b1)*W2^T+b2;  x += gamma2 * CTR(y)
 * At scale step `cache_step` (unpruned) every sublayer's y is stored (bf16) as that sublayer's cache.
 */
typedef struct {
  int32_t L;          /* transformer blocks                                                        */
  int32_t C;          /* width; C % 64 == 0                                                        */
  int32_t H;          /* heads; C / H must be 64 or 128                                            */
  int32_t mlp_ratio;  /* hidden = mlp_ratio * C                                                    */
  int32_t cross_len;  /* text tokens T (0 = no cross-attention sublayer); T % 8 == 0                */
  int32_t B_max;      /* largest batch any call will use                                           */
  int32_t n_steps;    /* number of scale steps K                                                   */
  const int32_t *h;   /* HOST arrays [n_steps]: token-map height / width per step (copied)         */
  const int32_t *w;
  int32_t cache_step; /* 0-based index of step K-N, the last unpruned step; -1 = never cache       */
  int32_t kv_capacity;/* KV rows per image per block the caller provides room for; % 8 == 0        */
  int32_t granularity;/* 0: selection / restoration around every attention and FFN layer (the paper).
                         1: around the whole stack of blocks of a scale step (see fv_var_step)          */
  /* Optional pieces of the pruned backbones (the paper names none of them; 0 = off, the default):       */
  float rope_base;    /* > 0: 2-D rotary positions on the self-attention's q and k.  Token (y, x) of the
                         (h, w) map sits at (y*h_K/h, x*w_K/w) in the last scale's frame; of a head's hd
                         channels the first half turns with the row, the second with the column coordinate,
                         pair (2j, 2j+1) of a half by coordinate * rope_base^(-j/(hd/4)).  At a pruned step
                         the angle is that of the token's ORIGINAL slot (its kept index), not of its row
                         in the compact tensor.                                                          */
  int32_t interp_mode;/* interpolate(.) of Eq. 6: 0 nearest (src = floor(dst*in/out)); 1 bilinear with
                         half-pixel centres (src = (dst+0.5)*in/out - 0.5, clamped); 2 bicubic (cubic
                         convolution, a = -0.75, 4 x 4 cached tokens, tap indices clamped to the map)     */
  int32_t resid_dtype;/* residual stream (the token maps of fv_var_step) in 0: fp32 (default); 1: bf16.  The paper
                         fixes no precision.  With 1 every read of the stream -- Eq. 4's sums, Eq. 5's scores, the
                         gather, the restoration -- moves half the bytes, and every update rounds the stream to bf16
                         once (the arithmetic stays fp32).  Supported with granularity 0, interp_mode 0, keep ratios
                         in (0, 1]; fv_generate and skipped steps need the fp32 stream (UNSUPPORTED otherwise)    */
} fv_config;

typedef struct { /* HOST arrays of length L holding DEVICE pointers; bf16 unless noted; borrowed   */
  const void *const *w_qkv;  /* [3C, C]  rows: Q then K then V; head h owns channels [h*hd,(h+1)*hd) */
  const void *const *b_qkv;  /* [3C]                                                               */
  const void *const *w_o;    /* [C, C]                                                             */
  const void *const *b_o;    /* [C]                                                                */
  const void *const *w_fc1;  /* [mlp_ratio*C, C]                                                   */
  const void *const *b_fc1;  /* [mlp_ratio*C]                                                      */
  const void *const *w_fc2;  /* [C, mlp_ratio*C]                                                   */
  const void *const *b_fc2;  /* [C]                                                                */
  const void *const *w_q_x;  /* [C, C]   cross-attention (arrays may be NULL when cross_len == 0)  */
  const void *const *w_kv_x; /* [2C, C]  rows: K then V                                            */
  const void *const *w_o_x;  /* [C, C]                                                             */
  const float *mod_dev;      /* [L, B_max, 6, C] fp32: sigma1, beta1, gamma1, sigma2, beta2, gamma2 */
  const void *text_dev;      /* [B_max, cross_len, C] bf16 or NULL                                 */
  const float *qk_scale_dev; /* NULL, or [L, H] fp32: cosine attention in the self-attention sublayer -- every
                                head's q and k are divided by their Euclidean norm (floored at 1e-12) and q is
                                multiplied by the head's scale; applied before the rotary rotation          */
} fv_weights;

size_t fv_workspace_bytes(const fv_config *cfg); /* scratch for fv_var_step                         */
size_t fv_kv_bytes(const fv_config *cfg);        /* KV cache of all blocks (+ text K/V)             */
size_t fv_cache_bytes(const fv_config *cfg);     /* output map of step K-N (fp32) + sublayer caches  */

/* Builds a context over caller-owned buffers (sizes from the three queries above, 1024-byte aligned).
 * Clears the KV buffer once (synchronously) so that never-written rows hold zeros.
 * Errors: INVALID_ARG, UNSUPPORTED (head dim not 64/128, C > 2048, ...), CUDA. */
fv_status fv_create(const fv_config *cfg, const fv_weights *weights, void *kv_dev, void *cache_dev,
                    void *workspace_dev, fv_ctx **out);
void fv_destroy(fv_ctx *ctx);
/* Rewinds to the start of a schedule: next step 0, empty KV cache. No device work. */
fv_status fv_reset(fv_ctx *ctx);
/* Resume support: read / set (next scale step, KV rows already held per image).  Setting a state
 * past `cache_step` asserts that the caller has filled the sublayer caches and KV prefix itself. */
fv_status fv_get_state(const fv_ctx *ctx, int32_t *next_step_host, int32_t *kv_len_host);
fv_status fv_set_state(fv_ctx *ctx, int32_t next_step, int32_t kv_len);
/* Device addresses inside the caller's buffers (for tests / resume): K rows [B_max, kv_capacity, C]
 * and V^T [B_max, C, kv_capacity] of one block; the cache [B_max, n_cache, C] of (block, sublayer). */
fv_status fv_kv_pointers(const fv_ctx *ctx, int32_t block, void **k_dev, void **vt_dev);
fv_status fv_cache_pointer(const fv_ctx *ctx, int32_t block, int32_t sublayer, void **cache_dev);
/* Projects the text tokens to per-block K / V^T for cross-attention (step-invariant).  Called by
 * fv_var_step at scale step 0; call it yourself after fv_set_state on a fresh context. */
fv_status fv_prepare_text(fv_ctx *ctx, int32_t B, void *stream);
/* Synchronises `stream` and reads the context's device status word: FV_OK, or -- with the kernel's code in
 * *code_host -- FV_ERR_TIMEOUT if a bounded wait expired since the last call (codes 101-105: operand loads, MMA
 * issue, epilogue, softmax, the self-test below) or FV_ERR_DEVICE_DATA if a kernel met an index outside its range
 * and clamped it (40: a token id outside the codebook; 41: a kept-row index outside the token map).  Clears the word. */
fv_status fv_device_status(fv_ctx *ctx, int32_t *code_host, void *stream);
/* Self-test of the convention above (no counterpart in the paper): one warp waits, with the library's bounded
 * wait, for limit_ns nanoseconds (at most 1e9) on a barrier that nothing ever completes, then records code 105
 * and returns normally.  Nothing traps; the context stays usable.  fv_device_status then reports FV_ERR_TIMEOUT. */
fv_status fv_selftest_expired_wait(fv_ctx *ctx, uint64_t limit_ns, void *stream);

/* One scale step over all L blocks.
 *   tokens_dev  [B, h*w, C] fp32 (bf16 with resid_dtype 1): residual stream entering block 0 at this scale.
 *   out_dev     [B, h*w, C] same type: residual stream after block L-1 (may alias tokens_dev).
 *   scale_idx   must equal the context's next step (steps are taken in order).
 *   keep_ratio  1.0 = unpruned path (no select / gather / restore work at all); in (0, 1) = FastVAR;
 *               0.0 = the step is skipped (the paper's 100 % pruning ratio, Sec. 4.1): out_dev is the output
 *               map of step cache_step interpolated (nearest) to this scale, nothing enters the KV cache.
 *   forced_idx_dev NULL, or int32 [L, n_sub, B, k]: use these kept indices (ascending per image)
 *               instead of selecting -- separates index parity from floating-point parity in tests.
 *   idx_trace_dev  NULL, or int32 [L, n_sub, B, k]: receives the kept indices of every sublayer.
 * n_sub = 3 with cross-attention else 2; sublayer order: self-attention, [cross-attention], FFN.
 *
 * granularity 1 (not the paper's configuration; the coarser reading "select once per scale step"): at a
 * pruned step PTS runs once on tokens_dev, the kept rows are gathered into a compact fp32 residual stream,
 * all L blocks run on those rows only (each block appends their K/V), and one CTR builds out_dev from the
 * compact result and the cached OUTPUT map of step cache_step (fp32 [B_max, n_cache, C]; that is what the
 * cache buffer then holds, fv_cache_pointer(ctx, 0, 0)).  forced_idx_dev / idx_trace_dev are int32 [B, k].
 * Errors: INVALID_ARG, BAD_STATE (wrong scale_idx; pruned step before the cache step),
 *         CAPACITY (kv_len + k > kv_capacity), CUDA. */
fv_status fv_var_step(fv_ctx *ctx, const void *tokens_dev, int32_t B, int32_t scale_idx,
                      double keep_ratio, void *out_dev, const int32_t *forced_idx_dev,
                      int32_t *idx_trace_dev, void *stream);

/* fv_var_step with the token maps in HOST memory (pinned memory makes the copies asynchronous).  Enqueues the
 * copy of tokens_host [B, h*w, C] fp32 to the device, the step (on `stream`), and the copy of its result to
 * out_host [B, h*w, C].  The copies run on two streams owned by the context, ordered against `stream` by events
 * over two staging buffers per direction, so the input of the next call and the result of the previous one
 * travel while a step computes.  tokens_host must hold its data when the call is made (the copy does not wait
 * for earlier work of `stream`).  out_host is valid after fv_host_io_flush(ctx, stream) and the completion of
 * `stream`.
 *   staging_dev: device scratch of fv_var_step_host_staging_bytes(cfg) bytes, 1024-byte aligned (two input and
 *   two output maps at their largest).  No forced indices / trace.  Errors: those of fv_var_step, CAPACITY.
 * fv_host_io_flush makes `stream` wait for every result copy enqueued so far. */
size_t fv_var_step_host_staging_bytes(const fv_config *cfg);
fv_status fv_var_step_host(fv_ctx *ctx, const void *tokens_host, int32_t B, int32_t scale_idx,
                           double keep_ratio, void *out_host, void *staging_dev, size_t staging_bytes,
                           void *stream);
fv_status fv_host_io_flush(fv_ctx *ctx, void *stream);

/* ------------------------------------------------------------------------------------------------
 * Building blocks of the step, exported for kernel-level parity tests and profiling.            */

/* Gather + LayerNorm + AdaLN modulate (the compaction of Algorithm 1's gather fused with the block's
 * pre-norm): a[b,j,:] = LN(x[b, idx[b,j], :]) * (1 + sigma[b,:]) + beta[b,:]  -> bf16.
 *   idx_dev NULL = all rows (k = n_tokens);  sigma_dev / beta_dev NULL = plain LayerNorm;
 *   their per-image stride is mod_stride floats.  C % 4 == 0, C <= 2048.
 *   status_dev NULL, or an int32 device word: an index outside [0, n_tokens) is clamped into the map (the read
 *   stays in bounds) and code 41 is left there. */
fv_status fv_gather_ln(const float *x_dev, const int32_t *idx_dev, int32_t B, int32_t n_tokens,
                       int32_t k, int32_t C, const float *sigma_dev, const float *beta_dev,
                       int32_t mod_stride, void *a_out_dev, int32_t *status_dev, void *stream);

/* Restore fused with gate and residual (Eq. 6 + the block's x += gamma * y):
 *   x[b,t,:] += gamma[b,:] * (inv[b,t] >= 0 ? y[b, inv[b,t], :] : cache[b, src(t), :]).
 * gamma_dev NULL = 1.  y, cache bf16; x fp32 in place.  C % 8 == 0.  interp_mode as for fv_restore (with 1
 * the cache term is the bilinear blend of four cached rows).
 *   colsum_ws_dev NULL, or a selection workspace (fv_prune_select_workspace_bytes(B, h*w, C) bytes, 16-byte
 *               aligned): the kernel then also leaves there the per-image column sums of the UPDATED map
 *               -- Eq. 4's sum over tokens for the next sublayer's selection -- so that
 *               fv_prune_select_after_restore can rank the map without summing it again.  They are kept as
 *               a few partial sums per image, see fv_prune_select_workspace_layout.
 *   part        0: every row.  1: only the rows that were NOT kept (they need the selection and the cache
 *               alone, so inside a step they run beside the sublayer's GEMMs).  2: only the kept rows, after
 *               part 1 on the same workspace (its sums continue part 1's and are then folded per image).
 *               Parts 1 and 2 together give the bits of part 0 in x (the sums add the rows in another order).
 * Errors: INVALID_ARG, CAPACITY (workspace too small), CUDA. */
fv_status fv_restore_residual(float *x_dev, const void *y_dev, const void *cache_dev,
                              const int32_t *inv_dev, const float *gamma_dev, int32_t mod_stride,
                              int32_t B, int32_t k, int32_t h, int32_t w, int32_t hc, int32_t wc,
                              int32_t C, int32_t interp_mode, void *colsum_ws_dev, size_t colsum_ws_bytes,
                              int32_t part, void *stream);
/* Pivotal Token Selection (as fv_prune_select) of a map whose column sums fv_restore_residual has left in
 * workspace_dev: the form every selection after the first takes inside fv_var_step. */
fv_status fv_prune_select_after_restore(const float *x_dev, int32_t B, int32_t h, int32_t w, int32_t C,
                                        double keep_ratio, int32_t *idx_out_dev, int32_t *inv_out_dev,
                                        float *score_out_dev, int32_t *near_tie_dev, int32_t *k_out_host,
                                        void *workspace_dev, size_t workspace_bytes, void *stream);
/* Where a selection workspace keeps the column sums (for tests): they sit at byte offset *offset_host as
 * fp32 [B, *n_partials_host, C]; the sum over the partials of image b is the column sum of its map. */
fv_status fv_prune_select_workspace_layout(int32_t B, int32_t n_tokens, int32_t C, size_t *offset_host,
                                           int32_t *n_partials_host);
/* Test / profiling hook (process-wide).  on != 0: inside fv_var_step every free-running selection becomes ONE launch
 * that also restores the previous sublayer's kept rows before it and gathers + normalises the newly kept rows after
 * it (its CTAs wait on one another with bounded waits; the grid never exceeds what the GPU holds at once).  Off by
 * default: measured on B200 the separate kernels (selection, gather + LayerNorm, kept-row restoration), whose launch
 * gaps programmatic dependent launch already hides, are as fast or faster.  The two forms add Eq. 4's column sums in
 * a different order, so their scores agree to fp32 rounding and a near-tie at the threshold may fall the other way;
 * given the kept sets the token maps are the same bit for bit.  Forced-index steps always take the separate kernels. */
fv_status fv_step_fused_selection(int32_t on);
/* Test / profiling hook (process-wide): how the kept-row part of a restoration folds its column sums.
 * 0 = chosen per shape (default); 1 = always through global memory (arrival counters); 2 = inside
 * thread-block clusters wherever the shape allows it. */
fv_status fv_restore_force_fold(int32_t mode);

/* tcgen05 GEMM  out = epilogue(A[M,K] * W[N,K]^T + bias), bf16 operands, fp32 accumulation in TMEM.
 *   epilogue 0: bf16 store to out [M, N].          1: tanh-GELU then bf16 store.
 *   epilogue 2: fp32 residual: out[m,n] += gamma[m / rows_per_image, n] * (acc + bias)  (out fp32;
 *               gamma NULL = 1; if aux_dev != NULL the bf16 value of acc+bias is also stored there).
 *   epilogue 4: fp32 store of acc + bias to out [M, N] (aux_dev, gamma_dev ignored).  3 is not a public value.
 *   epilogue 5: as 2 for a bf16 residual stream: out bf16 [M, N] in place, out = bf16(float(out) + gamma * (acc + bias)).
 *   K % 8 == 0, N % 8 == 0, all pointers 16-byte aligned.  bias_dev may be NULL.
 *   W is treated as a constant of the stream: its first tiles are requested as soon as the kernel starts,
 *   which (programmatic dependent launch) can be while the kernel enqueued just before it is still
 *   finishing -- do not produce W with that kernel.  A, bias and the outputs are touched only after it.
 *   status_dev: int32 device word that receives a non-zero code if a bounded wait expires (or NULL).
 *   splitk_ws_dev: NULL, or scratch of fv_gemm_splitk_workspace_bytes() bytes whose first 4096 bytes are
 *               zero (the kernel leaves them zero): shapes with too few output tiles to occupy the GPU
 *               (few rows against a large weight matrix) are then split along K, the slices' fp32
 *               partial sums added in slice order.  CAPACITY if splitk_ws_bytes is too small. */
size_t fv_gemm_splitk_workspace_bytes(void);
/* Test / profiling hook (process-wide): which GEMM kernel fv_gemm_bf16 and the step use when no K split is
 * taken.  0 = chosen per shape (default); 1 = one CTA per 128-row tile, width chosen per shape; 2 = CTA
 * pairs sharing 256 x 256 tiles (tcgen05 cta_group::2); 3 = CTA pairs, 256 x 128 tiles; 4 / 5 / 6 = one CTA
 * per tile of width 128 / 192 / 256; 7 = one CTA per tile of width 64; 8 / 9 = K split over a cluster of 4 / 2
 * CTAs per 128-wide tile, 10 / 11 = the same with 64-wide tiles (partials reduced through distributed shared
 * memory; no scratch).  INVALID_ARG outside 0..11. */
fv_status fv_gemm_force_path(int32_t path);
fv_status fv_gemm_bf16(const void *a_dev, const void *w_dev, const void *bias_dev, int32_t M,
                       int32_t N, int32_t K, int32_t epilogue, void *out_dev, void *aux_dev,
                       const float *gamma_dev, int32_t mod_stride, int32_t rows_per_image,
                       int32_t *status_dev, void *splitk_ws_dev, size_t splitk_ws_bytes, void *stream);

/* Flash-style attention over a KV cache (Sec. 3.1 KV cache; Sec. 3.3: pivotal queries attend to the
 * cached keys of all earlier scales plus the current pivotal keys; no mask inside a step).
 *   q_dev  [B*rows, C] bf16 (image b owns rows [b*rows, (b+1)*rows)); head h = channels [h*hd, ..).
 *   k_dev  [B, kv_capacity, C] bf16;  vt_dev [B, C, kv_capacity] bf16 (V transposed).
 *   kv_len keys are attended (rows [0, kv_len) of every image).  out_dev [B*rows, C] bf16.
 *   hd = C / H in {64, 128}; kv_capacity % 8 == 0.
 *   workspace_dev NULL: one CTA per (256 queries, head, image).  Else fv_attention_workspace_bytes() bytes of
 *               scratch, 16-byte aligned, whose first 65536 bytes are zero (the kernel leaves them zero): the
 *               (queries, head, image, key tile) work is then cut into equal pieces, one per SM, and the
 *               pieces of one query block are merged in key order (same bits run to run).
 *               CAPACITY if workspace_bytes is too small. */
size_t fv_attention_workspace_bytes(void);
fv_status fv_attention(const void *q_dev, const void *k_dev, const void *vt_dev, int32_t B,
                       int32_t rows, int32_t H, int32_t C, int32_t kv_len, int32_t kv_capacity,
                       void *out_dev, int32_t *status_dev, void *workspace_dev, size_t workspace_bytes,
                       void *stream);
/* Test / profiling hook (process-wide): number of CTAs of a fv_attention launch that is given a workspace
 * (0 = one per SM where that pays, the default; n > 0 = always n pieces, capped at 160 and at what the work
 * allows; -1 = never cut the work, as if no workspace were given). */
fv_status fv_attention_force_ctas(int32_t ctas);

/* ------------------------------------------------------------------------------------------------
 * (4) The generation loop around the scale step -- Sec. 3.1: step k turns the token map of scale k into a
 *     residual f_k and the running prediction follows Eq. 2,
 *         r_k = interpolate(r_{k-1}, (h_k, w_k)) + f_k        (Eq. 3 is its unfolded form).
 *     The paper does not say how f_k is read off the transformer output nor how the next token map is
 *     built; this library and its CPU oracle take the plain construction of VAR-style models:
 *         logits = (LayerNorm(y) * (1 + sigma_h) + beta_h) * W_head^T + b_head       (V codebook entries)
 *         id     = argmax_v (logits_v + tau * noise_v), lowest id on ties   (noise NULL: greedy;
 *                  standard Gumbel noise: a draw from softmax(logits / tau).  The noise is an INPUT.)
 *         f_k    = codebook[id];   r_1 = f_1
 *         x_{k+1} = interpolate(r_k, (h_{k+1}, w_{k+1})) * W_in^T + b_in + pos_{k+1}
 *     interpolate = nearest neighbour, src = floor(dst * in / out) per axis, as for Eq. 6.            */

/* Head + token choice for one scale step.
 *   y_dev [B, n, C] fp32 (output of fv_var_step); mod_head_dev fp32 [B, 2, C] (sigma_h, beta_h);
 *   w_head_dev bf16 [V, C]; b_head_dev bf16 [V] or NULL; noise_dev fp32 [B*n, V] or NULL;
 *   ids_out_dev int32 [B, n]; logits_out_dev fp32 [B*n, V] or NULL (then the logits live in the workspace).
 *   workspace_dev: fv_head_workspace_bytes(B*n, C, V) bytes, 256-byte aligned; status_dev as in fv_gemm_bf16.
 *   The GEMM is the bf16 tensor-core GEMM (fp32 accumulation, fp32 logits); the comparison is exact on
 *   those fp32 values.  V % 8 == 0, C % 8 == 0, C <= 2048.  Errors: INVALID_ARG, CAPACITY, CUDA. */
size_t fv_head_workspace_bytes(int32_t rows, int32_t C, int32_t V);
fv_status fv_head_tokens(const float *y_dev, int32_t B, int32_t n, int32_t C, const float *mod_head_dev,
                         const void *w_head_dev, const void *b_head_dev, int32_t V,
                         const float *noise_dev, float tau, int32_t *ids_out_dev, float *logits_out_dev,
                         void *workspace_dev, size_t workspace_bytes, int32_t *status_dev, void *stream);

/* Token choice alone: ids[r] = argmax_v (logits[r, v] + tau * noise[r, v]), lowest v on ties.
 * logits_dev fp32 [rows, V]; noise_dev fp32 [rows, V] or NULL; V % 4 == 0. */
fv_status fv_argmax_rows(const float *logits_dev, const float *noise_dev, float tau, int32_t rows,
                         int32_t V, int32_t *ids_out_dev, void *stream);

/* Eq. 2: r_out[b, t, :] = (r_prev ? r_prev[b, src(t), :] : 0) + codebook[ids[b, t], :].
 *   ids_dev int32 [B, h*w] in [0, V) (an id outside is clamped and sets *status_dev, if given, to a
 *   non-zero code); codebook_dev fp32 [V, d]; r_prev_dev fp32 [B, hp*wp, d] or NULL (first step);
 *   r_out_dev fp32 [B, h*w, d] (must not alias r_prev_dev).  d % 4 == 0. */
fv_status fv_residual_accumulate(const int32_t *ids_dev, int32_t B, int32_t h, int32_t w,
                                 const float *codebook_dev, int32_t V, int32_t d,
                                 const float *r_prev_dev, int32_t hp, int32_t wp, float *r_out_dev,
                                 int32_t *status_dev, void *stream);

/* Token map entering the next scale: x[b, t, :] = r[b, src(t), :] * W_in^T + b_in + pos[t, :].
 *   r_dev fp32 [B, h*w, d]; w_in_dev fp32 [C, d]; b_in_dev fp32 [C] or NULL; pos_dev fp32 [h2*w2, C] or
 *   NULL; x_out_dev fp32 [B, h2*w2, C].  d in {8, 16, 32, 64}; C % 4 == 0. */
fv_status fv_next_scale_input(const float *r_dev, int32_t B, int32_t h, int32_t w, int32_t d, int32_t h2,
                              int32_t w2, const float *w_in_dev, const float *b_in_dev,
                              const float *pos_dev, int32_t C, float *x_out_dev, void *stream);

typedef struct {
  int32_t V, d;                 /* codebook entries and their width                                    */
  const float *codebook_dev;    /* [V, d] fp32                                                         */
  const void *w_head_dev;       /* [V, C] bf16                                                         */
  const void *b_head_dev;       /* [V] bf16 or NULL                                                    */
  const float *mod_head_dev;    /* [B_max, 2, C] fp32: sigma_h, beta_h                                 */
  const float *w_in_dev;        /* [C, d] fp32                                                         */
  const float *b_in_dev;        /* [C] fp32 or NULL                                                    */
  const float *const *pos_dev;  /* HOST array [n_steps] of device pointers [h_k*w_k, C] (entry 0 unused; NULL entries = none) */
  float tau;                    /* scale of the noise                                                  */
} fv_generator;

/* The whole K-step loop on `stream`: for every scale step of the context, fv_var_step, head + token
 * choice, Eq. 2, and the next token map.  The context is reset first.
 *   start_dev [B, h_0*w_0, C] fp32 : token map entering step 0 (not modified).
 *   keep_host [n_steps]           : keep ratio per step, as for fv_var_step.
 *   noise_host NULL, or HOST array [n_steps] of device pointers fp32 [B*h_k*w_k, V] (NULL entries = greedy).
 *   ids_out_dev int32 [B * sum_k h_k*w_k]: step k's ids [B, h_k*w_k] start at B * sum_{j<k} h_j*w_j.
 *   r_out_dev fp32 [B, h_K*w_K, d]: the final prediction r_K.
 *   workspace_dev: fv_generate_workspace_bytes(ctx, gen) bytes, 1024-byte aligned.
 * Device-side codes of every stage (an expired wait in the head GEMM, a token id outside the codebook) land in
 * the context's status word: read them with fv_device_status.  Errors: those of the calls it makes. */
size_t fv_generate_workspace_bytes(const fv_ctx *ctx, const fv_generator *gen);
fv_status fv_generate(fv_ctx *ctx, const fv_generator *gen, const float *start_dev, int32_t B,
                      const double *keep_host, const float *const *noise_host, int32_t *ids_out_dev,
                      float *r_out_dev, void *workspace_dev, size_t workspace_bytes, void *stream);

/* ------------------------------------------------------------------------------------------------
 * Measurement support (no counterpart in the paper; Appendix "efficiency profiling" motivates the
 * per-module breakdown).  Kernel classes, in array order: 0 select (column mean + score + top-k),
 * 1 gather+LayerNorm, 2 GEMM, 3 attention, 4 restore.
 *   fv_kernel_launches : kernels this library has launched since the last fv_profile_read.
 *   fv_profile_enable  : when on, every launch is bracketed by CUDA events on its stream.
 *   fv_profile_read    : synchronises the device; fills (each [5], HOST, may be NULL) the summed device
 *                        milliseconds per class (0 unless timing was on), launches per class, the
 *                        algorithmic work per class (bytes for classes 0,1,4; flops for 2,3) and the bytes
 *                        each class has to move to and from HBM once (operands + results), then clears. */
/* sizeof(fv_config), sizeof(fv_weights), sizeof(fv_generator) as this library was compiled: a binding checks
 * its own struct definitions against them before passing any struct. */
void fv_struct_sizes(size_t *sizes3_host);
uint64_t fv_kernel_launches(void);
fv_status fv_profile_enable(int32_t on);
fv_status fv_profile_read(double *ms_host, uint64_t *launches_host, double *work_host,
                          double *dram_bytes_host);

#ifdef __cplusplus
}
#endif
#endif /* FASTVAR_H_ */
