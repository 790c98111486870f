// The generation loop around the scale step (Sec. 3.1, Eq. 2-3): output head + token choice, residual
// accumulation r_k = interpolate(r_{k-1}) + codebook[id], and the token map entering the next scale.
// The head's contraction is the library's tcgen05 GEMM with an fp32 epilogue; the rest is memory-bound
// and lives here: a row-wise argmax (one warp per row of logits), a gather-and-add over the codebook, and
// the small d -> C map (d <= 64: a dot product per output element, no tensor-core shape).
#include <cuda_runtime.h>

#include <climits>
#include <cstdint>
#include <vector>

#include "internal.h"
#include "sm100.cuh"   // the device status codes

namespace fv {
namespace {

// ---- ids[r] = argmax_v (logits[r, v] + tau * noise[r, v]), lowest v on ties; one warp per row ----
__global__ void __launch_bounds__(256) argmax_rows_kernel(const float4* __restrict__ logits, const float4* __restrict__ noise, float tau,
                                                          int rows, int V4, int32_t* __restrict__ ids) {
  pdl_trigger();
  const int lane = threadIdx.x & 31;
  const int row = blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
  pdl_wait();
  if (row >= rows) return;
  const float4* lp = logits + (size_t)row * V4;
  const float4* np = noise ? noise + (size_t)row * V4 : nullptr;
  float best = -INFINITY;
  int bi = INT_MAX;
  for (int j0 = 0; j0 < V4; j0 += 128) {   // four loads per lane in flight
    float4 z[4];
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      const int j = j0 + lane + 32 * i;
      z[i] = j < V4 ? __ldcs(lp + j) : make_float4(-INFINITY, -INFINITY, -INFINITY, -INFINITY);
    }
    if (np) {
#pragma unroll
      for (int i = 0; i < 4; ++i) {
        const int j = j0 + lane + 32 * i;
        if (j < V4) {
          const float4 g = __ldcs(np + j);
          z[i].x = fmaf(tau, g.x, z[i].x); z[i].y = fmaf(tau, g.y, z[i].y); z[i].z = fmaf(tau, g.z, z[i].z); z[i].w = fmaf(tau, g.w, z[i].w);
        }
      }
    }
    // indices grow within a lane, so a strict comparison keeps the first occurrence
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      const int j = j0 + lane + 32 * i;
      if (z[i].x > best) { best = z[i].x; bi = 4 * j; }
      if (z[i].y > best) { best = z[i].y; bi = 4 * j + 1; }
      if (z[i].z > best) { best = z[i].z; bi = 4 * j + 2; }
      if (z[i].w > best) { best = z[i].w; bi = 4 * j + 3; }
    }
  }
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) {
    const float ov = __shfl_xor_sync(0xFFFFFFFFu, best, o);
    const int oi = __shfl_xor_sync(0xFFFFFFFFu, bi, o);
    if (ov > best || (ov == best && oi < bi)) { best = ov; bi = oi; }
  }
  if (lane == 0) ids[row] = bi == INT_MAX ? 0 : bi;   // a row of NaN / -inf: id 0
}

// ---- Eq. 2: r_out[b,t,:] = (r_prev ? r_prev[b, src(t), :] : 0) + codebook[ids[b,t], :] ----
__global__ void __launch_bounds__(256) residual_accumulate_kernel(const int32_t* __restrict__ ids, const float4* __restrict__ codebook,
                                                                  const float4* __restrict__ r_prev, int hp, int wp, int B, int h,
                                                                  int w, int d4, int V, float4* __restrict__ r_out, int32_t* status) {
  pdl_trigger();
  pdl_wait();
  const int n = h * w;
  const long total = (long)B * n * d4;
  for (long i = (long)blockIdx.x * blockDim.x + threadIdx.x; i < total; i += (long)gridDim.x * blockDim.x) {
    const int c = (int)(i % d4);
    const long tok = i / d4;
    const int t = (int)(tok % n), b = (int)(tok / n);
    int id = ids[tok];
    if (id < 0 || id >= V) {
      if (status) atomicCAS(status, 0, DEV_BAD_TOKEN_ID);
      id = id < 0 ? 0 : V - 1;
    }
    float4 f = __ldg(codebook + (size_t)id * d4 + c);
    if (r_prev) {
      const int y = t / w, x = t - y * w;
      const int src = (int)(((long)y * hp) / h) * wp + (int)(((long)x * wp) / w);
      const float4 p = r_prev[((size_t)b * hp * wp + src) * d4 + c];
      f.x += p.x; f.y += p.y; f.z += p.z; f.w += p.w;
    }
    r_out[i] = f;
  }
}

// ---- x[b,t,:] = r[b, src(t), :] * W_in^T + b_in + pos[t,:];  CTA = 32 tokens x all channels ----
constexpr int kNextTokens = 32;
template <int D>
__global__ void __launch_bounds__(256) next_input_kernel(const float* __restrict__ r, int h, int w, int h2, int w2, const float* __restrict__ w_in,
                                                         const float* __restrict__ b_in, const float* __restrict__ pos, int C, int B,
                                                         float* __restrict__ x_out) {
  __shared__ __align__(16) float r_s[kNextTokens][D];
  __shared__ int s_t2[kNextTokens];      // token index inside the next map (row of pos), per staged token
  pdl_trigger();
  const int n = h * w, n2 = h2 * w2;
  const long rows = (long)B * n2;
  const long row0 = (long)blockIdx.x * kNextTokens;
  pdl_wait();
  for (int i = threadIdx.x; i < kNextTokens * D; i += blockDim.x) {
    const int t = i / D, j = i - t * D;
    const long row = row0 + t;
    float v = 0.f;
    if (row < rows) {
      const int b = (int)(row / n2), t2 = (int)(row - (long)b * n2);
      const int y = t2 / w2, x = t2 - y * w2;
      const int src = (int)(((long)y * h) / h2) * w + (int)(((long)x * w) / w2);
      v = r[((size_t)b * n + src) * D + j];
      if (j == 0) s_t2[t] = t2;
    }
    r_s[t][j] = v;
  }
  __syncthreads();
  const int t_valid = (int)min((long)kNextTokens, rows - row0);
  for (int c = threadIdx.x; c < C; c += blockDim.x) {
    float wr[D];
#pragma unroll
    for (int j = 0; j < D; j += 4) {
      const float4 q = __ldg(reinterpret_cast<const float4*>(w_in + (size_t)c * D + j));
      wr[j] = q.x; wr[j + 1] = q.y; wr[j + 2] = q.z; wr[j + 3] = q.w;
    }
    const float bias = b_in ? __ldg(b_in + c) : 0.f;
    float* out = x_out + (size_t)row0 * C + c;
    for (int t0 = 0; t0 < t_valid; t0 += 8) {   // eight tokens at a time: their position-embedding loads go out together
      float pe[8];
#pragma unroll
      for (int u = 0; u < 8; ++u) pe[u] = (pos && t0 + u < t_valid) ? __ldg(pos + (size_t)s_t2[t0 + u] * C + c) : 0.f;
#pragma unroll
      for (int u = 0; u < 8; ++u) {
        if (t0 + u < t_valid) {
          float acc = 0.f;
#pragma unroll
          for (int j = 0; j < D; j += 4) {      // the token's vector is read as float4 broadcasts
            const float4 q = *reinterpret_cast<const float4*>(&r_s[t0 + u][j]);
            acc = fmaf(q.x, wr[j], acc); acc = fmaf(q.y, wr[j + 1], acc); acc = fmaf(q.z, wr[j + 2], acc); acc = fmaf(q.w, wr[j + 3], acc);
          }
          acc += bias;
          acc += pe[u];
          out[(size_t)(t0 + u) * C] = acc;
        }
      }
    }
  }
}

struct HeadLayout { size_t a, logits, splitk, total; };
HeadLayout head_layout(int rows, int C, int V, bool own_logits) {
  HeadLayout l{};
  size_t off = 0;
  l.a = off; off = align_up(off + (size_t)rows * C * 2, 256);
  l.logits = off; if (own_logits) off = align_up(off + (size_t)rows * V * 4, 256);
  l.splitk = off; off = align_up(off + gemm_splitk_ws_bytes(), 256);
  l.total = off;
  return l;
}

}  // namespace

cudaError_t launch_argmax_rows(const float* logits, const float* noise, float tau, int rows, int V, int32_t* ids, cudaStream_t st) {
  const double bytes = (double)rows * V * 4.0 * (noise ? 2.0 : 1.0) + 4.0 * rows;
  LaunchScope scope(KC_SELECT, 1, bytes, bytes, st);
  return launch_pdl(argmax_rows_kernel, dim3((rows + 7) / 8), dim3(256), 0, st, reinterpret_cast<const float4*>(logits),
                    reinterpret_cast<const float4*>(noise), tau, rows, V / 4, ids);
}

cudaError_t launch_residual_accumulate(const int32_t* ids, int B, int h, int w, const float* codebook, int V, int d, const float* r_prev,
                                       int hp, int wp, float* r_out, int32_t* status, cudaStream_t st) {
  const long total = (long)B * h * w * (d / 4);
  const double bytes = (double)B * h * w * (4.0 + (r_prev ? 3.0 : 2.0) * d * 4.0);
  LaunchScope scope(KC_RESTORE, 1, bytes, bytes, st);
  const long blocks = (total + 255) / 256;
  return launch_pdl(residual_accumulate_kernel, dim3((unsigned)(blocks < 148 * 16 ? blocks : 148 * 16)), dim3(256), 0, st, ids,
                    reinterpret_cast<const float4*>(codebook), reinterpret_cast<const float4*>(r_prev), hp, wp, B, h, w, d / 4, V,
                    reinterpret_cast<float4*>(r_out), status);
}

cudaError_t launch_next_input(const float* r, int B, int h, int w, int d, int h2, int w2, const float* w_in, const float* b_in,
                              const float* pos, int C, float* x_out, cudaStream_t st) {
  const long rows = (long)B * h2 * w2;
  const double bytes = (double)rows * C * (pos ? 8.0 : 4.0) + (double)rows * d * 4.0;
  LaunchScope scope(KC_RESTORE, 1, bytes, bytes, st);
  const dim3 grid((unsigned)((rows + kNextTokens - 1) / kNextTokens));
  switch (d) {
    case 8: return launch_pdl(next_input_kernel<8>, grid, dim3(256), 0, st, r, h, w, h2, w2, w_in, b_in, pos, C, B, x_out);
    case 16: return launch_pdl(next_input_kernel<16>, grid, dim3(256), 0, st, r, h, w, h2, w2, w_in, b_in, pos, C, B, x_out);
    case 32: return launch_pdl(next_input_kernel<32>, grid, dim3(256), 0, st, r, h, w, h2, w2, w_in, b_in, pos, C, B, x_out);
    case 64: return launch_pdl(next_input_kernel<64>, grid, dim3(256), 0, st, r, h, w, h2, w2, w_in, b_in, pos, C, B, x_out);
    default: return cudaErrorInvalidValue;
  }
}

}  // namespace fv

using namespace fv;

namespace {
bool al16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }
fv_status cu(cudaError_t e) { return e == cudaSuccess ? FV_OK : FV_ERR_CUDA; }
}  // namespace

extern "C" {

size_t fv_head_workspace_bytes(int32_t rows, int32_t C, int32_t V) {
  if (rows <= 0 || C <= 0 || V <= 0) return 0;
  return head_layout(rows, C, V, true).total;
}

fv_status fv_argmax_rows(const float* logits_dev, const float* noise_dev, float tau, int32_t rows, int32_t V, int32_t* ids_out_dev,
                         void* stream) {
  if (!logits_dev || !ids_out_dev || rows <= 0 || V <= 0 || (V % 4) || !al16(logits_dev) || (noise_dev && !al16(noise_dev)))
    return FV_ERR_INVALID_ARG;
  return cu(launch_argmax_rows(logits_dev, noise_dev, tau, rows, V, ids_out_dev, static_cast<cudaStream_t>(stream)));
}

fv_status fv_head_tokens(const float* y_dev, int32_t B, int32_t n, int32_t C, const float* mod_head_dev, const void* w_head_dev,
                         const void* b_head_dev, int32_t V, const float* noise_dev, float tau, int32_t* ids_out_dev,
                         float* logits_out_dev, void* workspace_dev, size_t workspace_bytes, int32_t* status_dev, void* stream) {
  if (!y_dev || !mod_head_dev || !w_head_dev || !ids_out_dev || !workspace_dev || B <= 0 || n <= 0) return FV_ERR_INVALID_ARG;
  if (C <= 0 || (C % 8) || C > 2048 || V <= 0 || (V % 8)) return FV_ERR_INVALID_ARG;
  if ((reinterpret_cast<uintptr_t>(workspace_dev) & 255u) || (logits_out_dev && !al16(logits_out_dev))) return FV_ERR_INVALID_ARG;
  const int rows = B * n;
  const HeadLayout l = head_layout(rows, C, V, logits_out_dev == nullptr);
  if (workspace_bytes < l.total) return FV_ERR_CAPACITY;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  char* ws = static_cast<char*>(workspace_dev);
  float* logits = logits_out_dev ? logits_out_dev : reinterpret_cast<float*>(ws + l.logits);
  // the K-split arrival counters must start at zero (the GEMM leaves them zero)
  if (cudaMemsetAsync(ws + l.splitk, 0, gemm_splitk_ticket_bytes(), st) != cudaSuccess) return FV_ERR_CUDA;
  fv_status s = fv_gather_ln(y_dev, nullptr, B, n, n, C, mod_head_dev, mod_head_dev + C, 2 * C, ws + l.a, status_dev, stream);
  if (s != FV_OK) return s;
  s = fv_gemm_bf16(ws + l.a, w_head_dev, b_head_dev, rows, V, C, EPI_F32, logits, nullptr, nullptr, 0, n, status_dev, ws + l.splitk,
                   gemm_splitk_ws_bytes(), stream);
  if (s != FV_OK) return s;
  return cu(launch_argmax_rows(logits, noise_dev, tau, rows, V, ids_out_dev, st));
}

fv_status fv_residual_accumulate(const int32_t* ids_dev, int32_t B, int32_t h, int32_t w, const float* codebook_dev, int32_t V, int32_t d,
                                 const float* r_prev_dev, int32_t hp, int32_t wp, float* r_out_dev, int32_t* status_dev, void* stream) {
  if (!ids_dev || !codebook_dev || !r_out_dev || B <= 0 || h <= 0 || w <= 0 || V <= 0 || d <= 0 || (d % 4)) return FV_ERR_INVALID_ARG;
  if (r_prev_dev && (hp <= 0 || wp <= 0 || r_prev_dev == r_out_dev)) return FV_ERR_INVALID_ARG;
  if (!al16(codebook_dev) || !al16(r_out_dev) || (r_prev_dev && !al16(r_prev_dev))) return FV_ERR_INVALID_ARG;
  return cu(launch_residual_accumulate(ids_dev, B, h, w, codebook_dev, V, d, r_prev_dev, hp, wp, r_out_dev, status_dev,
                                       static_cast<cudaStream_t>(stream)));
}

fv_status fv_next_scale_input(const float* r_dev, int32_t B, int32_t h, int32_t w, int32_t d, int32_t h2, int32_t w2, const float* w_in_dev,
                              const float* b_in_dev, const float* pos_dev, int32_t C, float* x_out_dev, void* stream) {
  if (!r_dev || !w_in_dev || !x_out_dev || B <= 0 || h <= 0 || w <= 0 || h2 <= 0 || w2 <= 0 || C <= 0 || (C % 4)) return FV_ERR_INVALID_ARG;
  if (d != 8 && d != 16 && d != 32 && d != 64) return FV_ERR_UNSUPPORTED;
  if (!al16(w_in_dev)) return FV_ERR_INVALID_ARG;
  return cu(launch_next_input(r_dev, B, h, w, d, h2, w2, w_in_dev, b_in_dev, pos_dev, C, x_out_dev, static_cast<cudaStream_t>(stream)));
}

namespace {
struct GenLayout { size_t status, x, y, r0, r1, head, total; };
GenLayout gen_layout(const fv_config& c, const fv_generator& g) {
  int n_max = 0;
  for (int i = 0; i < c.n_steps; ++i) n_max = n_max > c.h[i] * c.w[i] ? n_max : c.h[i] * c.w[i];
  const size_t rows = (size_t)c.B_max * n_max;
  GenLayout l{};
  size_t off = 0;
  l.status = off; off = align_up(off + 256, 1024);
  l.x = off; off = align_up(off + rows * c.C * 4, 1024);
  l.y = off; off = align_up(off + rows * c.C * 4, 1024);
  l.r0 = off; off = align_up(off + rows * g.d * 4, 1024);
  l.r1 = off; off = align_up(off + rows * g.d * 4, 1024);
  l.head = off; off = align_up(off + head_layout((int)rows, c.C, g.V, true).total, 1024);
  l.total = off;
  return l;
}
}  // namespace

size_t fv_generate_workspace_bytes(const fv_ctx* ctx, const fv_generator* gen) {
  if (!ctx || !gen || gen->V <= 0 || gen->d <= 0) return 0;
  return gen_layout(*ctx_config(ctx), *gen).total;
}

fv_status fv_generate(fv_ctx* ctx, const fv_generator* gen, const float* start_dev, int32_t B, const double* keep_host,
                      const float* const* noise_host, int32_t* ids_out_dev, float* r_out_dev, void* workspace_dev, size_t workspace_bytes,
                      void* stream) {
  if (!ctx || !gen || !start_dev || !keep_host || !ids_out_dev || !r_out_dev || !workspace_dev) return FV_ERR_INVALID_ARG;
  if (!gen->codebook_dev || !gen->w_head_dev || !gen->mod_head_dev || !gen->w_in_dev) return FV_ERR_INVALID_ARG;
  const fv_config& c = *ctx_config(ctx);
  if (B <= 0 || B > c.B_max || (reinterpret_cast<uintptr_t>(workspace_dev) & 1023u)) return FV_ERR_INVALID_ARG;
  if (c.resid_dtype != 0) return FV_ERR_UNSUPPORTED;   // the head reads an fp32 token map
  const GenLayout l = gen_layout(c, *gen);
  if (workspace_bytes < l.total) return FV_ERR_CAPACITY;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  char* ws = static_cast<char*>(workspace_dev);
  // the head GEMM and Eq. 2 report into the context's own status word, which fv_device_status reads
  int32_t* status = ctx_status_word(ctx);
  float* x = reinterpret_cast<float*>(ws + l.x);
  float* y = reinterpret_cast<float*>(ws + l.y);
  float* r[2] = {reinterpret_cast<float*>(ws + l.r0), reinterpret_cast<float*>(ws + l.r1)};
  const size_t head_bytes = l.total - l.head;
  fv_status s = fv_reset(ctx);
  if (s != FV_OK) return s;
  (void)st;
  const int K = c.n_steps;
  size_t id_off = 0;
  for (int k = 0; k < K; ++k) {
    const int h = c.h[k], w = c.w[k], n = h * w;
    const float* xin = k == 0 ? start_dev : x;
    s = fv_var_step(ctx, xin, B, k, keep_host[k], y, nullptr, nullptr, stream);
    if (s != FV_OK) return s;
    int32_t* ids = ids_out_dev + id_off;
    s = fv_head_tokens(y, B, n, c.C, gen->mod_head_dev, gen->w_head_dev, gen->b_head_dev, gen->V,
                       noise_host ? noise_host[k] : nullptr, gen->tau, ids, nullptr, ws + l.head, head_bytes, status, stream);
    if (s != FV_OK) return s;
    float* r_cur = (k + 1 == K) ? r_out_dev : r[k & 1];
    const float* r_prev = k ? r[(k - 1) & 1] : nullptr;
    s = fv_residual_accumulate(ids, B, h, w, gen->codebook_dev, gen->V, gen->d, r_prev, k ? c.h[k - 1] : 0, k ? c.w[k - 1] : 0, r_cur,
                               status, stream);
    if (s != FV_OK) return s;
    if (k + 1 < K) {
      s = fv_next_scale_input(r_cur, B, h, w, gen->d, c.h[k + 1], c.w[k + 1], gen->w_in_dev, gen->b_in_dev,
                              gen->pos_dev ? gen->pos_dev[k + 1] : nullptr, c.C, x, stream);
      if (s != FV_OK) return s;
    }
    id_off += (size_t)B * n;
  }
  return FV_OK;
}

}  // extern "C"
