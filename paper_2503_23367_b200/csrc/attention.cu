// Flash-style attention of the kept queries over the KV cache (Sec. 3.1: the KV cache of previous
// scale steps; Sec. 3.3: at pruned steps the cache holds only pivotal keys, and FastVAR never reads
// the attention map, so a fused kernel applies).  Within a scale step there is no mask: a query sees
// every cached key of the earlier scales and all keys appended by its own step.
//
// Work item = 256 queries (two tiles of 128) of one head of one image; keys are consumed in tiles of 128.
// The kept-row counts of the pruned steps give item counts that fit the GPU badly (64, 80, 128 or 208 items
// on 148 SMs, the last item of a head often a single, part-filled tile), so the (item, key tile) units are
// laid out on one line (a weight per item kind; both kinds cost the same per key tile as measured) and the line
// is cut into equal pieces, one per CTA (one CTA per SM), when that beats one whole item per CTA.  A CTA walks its piece as segments: a range of key tiles of
// one item.  A segment that covers all key tiles of its item writes the output itself; otherwise it leaves
// its unnormalised partial (O, running maximum, row sum) in scratch, and the last part of an item to arrive
// (arrival counter) merges the parts IN KEY ORDER, so the result does not depend on arrival order.
// Without scratch the kernel runs one whole item per CTA.
//
// The two query tiles of a segment take turns on the tensor core: while the softmax warps of one tile work
// on its scores, the MMAs of the other tile run.
//   warp 8   : TMA producer (both Q tiles per segment; K tiles [128 keys x hd]; V^T tiles [hd x 128 keys]).
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
// Every wait is bounded (status word + normal unwind on expiry); a thread whose wait expired skips the
// rest of its work but still takes part in every CTA-level barrier.
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
  // one partial of a segment in scratch: (maximum, row sum) [2 tiles][128 rows], then O [2 tiles][HD/4][128 rows] float4
  static constexpr size_t kPartMlBytes = 2 * QT * sizeof(float2);
  static constexpr size_t kPartBytes = kPartMlBytes + (size_t)2 * QT * HD * sizeof(float);
};

// Scratch of a split launch: arrival counters (one per item, zero between launches), then two partial slots
// per CTA -- slot 0 for a segment that continues an item begun by an earlier CTA, slot 1 for a segment that
// begins an item and leaves its end to later CTAs.  A CTA has at most one segment of either kind.
constexpr int kAttnMaxItems = 16384;
constexpr int kAttnMaxCtas = 160;
constexpr size_t kAttnTicketBytes = (size_t)kAttnMaxItems * sizeof(unsigned int);
// Cost of a key tile for an item of two query tiles / of one.  Measured equal: with one tile there is nothing to
// overlap the S -> softmax -> P V -> next S chain with, so the tile takes as long as the pair's two.
constexpr int kWeightPair = 1, kWeightSingle = 1;

struct AttnDev {
  __nv_bfloat16* out;
  int rows, C, kv_len, kv_capacity;
  float scale_log2;  // log2(e) / sqrt(hd)
  int32_t* status;
  int B, H, P, single;       // images; heads; items per (image, head); 1 if the last item of a head has one query tile
  int T;                     // key tiles
  int split;                 // 0: CTA c runs item c whole; 1: the cost line is cut into gridDim.x pieces
  int total_cost, cost_group, cost_full;   // whole line; one (image, head); its two-tile items (all below 2^31 / 3)
  unsigned int* tickets;
  char* parts;
};

// First (item, key tile) unit, as item * T + tile, at cost position pos of the line.
__device__ __forceinline__ int unit_at(const AttnDev& p, int pos) {
  const int g = pos / p.cost_group, r = pos - g * p.cost_group;
  int it, j;
  if (r < p.cost_full) { it = r / (kWeightPair * p.T); j = (r - it * (kWeightPair * p.T)) / kWeightPair; }
  else { it = p.P - 1; j = (r - p.cost_full) / kWeightSingle; }
  return (g * p.P + it) * p.T + j;
}
// First unit of CTA c's piece (c == gridDim.x: one past the last unit).
__device__ __forceinline__ int piece_begin(const AttnDev& p, int c, int nctas, int units) {
  if (c >= nctas) return units;
  if (!p.split) return c * p.T;
  return unit_at(p, (int)(((long long)p.total_cost * c) / nctas));
}

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

// Where a segment of CTA `c` that is part of item `item` (units [item*T, (item+1)*T)) stands among the item's
// parts: the first and the number of the CTAs whose pieces overlap the item (pieces are never empty).
__device__ __noinline__ void item_parts(const AttnDev& p, int c, int nctas, int units, int item, int* c_first, int* nparts) {
  const int u0 = item * p.T, u1 = u0 + p.T;
  int a = c;
  while (a > 0 && piece_begin(p, a, nctas, units) > u0) --a;         // piece a holds unit u0
  int b = c;
  while (b + 1 < nctas && piece_begin(p, b + 1, nctas, units) < u1) ++b;   // piece b holds unit u1 - 1
  *c_first = a;
  *nparts = b - a + 1;
}

// Online softmax of one query row over the key tiles [ja, jb) of a segment: scores out of TMEM, probabilities
// back into it, the O accumulator rescaled in place when the running maximum moves.  Returns false if a wait
// expired.  `tiles` counts the score tiles this thread's query tile has consumed (the phase of the barriers).
// Out of line so that the loop keeps the whole register file to itself (a thread holds a score row of 128 floats).
template <int HD>
__device__ __noinline__ bool softmax_key_tiles(const AttnDev& p, int ja, int jb, uint32_t s_addr, uint32_t o_addr, uint64_t* s_full_t,
                                               uint64_t* p_full_t, uint64_t* o_done_t, uint32_t& tiles, float& m_out, float& l_out) {
  float m_run = -INFINITY, l_run = 0.f;
  uint32_t sc_cnt = tiles;
  const float scale_log2 = p.scale_log2;
  for (int j = ja; j < jb; ++j, ++sc_cnt) {
    if (!mbar_wait(s_full_t, sc_cnt & 1)) { report(p.status, DEV_TIMEOUT_SOFTMAX); tiles = sc_cnt; return false; }
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
    const float mx = fmaxf(fmaxf(mx0, mx1), fmaxf(mx2, mx3)) * scale_log2;
    // Raise the running maximum only when it would grow by more than the threshold: probabilities
    // may then exceed 1 (by at most 2^threshold), which fp32 sums and bf16 P hold without loss.
    float alpha = 1.f;
    if (mx > m_run + kRescaleThreshold) {
      alpha = fast_exp2(m_run - mx);  // 0 on the first tile (m_run = -inf)
      m_run = mx;
    }
    // S_t of tile j was issued after P V of tile j-1, so O_t is at rest here.
    if (j > ja && __any_sync(0xffffffffu, alpha != 1.f)) {
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
    const float rs = tile_exp_store(sc, s_addr, scale_log2, m_run);
    l_run = fmaf(l_run, alpha, rs);
    tmem_wait_st();
    tc_fence_before();
    mbar_arrive(p_full_t);
  }
  tiles = sc_cnt;
  m_out = m_run; l_out = l_run;
  if (!mbar_wait(o_done_t, (sc_cnt - 1) & 1)) { report(p.status, DEV_TIMEOUT_SOFTMAX); return false; }
  tc_fence_after();
  return true;
}

// End of a segment for one softmax thread (query row r of tile t): O_t leaves tensor memory -- as the normalised
// bf16 output when the segment covered every key tile of its item, else as this part's unnormalised partial in
// scratch, after which the last part of the item to arrive merges all of them in key order.  Kept out of line so
// that its registers do not weigh on the key loop.
template <int HD>
__device__ __noinline__ void finish_segment(const AttnDev& p, int u0, int u_hi, int t, int r, uint32_t o_addr, float m_run, float l_run,
                                            bool ok, uint64_t* o_free_t, volatile int* s_info) {
  using Cfg = AttnCfg<HD>;
  const int cta = blockIdx.x, nctas = gridDim.x;
  const int item = u0 / p.T, ja = u0 - item * p.T;
  const int jb = (p.T - ja) < (u_hi - u0) ? p.T : ja + (u_hi - u0);
  const int g = item / p.P, ip = item - g * p.P;
  const int img = g / p.H, head = g - img * p.H;
  const int q0 = ip * (2 * QT);
  const bool active = t < ((p.rows - q0 > QT) ? 2 : 1);
  const bool whole = jb - ja == p.T;
  const int row = q0 + t * QT + r;
  if (active && ok) {
    if (whole) {
      const float inv_l = 1.f / l_run;
      __nv_bfloat16* dst = p.out + ((size_t)img * p.rows + row) * p.C + head * HD;
#pragma unroll
      for (int c = 0; c < HD / 32; ++c) {
        uint32_t o[32];
        tmem_ld32(o_addr + c * 32, o);
        tmem_wait_ld();
        if (row < p.rows) {
#pragma unroll
          for (int gq = 0; gq < 4; ++gq) {
            uint4 v;
            v.x = pack_bf16x2(__uint_as_float(o[8 * gq + 0]) * inv_l, __uint_as_float(o[8 * gq + 1]) * inv_l);
            v.y = pack_bf16x2(__uint_as_float(o[8 * gq + 2]) * inv_l, __uint_as_float(o[8 * gq + 3]) * inv_l);
            v.z = pack_bf16x2(__uint_as_float(o[8 * gq + 4]) * inv_l, __uint_as_float(o[8 * gq + 5]) * inv_l);
            v.w = pack_bf16x2(__uint_as_float(o[8 * gq + 6]) * inv_l, __uint_as_float(o[8 * gq + 7]) * inv_l);
            reinterpret_cast<uint4*>(dst + c * 32)[gq] = v;
          }
        }
      }
    } else {
      // this part of the item: (running maximum, row sum) and the unnormalised O, for the merge
      char* slot = p.parts + ((size_t)cta * 2 + (ja == 0 ? 1 : 0)) * Cfg::kPartBytes;
      reinterpret_cast<float2*>(slot)[t * QT + r] = make_float2(m_run, l_run);
      float4* od = reinterpret_cast<float4*>(slot + Cfg::kPartMlBytes) + (size_t)t * (HD / 4) * QT + r;
#pragma unroll
      for (int c = 0; c < HD / 32; ++c) {
        uint32_t o[32];
        tmem_ld32(o_addr + c * 32, o);
        tmem_wait_ld();
#pragma unroll
        for (int gq = 0; gq < 8; ++gq)
          __stcg(od + (size_t)(c * 8 + gq) * QT, make_float4(__uint_as_float(o[4 * gq]), __uint_as_float(o[4 * gq + 1]),
                                                              __uint_as_float(o[4 * gq + 2]), __uint_as_float(o[4 * gq + 3])));
      }
    }
  }
  // O_t of this segment has left TMEM (or the thread has given up): the next segment that uses the tile may overwrite it
  tc_fence_before();
  if (active) mbar_arrive(o_free_t);
  if (whole) return;
  // ---- the last part of the item to arrive merges all of them, in key order
  __threadfence();
  asm volatile("bar.sync 1, 256;" ::: "memory");
  if (threadIdx.x == 0) {
    int c_first, nparts;
    item_parts(p, cta, nctas, p.P * p.H * p.B * p.T, item, &c_first, &nparts);
    const unsigned int prev = atomicAdd(p.tickets + item, 1u);
    const int last = prev == (unsigned int)(nparts - 1);
    if (last) p.tickets[item] = 0u;     // every part has arrived: the counter is ready for the next launch
    s_info[0] = c_first; s_info[1] = nparts; s_info[2] = last;
  }
  asm volatile("bar.sync 1, 256;" ::: "memory");
  const int c_first = s_info[0], nparts = s_info[1], last = s_info[2];
  asm volatile("bar.sync 1, 256;" ::: "memory");   // s_info consumed before a later segment rewrites it
  if (!last || !active || row >= p.rows) return;
  __threadfence();
  // part q of the item was left by CTA c_first + q: the first in its slot 1, the others in slot 0
  auto part_slot = [&](int q) { return p.parts + ((size_t)(c_first + q) * 2 + (q == 0 ? 1 : 0)) * Cfg::kPartBytes; };
  float m_star = -INFINITY;
  for (int q = 0; q < nparts; ++q) m_star = fmaxf(m_star, __ldcg(reinterpret_cast<const float2*>(part_slot(q)) + t * QT + r).x);
  float l_star = 0.f;
  for (int q = 0; q < nparts; ++q) {
    const float2 ml = __ldcg(reinterpret_cast<const float2*>(part_slot(q)) + t * QT + r);
    l_star = fmaf(ml.y, fast_exp2(ml.x - m_star), l_star);
  }
  const float inv_l = 1.f / l_star;
  __nv_bfloat16* dst = p.out + ((size_t)img * p.rows + row) * p.C + head * HD;
  // 32 output channels at a time: the eight float4 of a part are requested together (the loop is bound by the
  // latency of these loads, not by their bytes), parts added in key order
#pragma unroll 1
  for (int c32 = 0; c32 < HD / 32; ++c32) {
    float4 acc[8];
#pragma unroll
    for (int i = 0; i < 8; ++i) acc[i] = make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll 1
    for (int q = 0; q < nparts; ++q) {
      const char* slot = part_slot(q);
      const float4* os = reinterpret_cast<const float4*>(slot + Cfg::kPartMlBytes) + ((size_t)t * (HD / 4) + c32 * 8) * QT + r;
      float4 v[8];
#pragma unroll
      for (int i = 0; i < 8; ++i) v[i] = __ldcg(os + (size_t)i * QT);
      const float wq = fast_exp2(__ldcg(reinterpret_cast<const float2*>(slot) + t * QT + r).x - m_star) * inv_l;
#pragma unroll
      for (int i = 0; i < 8; ++i) {
        acc[i].x = fmaf(v[i].x, wq, acc[i].x); acc[i].y = fmaf(v[i].y, wq, acc[i].y);
        acc[i].z = fmaf(v[i].z, wq, acc[i].z); acc[i].w = fmaf(v[i].w, wq, acc[i].w);
      }
    }
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      uint4 v;
      v.x = pack_bf16x2(acc[2 * i].x, acc[2 * i].y); v.y = pack_bf16x2(acc[2 * i].z, acc[2 * i].w);
      v.z = pack_bf16x2(acc[2 * i + 1].x, acc[2 * i + 1].y); v.w = pack_bf16x2(acc[2 * i + 1].z, acc[2 * i + 1].w);
      reinterpret_cast<uint4*>(dst + c32 * 32)[i] = v;
    }
  }
}

template <int HD>
__global__ void __launch_bounds__(kAttnThreads, 1)
attention_kernel(const __grid_constant__ CUtensorMap tmQ, const __grid_constant__ CUtensorMap tmK,
                 const __grid_constant__ CUtensorMap tmV, const __grid_constant__ AttnDev p) {
  using Cfg = AttnCfg<HD>;
  constexpr int NS = Cfg::kStages;
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  uint8_t* q_s = smem;                          // two query tiles
  uint8_t* k_s = q_s + 2 * Cfg::kQBytes;
  uint8_t* v_s = k_s + NS * Cfg::kKBytes;
  uint64_t* bars = reinterpret_cast<uint64_t*>(v_s + NS * Cfg::kVBytes);
  uint64_t* q_full = bars;
  uint64_t* q_empty = bars + 1;      // every Q K^T of the segment has been executed: the query tiles may be replaced
  uint64_t* k_full = bars + 2;
  uint64_t* k_empty = k_full + NS;
  uint64_t* v_full = k_empty + NS;
  uint64_t* v_empty = v_full + NS;
  uint64_t* s_full = v_empty + NS;   // [2] scores of query tile t are in TMEM
  uint64_t* p_full = s_full + 2;     // [2] probabilities of query tile t are in TMEM (128 arrivals)
  uint64_t* o_done = p_full + 2;     // [2] the latest P V of query tile t has completed
  uint64_t* o_free = o_done + 2;     // [2] the segment's O of query tile t has been read out of TMEM (128 arrivals)
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(o_free + 2);
  volatile int* s_info = reinterpret_cast<volatile int*>(tmem_slot + 1);   // [0] first CTA of the item, [1] parts, [2] last arriver

  pdl_trigger();
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int cta = blockIdx.x, nctas = gridDim.x;
  const int units = p.P * p.H * p.B * p.T;
  const int u_lo = piece_begin(p, cta, nctas, units), u_hi = piece_begin(p, cta + 1, nctas, units);

  if (threadIdx.x == 0) {
    mbar_init(q_full, 1); mbar_init(q_empty, 1);
    for (int s = 0; s < NS; ++s) { mbar_init(&k_full[s], 1); mbar_init(&k_empty[s], 1); mbar_init(&v_full[s], 1); mbar_init(&v_empty[s], 1); }
    for (int t = 0; t < 2; ++t) { mbar_init(&s_full[t], 1); mbar_init(&p_full[t], QT); mbar_init(&o_done[t], 1); mbar_init(&o_free[t], QT); }
    mbar_fence_init();
    tma_prefetch_desc(&tmQ); tma_prefetch_desc(&tmK); tma_prefetch_desc(&tmV);
  }
  if (warp == 9) { tmem_alloc(tmem_slot, Cfg::kTmemCols); tmem_relinquish(); }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;
  pdl_wait();  // set-up above overlaps the previous kernel; Q / K / V, the scratch and the output are touched only from here

  // Segment seg of this CTA: key tiles [ja, jb) of `item`; every role walks the same list.
  struct Seg { int item, ja, jb, q0, head, img, ntiles; };
  auto segment_at = [&](int u) {
    Seg sg;
    sg.item = u / p.T;
    sg.ja = u - sg.item * p.T;
    const int left = u_hi - u;
    sg.jb = (p.T - sg.ja) < left ? p.T : sg.ja + left;
    const int g = sg.item / p.P, ip = sg.item - g * p.P;
    sg.img = g / p.H; sg.head = g - sg.img * p.H;
    sg.q0 = ip * (2 * QT);
    sg.ntiles = (p.rows - sg.q0 > QT) ? 2 : 1;
    return sg;
  };

  // A softmax thread holds a whole score row (128 fp32) in registers, so the register file is re-divided
  // between the warpgroups: 2 x 128 x 208 + 128 x 88 = 384 x 168, what the CTA was launched with (a larger request would
  // wait forever); 88 rather than fewer for the producer / MMA warps measured 3 % faster here.
  if (warp >= 8) {
   asm volatile("setmaxnreg.dec.sync.aligned.u32 88;");
   if (warp == 8) {
    if (lane == 0) {
      uint32_t kt = 0;      // key tiles loaded so far: ring position of the K and V^T stages
      int seg = 0;
      bool ok = true;
      for (int u = u_lo; ok && u < u_hi; ++seg) {
        const Seg sg = segment_at(u);
        u += sg.jb - sg.ja;
        for (int j = sg.ja; j < sg.jb; ++j, ++kt) {
          const int s = kt % NS;
          const uint32_t ph = (kt / NS) & 1;
          if (!mbar_wait(&k_empty[s], ph ^ 1)) { report(p.status, DEV_TIMEOUT_TMA); ok = false; break; }
          mbar_expect_tx(&k_full[s], Cfg::kKBytes);
          for (int a = 0; a < HD / 64; ++a)
            tma_load_2d(k_s + s * Cfg::kKBytes + a * (KT * 128), &tmK, sg.head * HD + a * 64, sg.img * p.kv_capacity + j * KT, &k_full[s]);
          if (j == sg.ja) {   // the segment's query tiles, once the previous segment's Q K^T have all run
            if (seg > 0 && !mbar_wait(q_empty, (seg - 1) & 1)) { report(p.status, DEV_TIMEOUT_TMA); ok = false; break; }
            mbar_expect_tx(q_full, sg.ntiles * Cfg::kQBytes);
            for (int t = 0; t < sg.ntiles; ++t)
              for (int a = 0; a < HD / 64; ++a)
                tma_load_2d(q_s + t * Cfg::kQBytes + a * (QT * 128), &tmQ, sg.head * HD + a * 64, sg.img * p.rows + sg.q0 + t * QT, q_full);
          }
          if (!mbar_wait(&v_empty[s], ph ^ 1)) { report(p.status, DEV_TIMEOUT_TMA); ok = false; break; }
          mbar_expect_tx(&v_full[s], Cfg::kVBytes);
          for (int a = 0; a < KT / 64; ++a)
            tma_load_2d(v_s + s * Cfg::kVBytes + a * (HD * 128), &tmV, j * KT + a * 64, sg.img * p.C + sg.head * HD, &v_full[s]);
        }
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
      uint32_t kt = 0;             // key tiles consumed so far (ring position)
      uint32_t pc[2] = {0, 0};     // probability tiles consumed per query tile (phase of p_full)
      uint32_t oc[2] = {0, 0};     // segments so far that used query tile t (phase of o_free)
      int seg = 0;
      bool ok = true;
      for (int u = u_lo; ok && u < u_hi; ++seg) {
        const Seg sg = segment_at(u);
        const int Tseg = sg.jb - sg.ja;
        u += Tseg;
        if (!mbar_wait(q_full, seg & 1) || !mbar_wait(&k_full[kt % NS], (kt / NS) & 1)) { report(p.status, DEV_TIMEOUT_MMA); ok = false; break; }
        tc_fence_after();
        for (int t = 0; t < sg.ntiles; ++t) issue_qk(t, kt % NS);
        umma_commit(&k_empty[kt % NS]);
        if (Tseg == 1) umma_commit(q_empty);
        for (int jj = 0; ok && jj < Tseg; ++jj) {
          const uint32_t cur = kt + jj, nxt = cur + 1;
          const int s = cur % NS, sn = nxt % NS;
          const bool more = jj + 1 < Tseg;
          if (!mbar_wait(&v_full[s], (cur / NS) & 1) || (more && !mbar_wait(&k_full[sn], (nxt / NS) & 1))) {
            report(p.status, DEV_TIMEOUT_MMA); ok = false; break;
          }
          const uint32_t v_addr = smem_u32(v_s + s * Cfg::kVBytes);
          for (int t = 0; t < sg.ntiles; ++t) {
            // the first P V of a segment overwrites O_t: the O of the last segment that used tile t must have been
            // read out (its softmax threads arrive once per segment in which the tile is used, so neither side can
            // get a whole phase ahead of the other)
            if (jj == 0 && oc[t] > 0 && !mbar_wait(&o_free[t], (oc[t] - 1) & 1)) { report(p.status, DEV_TIMEOUT_MMA); ok = false; break; }
            if (!mbar_wait(&p_full[t], pc[t] & 1)) { report(p.status, DEV_TIMEOUT_MMA); ok = false; break; }
            ++pc[t];
            tc_fence_after();
            const uint32_t p_tmem = tmem_base + t * KT;              // P_t over the first 64 columns of S_t
            const uint32_t o_tmem = tmem_base + 256 + t * 128;
#pragma unroll
            for (int kk = 0; kk < KT / 16; ++kk) {
              const uint32_t b_off = (kk >> 2) * (HD * 128) + (kk & 3) * 32;
              umma_bf16_ts(o_tmem, p_tmem + kk * 8, umma_desc_k_sw128(v_addr + b_off), idesc_pv, (jj | kk) != 0);
            }
            umma_commit(&o_done[t]);
            if (more) issue_qk(t, sn);
          }
          if (!ok) break;
          umma_commit(&v_empty[s]);
          if (more) umma_commit(&k_empty[sn]);
          if (more && jj + 2 == Tseg) umma_commit(q_empty);   // the segment's last Q K^T have been issued
        }
        kt += Tseg;
        for (int t = 0; t < sg.ntiles; ++t) ++oc[t];
      }
    }
   }
  } else {
    asm volatile("setmaxnreg.inc.sync.aligned.u32 208;");
    // ---- softmax + output: thread = one query row of tile t ----
    const int t = warp >> 2;
    const int quarter = warp & 3;                 // the TMEM lanes this warp may touch
    const int r = quarter * 32 + lane;
    const uint32_t lane_off = uint32_t(quarter * 32) << 16;
    const uint32_t s_addr = tmem_base + lane_off + t * KT;
    const uint32_t o_addr = tmem_base + lane_off + 256 + t * 128;
    uint32_t sc_cnt = 0;     // score tiles consumed by this thread's query tile (phase of s_full / o_done)
    bool ok = true;
    for (int u = u_lo; u < u_hi;) {
      const int u0 = u;
      const Seg sg = segment_at(u);
      u += sg.jb - sg.ja;
      const bool active = t < sg.ntiles;
      float m_run = -INFINITY, l_run = 0.f;
      if (active && ok) ok = softmax_key_tiles<HD>(p, sg.ja, sg.jb, s_addr, o_addr, &s_full[t], &p_full[t], &o_done[t], sc_cnt, m_run, l_run);
      finish_segment<HD>(p, u0, u_hi, t, r, o_addr, m_run, l_run, ok, &o_free[t], s_info);
    }
  }
  tc_fence_before();
  __syncthreads();
  if (warp == 9) {
    __syncwarp();
    tmem_dealloc(tmem_base, Cfg::kTmemCols);
  }
}

// ---- One whole work item per CTA: grid (query blocks, heads, images).  The launcher takes this kernel whenever it does
// not cut the work into pieces: it is the kernel above without the segment bookkeeping, and its leaner loops hand
// the tiles between the softmax warpgroups and the MMA thread measurably faster (15 % per key tile).
struct WholeDev {
  __nv_bfloat16* out;
  int rows, C, kv_len, kv_capacity;
  float scale_log2;  // log2(e) / sqrt(hd)
  int32_t* status;
};

template <int HD>
__global__ void __launch_bounds__(kAttnThreads, 1)
attention_whole_kernel(const __grid_constant__ CUtensorMap tmQ, const __grid_constant__ CUtensorMap tmK,
                 const __grid_constant__ CUtensorMap tmV, const WholeDev p) {
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

int g_attn_sms = 148;
int g_attn_force_ctas = 0;

template <int HD> fv_status launch_hd(const AttnArgs& a, cudaStream_t st) {
  alignas(64) CUtensorMap tmQ, tmK, tmV;
  if (!make_tmap_rows(&tmQ, a.q, (uint64_t)a.B * a.rows, a.C, QT)) return FV_ERR_CUDA;
  if (!make_tmap_rows(&tmK, a.k, (uint64_t)a.B * a.kv_capacity, a.C, KT)) return FV_ERR_CUDA;
  if (!make_tmap_rows(&tmV, a.vt, (uint64_t)a.B * a.C, a.kv_capacity, HD)) return FV_ERR_CUDA;
  AttnDev p{};
  p.out = static_cast<__nv_bfloat16*>(a.out);
  p.rows = a.rows; p.C = a.C; p.kv_len = a.kv_len; p.kv_capacity = a.kv_capacity;
  p.scale_log2 = 1.4426950408889634f / sqrtf((float)HD);
  p.status = a.status;
  p.B = a.B; p.H = a.H;
  p.P = (a.rows + 2 * QT - 1) / (2 * QT);
  p.single = (a.rows - (p.P - 1) * 2 * QT) <= QT ? 1 : 0;
  p.T = (a.kv_len + KT - 1) / KT;
  const long long items = (long long)p.P * a.H * a.B;
  if (items * p.T * kWeightPair >= (1ll << 31)) return FV_ERR_UNSUPPORTED;
  p.cost_full = kWeightPair * p.T * (p.P - p.single);
  p.cost_group = p.cost_full + kWeightSingle * p.T * p.single;
  p.total_cost = p.cost_group * a.H * a.B;
  long long ctas = items;
  p.split = 0;
  if (a.workspace && items <= kAttnMaxItems && g_attn_force_ctas >= 0) {
    // One piece per SM when that beats whole items: a launch of whole items takes ceil(items / SMs) rounds of T key
    // tiles; the pieces take items * T / SMs key tiles plus what the cuts cost (query tiles loaded again, the
    // partials written and merged: about kSplitOverheadTiles key tiles, measured; short key ranges lose).  A forced
    // piece count always splits.
    constexpr long long kSplitOverheadTiles = 10;
    long long g = g_attn_force_ctas > 0 ? g_attn_force_ctas : g_attn_sms;
    if (g > kAttnMaxCtas) g = kAttnMaxCtas;
    const long long most = p.total_cost / (2 * kWeightPair);   // every piece at least two key tiles long
    if (g > most) g = most;
    const long long rounds = (items + g_attn_sms - 1) / g_attn_sms;
    // (the kernel that walks pieces also takes about 15 % longer per key tile than the one that runs whole items)
    const bool pays = g >= 1 && p.T >= 16 && 115 * (items * p.T / g + kSplitOverheadTiles) < 100 * rounds * p.T;
    if (g >= 1 && (pays || g_attn_force_ctas > 0)) {
      p.split = 1;
      ctas = g;
      p.tickets = static_cast<unsigned int*>(a.workspace);
      p.parts = static_cast<char*>(a.workspace) + kAttnTicketBytes;
    }
  }
  LaunchScope scope(KC_ATTENTION, 1, 4.0 * a.B * (double)a.rows * a.kv_len * a.C,
                    2.0 * a.B * a.C * (2.0 * a.rows + 2.0 * a.kv_len), st);  // Q in, O out, K and V^T once
  if (!p.split) {
    WholeDev w;
    w.out = p.out; w.rows = p.rows; w.C = p.C; w.kv_len = p.kv_len; w.kv_capacity = p.kv_capacity; w.scale_log2 = p.scale_log2; w.status = p.status;
    dim3 grid3((a.rows + 2 * QT - 1) / (2 * QT), a.H, a.B);
    return launch_pdl(attention_whole_kernel<HD>, grid3, dim3(kAttnThreads), AttnCfg<HD>::kSmemBytes, st, tmQ, tmK, tmV, w) == cudaSuccess
               ? FV_OK : FV_ERR_CUDA;
  }
  dim3 grid((unsigned)ctas);
  return launch_pdl(attention_kernel<HD>, grid, dim3(kAttnThreads), AttnCfg<HD>::kSmemBytes, st, tmQ, tmK, tmV, p) == cudaSuccess
             ? FV_OK : FV_ERR_CUDA;
}

}  // namespace

size_t attention_ws_bytes() { return kAttnTicketBytes + (size_t)kAttnMaxCtas * 2 * AttnCfg<128>::kPartBytes; }
size_t attention_ws_ticket_bytes() { return kAttnTicketBytes; }
void attention_force_ctas(int ctas) { g_attn_force_ctas = ctas; }

cudaError_t attention_init() {
  int dev = 0;
  cudaError_t e = cudaGetDevice(&dev);
  if (e == cudaSuccess) e = cudaDeviceGetAttribute(&g_attn_sms, cudaDevAttrMultiProcessorCount, dev);
  if (e != cudaSuccess) return e;
  e = cudaFuncSetAttribute(attention_kernel<64>, cudaFuncAttributeMaxDynamicSharedMemorySize, AttnCfg<64>::kSmemBytes);
  if (e == cudaSuccess) e = cudaFuncSetAttribute(attention_whole_kernel<64>, cudaFuncAttributeMaxDynamicSharedMemorySize, AttnCfg<64>::kSmemBytes);
  if (e == cudaSuccess) e = cudaFuncSetAttribute(attention_whole_kernel<128>, cudaFuncAttributeMaxDynamicSharedMemorySize, AttnCfg<128>::kSmemBytes);
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
