"""CPU oracle for FastVAR's cached token pruning (test infrastructure, NOT a product path).

A plain, slow, double-precision restatement of what the pruned next-scale-prediction step
computes, written from the paper: Pivotal Token Selection (Eq. 4, Eq. 5, Algorithm 1, first
routine), Cached Token Restoration (Eq. 6, Algorithm 1, second routine), the rule that the pair
wraps every attention and FFN layer at the pruned steps (Sec. 3.3 "Implementation", Fig. 3b),
the cache written at step K-N (Sec. 3.3 "Overview") and the reduced KV cache (Sec. 3.3, end of
the PTS paragraph).  Only tests, the smoke check and the benchmark's CPU-baseline leg may import
this file; it shares no code with the CUDA path and imports nothing from it.

Everything is numpy float64.  There is no blocking, fusion or reordering: each function is the
definition written out, with numpy's matmul / sort as library steps.

Readings taken where the paper is silent or inconsistent (each is also listed in the design notes):
  * score = SUM of squared deviations (Algorithm 1), not its square root (Eq. 5): same ranking.
  * the scored tensor is the residual stream entering the sublayer, before normalisation.
  * kept count k = ceil(keep_ratio * h*w) (keep ratio = 1 - the paper's pruning ratio).
  * ties in the score go to the LOWEST token index; the kept set is emitted in ascending index
    order (the set, not the order, is what the method defines: no later step depends on order).
  * interpolate(.) of Eq. 6 = nearest neighbour, src = floor(dst * in / out) per axis.
  * the cache holds the sublayer's branch output before gate and residual, one per wrapped sublayer,
    taken at the last unpruned step and never refreshed.
  * at a pruned step only the kept rows' K/V are appended to the KV cache.
  * the transformer block (not specified by the paper): pre-LayerNorm without affine (eps 1e-6),
    AdaLN modulation a = LN(x)*(1+sigma)+beta and gate x += gamma*y, tanh-GELU MLP, softmax scale
    1/sqrt(head_dim), biases on qkv / out / fc1 / fc2, optional cross-attention to text with plain
    LN, no biases and no gate.

Backbone extras (all off by default; the paper names none of them, they belong to the backbones it prunes,
so each is a reading stated here and pinned on its own):
  * `interp_mode="bilinear"`: interpolate(.) of Eq. 6 as a bilinear blend with half-pixel centres
    (source coordinate (dst + 0.5) * in / out - 0.5, clamped), the convention of library resizing routines.
    `interp_mode="bicubic"`: separable cubic convolution (Keys' kernel, a = -0.75) over 4 x 4 cached tokens at
    the same half-pixel coordinates, tap indices clamped to the map.
  * `qk_scale` [L, H]: cosine attention -- in the self-attention sublayer every head's query and key are
    divided by their Euclidean norm (floored at 1e-12) and the query is multiplied by the head's scale.
  * `rope_base`: two-dimensional rotary position embedding in the self-attention sublayer.  A token at
    row y, column x of the (h, w) map of its scale sits at (y * h_K / h, x * w_K / w) in the frame of the
    last scale, so that tokens of different scales covering the same image region get the same phase.  Of a
    head's hd channels the first half is rotated by the row coordinate, the second by the column coordinate;
    channel pairs (2j, 2j+1) of a half turn by coordinate * base^(-j / (hd/4)).  The position is that of the
    token's ORIGINAL slot in the map: at a pruned step row j of the compact tensor is token idx[j], and it is
    idx[j] that is rotated by -- the one place where pruning reaches into the attention arithmetic.
    Order: normalise, then rotate (a rotation keeps the norm).  Values are not touched.

Granularity.  The paper wraps EVERY attention / FFN layer with the selection / restoration pair
(Sec. 3.3 "Implementation"); that is `granularity="sublayer"`, the default.  `granularity="step"` is the
coarser variant in which the pair wraps the whole stack of blocks of a scale step: one selection on the
step's input token map, all blocks run on the kept rows only (their residual stream stays compact), and
one restoration from the cached OUTPUT token map of step K-N.  It is a different approximation (its
unkept tokens take the previous scale's output, interpolated, instead of accumulating cached layer
outputs); it is not the paper's configuration and is pinned only by its own invariants.

Parity pins: every function here is pinned by tests/test_oracle_pins.py (closed forms, brute force,
invariants, library special cases).  The paper prints no worked example of a whole step, so
`VarOracle.var_step` is pinned by what the method fixes: the unpruned schedule equals a library block-causal
forward over the whole sequence; a pruned step whose sublayers all keep one given set equals that library
forward over [earlier scales ; kept tokens] on the kept rows and the gated sum of the cached sublayer outputs
on the others; a free-running pruned step replays from its trace with a brute-force ranking of the current
stream at every sublayer; keep_ratio -> 1 equals the unpruned forward; KV length, order and image invariance.
"""
from __future__ import annotations

import math
from typing import Dict, List, Optional, Sequence

import numpy as np

F64 = np.float64


# ----------------------------------------------------------------------------------------------
# Pivotal Token Selection  (Sec. 3.3, Eq. 4-5, Algorithm 1 first routine)
# ----------------------------------------------------------------------------------------------

def kept_count(keep_ratio: float, h: int, w: int) -> int:
    """k = ceil(keep_ratio * h * w), clamped to [1, h*w].  The small epsilon keeps products
    that are integers in exact arithmetic (0.6 * 1600 = 960) from rounding up."""
    n = h * w
    k = int(math.ceil(float(keep_ratio) * n - 1e-9))
    return min(n, max(1, k))


def pts_mean(x: np.ndarray) -> np.ndarray:
    """Eq. 4: global average pool over the h*w tokens of each image.  x [B,n,C] -> [B,C]."""
    x = np.asarray(x, dtype=F64)
    return x.sum(axis=1) / x.shape[1]


def pts_score(x: np.ndarray) -> np.ndarray:
    """Eq. 5 in the squared form of Algorithm 1: s[b,n] = sum_c (x[b,n,c] - mean[b,c])^2."""
    x = np.asarray(x, dtype=F64)
    d = x - pts_mean(x)[:, None, :]
    return (d * d).sum(axis=2)


def pts_topk(score: np.ndarray, k: int) -> np.ndarray:
    """Index set I: the k largest scores per image (stable descending sort, so equal scores keep
    the lower index first), then emitted in ascending index order.  score [B,n] -> int64 [B,k]."""
    score = np.asarray(score)
    B, n = score.shape
    out = np.empty((B, k), dtype=np.int64)
    for b in range(B):
        order = np.argsort(-score[b], kind="stable")   # stable: ties -> lowest index first
        out[b] = np.sort(order[:k])
    return out


def inverse_map(idx: np.ndarray, n: int) -> np.ndarray:
    """inv[b,t] = position j with idx[b,j] == t, or -1 when token t was pruned."""
    B, k = idx.shape
    inv = np.full((B, n), -1, dtype=np.int64)
    for b in range(B):
        inv[b, idx[b]] = np.arange(k)
    return inv


def pts_gather(x: np.ndarray, idx: np.ndarray) -> np.ndarray:
    """x[b, I[b], :]  ->  [B,k,C]."""
    return np.stack([x[b, idx[b]] for b in range(x.shape[0])], axis=0)


def pivotal_token_selection(x: np.ndarray, h: int, w: int, keep_ratio: float):
    """Algorithm 1, first routine.  Returns (idx [B,k] ascending, score [B,n], kept rows [B,k,C])."""
    assert x.shape[1] == h * w
    k = kept_count(keep_ratio, h, w)
    s = pts_score(x)
    idx = pts_topk(s, k)
    return idx, s, pts_gather(np.asarray(x, dtype=F64), idx)


# ----------------------------------------------------------------------------------------------
# Cached Token Restoration  (Sec. 3.3, Eq. 6, Algorithm 1 second routine)
# ----------------------------------------------------------------------------------------------

def nearest_source(h: int, w: int, hc: int, wc: int) -> np.ndarray:
    """Nearest-neighbour source token of every destination token when a (hc,wc) map is
    interpolated to (h,w): sy = floor(y*hc/h), sx = floor(x*wc/w), row-major token order."""
    src = np.empty(h * w, dtype=np.int64)
    for y in range(h):
        sy = (y * hc) // h
        for xx in range(w):
            sx = (xx * wc) // w
            src[y * w + xx] = sy * wc + sx
    return src


def ctr_upsample(cache: np.ndarray, hc: int, wc: int, h: int, w: int) -> np.ndarray:
    """Eq. 6: y_cache_k = interpolate(y_{K-N}, (h_k, w_k)).  cache [B,hc*wc,C] -> [B,h*w,C]."""
    assert cache.shape[1] == hc * wc
    return cache[:, nearest_source(h, w, hc, wc), :]


def bilinear_taps(n_out: int, n_in: int):
    """Per destination index along one axis: the two source indices and the weight of the second one, for a
    blend with half-pixel centres: s = (dst + 0.5) * n_in / n_out - 0.5 clamped to [0, n_in - 1]."""
    i0 = np.empty(n_out, dtype=np.int64); i1 = np.empty(n_out, dtype=np.int64); t = np.empty(n_out, dtype=F64)
    for o in range(n_out):
        s = (o + 0.5) * n_in / n_out - 0.5
        s = min(max(s, 0.0), n_in - 1.0)
        i0[o] = int(math.floor(s))
        i1[o] = min(i0[o] + 1, n_in - 1)
        t[o] = s - i0[o]
    return i0, i1, t


def ctr_upsample_bilinear(cache: np.ndarray, hc: int, wc: int, h: int, w: int) -> np.ndarray:
    """Eq. 6 with interpolate = bilinear.  cache [B,hc*wc,C] -> [B,h*w,C]."""
    c = np.asarray(cache, dtype=F64).reshape(cache.shape[0], hc, wc, cache.shape[-1])
    y0, y1, ty = bilinear_taps(h, hc)
    x0, x1, tx = bilinear_taps(w, wc)
    ty = ty[None, :, None, None]; tx = tx[None, None, :, None]
    top = c[:, y0][:, :, x0] * (1 - tx) + c[:, y0][:, :, x1] * tx
    bot = c[:, y1][:, :, x0] * (1 - tx) + c[:, y1][:, :, x1] * tx
    return (top * (1 - ty) + bot * ty).reshape(cache.shape[0], h * w, cache.shape[-1])


def bicubic_taps(n_out: int, n_in: int, a: float = -0.75):
    """Per destination index along one axis: four source indices (clamped to the map) and their weights under
    cubic convolution (Keys' kernel with a = -0.75) at half-pixel centres, s = (dst + 0.5) * n_in / n_out - 0.5:
    W(d) = (a+2)|d|^3 - (a+3)|d|^2 + 1 for |d| <= 1,  a|d|^3 - 5a|d|^2 + 8a|d| - 4a for 1 < |d| < 2."""
    def kern(dist: float) -> float:
        dist = abs(dist)
        if dist <= 1.0:
            return (a + 2.0) * dist ** 3 - (a + 3.0) * dist ** 2 + 1.0
        if dist < 2.0:
            return a * dist ** 3 - 5.0 * a * dist ** 2 + 8.0 * a * dist - 4.0 * a
        return 0.0
    idx = np.empty((n_out, 4), dtype=np.int64); wt = np.empty((n_out, 4), dtype=F64)
    for o in range(n_out):
        s = (o + 0.5) * n_in / n_out - 0.5
        i0 = int(math.floor(s))
        for q in range(4):
            pos = i0 - 1 + q
            idx[o, q] = min(max(pos, 0), n_in - 1)
            wt[o, q] = kern(s - pos)
    return idx, wt


def ctr_upsample_bicubic(cache: np.ndarray, hc: int, wc: int, h: int, w: int) -> np.ndarray:
    """Eq. 6 with interpolate = bicubic (separable cubic convolution).  cache [B,hc*wc,C] -> [B,h*w,C]."""
    c = np.asarray(cache, dtype=F64).reshape(cache.shape[0], hc, wc, cache.shape[-1])
    yi, yw = bicubic_taps(h, hc)
    xi, xw = bicubic_taps(w, wc)
    out = np.zeros((cache.shape[0], h, w, cache.shape[-1]), dtype=F64)
    for qy in range(4):
        for qx in range(4):
            out += c[:, yi[:, qy]][:, :, xi[:, qx]] * (yw[:, qy][None, :, None, None] * xw[:, qx][None, None, :, None])
    return out.reshape(cache.shape[0], h * w, cache.shape[-1])


def cached_token_restoration(pivots: np.ndarray, idx: np.ndarray, cache: np.ndarray,
                             hc: int, wc: int, h: int, w: int, interp_mode: str = "nearest") -> np.ndarray:
    """Algorithm 1, second routine: upsample the cache to the current scale, then write the
    forwarded rows into their slots.  pivots [B,k,C], idx [B,k] -> [B,h*w,C]."""
    up = {"nearest": ctr_upsample, "bilinear": ctr_upsample_bilinear, "bicubic": ctr_upsample_bicubic}[interp_mode]
    out = np.array(up(np.asarray(cache, dtype=F64), hc, wc, h, w), dtype=F64, copy=True)
    for b in range(out.shape[0]):
        out[b, idx[b], :] = pivots[b]
    return out


# ----------------------------------------------------------------------------------------------
# Transformer sublayer pieces (standard definitions; the paper only names "Attention & FFN layer")
# ----------------------------------------------------------------------------------------------

def layernorm(x: np.ndarray, eps: float = 1e-6) -> np.ndarray:
    """Per-row LayerNorm over the last axis, biased variance, no affine."""
    x = np.asarray(x, dtype=F64)
    mu = x.mean(axis=-1, keepdims=True)
    var = ((x - mu) ** 2).mean(axis=-1, keepdims=True)
    return (x - mu) / np.sqrt(var + eps)


def modulate(a: np.ndarray, sigma: np.ndarray, beta: np.ndarray) -> np.ndarray:
    """AdaLN: a*(1+sigma)+beta with per-image vectors.  a [B,k,C]; sigma, beta [B,C]."""
    return a * (1.0 + sigma[:, None, :]) + beta[:, None, :]


def gelu_tanh(x: np.ndarray) -> np.ndarray:
    x = np.asarray(x, dtype=F64)
    return 0.5 * x * (1.0 + np.tanh(math.sqrt(2.0 / math.pi) * (x + 0.044715 * x ** 3)))


def linear(a: np.ndarray, W: np.ndarray, b: Optional[np.ndarray] = None) -> np.ndarray:
    """y = a @ W^T + b with W stored [out, in]."""
    y = np.asarray(a, dtype=F64) @ np.asarray(W, dtype=F64).T
    if b is not None:
        y = y + np.asarray(b, dtype=F64)
    return y


def softmax_rows(s: np.ndarray) -> np.ndarray:
    s = s - s.max(axis=-1, keepdims=True)
    e = np.exp(s)
    return e / e.sum(axis=-1, keepdims=True)


def qk_normalise(v: np.ndarray, H: int, scale: Optional[np.ndarray] = None, eps: float = 1e-12) -> np.ndarray:
    """Every head's vector divided by its Euclidean norm (floored at eps), times scale[h] if given.  v [k,C]."""
    k, C = v.shape
    hd = C // H
    vh = np.asarray(v, dtype=F64).reshape(k, H, hd)
    out = vh / np.maximum(np.sqrt((vh ** 2).sum(-1, keepdims=True)), eps)
    if scale is not None:
        out = out * np.asarray(scale, dtype=F64)[None, :, None]
    return out.reshape(k, C)


def rope_angles(tokens: np.ndarray, h: int, w: int, h_last: int, w_last: int, hd: int, base: float) -> np.ndarray:
    """Rotation angles [len(tokens), hd/2] of the tokens (row-major indices into the (h,w) map): columns
    [0, hd/4) = row coordinate * base^(-j/(hd/4)), columns [hd/4, hd/2) = column coordinate * the same."""
    quarter = hd // 4
    tok = np.asarray(tokens, dtype=np.int64)
    py = (tok // w).astype(F64) * h_last / h
    px = (tok % w).astype(F64) * w_last / w
    omega = np.asarray([base ** (-j / quarter) for j in range(quarter)], dtype=F64)
    return np.concatenate([py[:, None] * omega[None, :], px[:, None] * omega[None, :]], axis=1)


def apply_rope(v: np.ndarray, angles: np.ndarray, H: int) -> np.ndarray:
    """Rotates channel pairs (2i, 2i+1) of every head by angles[:, i], i < hd/2.  v [k,C], angles [k,hd/2]."""
    k, C = v.shape
    hd = C // H
    vh = np.asarray(v, dtype=F64).reshape(k, H, hd // 2, 2)
    c, s_ = np.cos(angles)[:, None, :], np.sin(angles)[:, None, :]
    out = np.empty_like(vh)
    out[..., 0] = vh[..., 0] * c - vh[..., 1] * s_
    out[..., 1] = vh[..., 0] * s_ + vh[..., 1] * c
    return out.reshape(k, C)


def attention(q: np.ndarray, K: np.ndarray, V: np.ndarray, H: int) -> np.ndarray:
    """Multi-head softmax(q K^T / sqrt(hd)) V with a materialised attention matrix, no mask.
    q [k,C], K [Lkv,C], V [Lkv,C]; head h owns channels [h*hd, (h+1)*hd)."""
    k, C = q.shape
    hd = C // H
    out = np.empty((k, C), dtype=F64)
    for h in range(H):
        sl = slice(h * hd, (h + 1) * hd)
        p = softmax_rows((q[:, sl] @ K[:, sl].T) / math.sqrt(hd))
        out[:, sl] = p @ V[:, sl]
    return out


# ----------------------------------------------------------------------------------------------
# The pruned scale step
# ----------------------------------------------------------------------------------------------

SUBLAYERS_SELF = ("attn", "ffn")
SUBLAYERS_CROSS = ("attn", "xattn", "ffn")


class VarOracle:
    """State (KV cache per block and image, sublayer caches) plus `var_step`.

    weights: dict of lists indexed by block, float arrays already widened from bf16:
      w_qkv [3C,C], b_qkv [3C], w_o [C,C], b_o [C], w_fc1 [F,C], b_fc1 [F], w_fc2 [C,F], b_fc2 [C],
      optional w_q_x [C,C], w_kv_x [2C,C] (K rows then V rows), w_o_x [C,C];
      'mod' [L,B,6,C] = (sigma1, beta1, gamma1, sigma2, beta2, gamma2); 'text' [B,T,C] or None.
    """

    def __init__(self, L: int, C: int, H: int, sides_hw: Sequence[Sequence[int]], cache_step: int,
                 weights: Dict, B: int, cross_len: int = 0, granularity: str = "sublayer",
                 interp_mode: str = "nearest", rope_base: Optional[float] = None, qk_scale: Optional[np.ndarray] = None):
        assert granularity in ("sublayer", "step") and interp_mode in ("nearest", "bilinear", "bicubic")
        self.granularity = granularity
        self.interp_mode, self.rope_base = interp_mode, rope_base
        self.qk_scale = None if qk_scale is None else np.asarray(qk_scale, dtype=F64)      # [L, H]
        self.L, self.C, self.H, self.B = L, C, H, B
        self.hw = [tuple(s) for s in sides_hw]
        self.cache_step = cache_step
        self.cross_len = cross_len
        self.w = weights
        self.subs = SUBLAYERS_CROSS if cross_len else SUBLAYERS_SELF
        self.reset()

    def reset(self) -> None:
        self.kv_len = 0
        self.step = 0
        self.Kc = [[np.zeros((0, self.C)) for _ in range(self.B)] for _ in range(self.L)]
        self.Vc = [[np.zeros((0, self.C)) for _ in range(self.B)] for _ in range(self.L)]
        self.cache: List[Dict[str, np.ndarray]] = [dict() for _ in range(self.L)]
        self.step_cache: Optional[np.ndarray] = None   # output token map of step K-N (granularity "step"; skipped steps)

    # -- one wrapped sublayer on compact rows ---------------------------------------------------
    def _branch(self, l: int, sub: str, xp: np.ndarray, tokens: Optional[np.ndarray] = None, scale_idx: int = 0) -> np.ndarray:
        """Sublayer branch output y for the compact rows xp [B,k,C] (before gate and residual).
        tokens [B,k]: the rows' original token indices in the map of scale `scale_idx` (rotary positions)."""
        w, mod = self.w, np.asarray(self.w["mod"][l], dtype=F64)      # mod [B,6,C]
        B = xp.shape[0]
        a = layernorm(xp)
        if sub == "attn":
            a = modulate(a, mod[:, 0], mod[:, 1])
            qkv = linear(a, w["w_qkv"][l], w["b_qkv"][l])
            q, kk, vv = qkv[..., :self.C], qkv[..., self.C:2 * self.C], qkv[..., 2 * self.C:]
            y = np.empty_like(xp)
            if self.qk_scale is not None or self.rope_base is not None:
                q, kk = np.array(q, copy=True), np.array(kk, copy=True)
                h_, w_ = self.hw[scale_idx]
                hl, wl = self.hw[-1]
                for b in range(B):
                    if self.qk_scale is not None:
                        q[b] = qk_normalise(q[b], self.H, self.qk_scale[l])
                        kk[b] = qk_normalise(kk[b], self.H)
                    if self.rope_base is not None:
                        ang = rope_angles(tokens[b], h_, w_, hl, wl, self.C // self.H, self.rope_base)
                        q[b] = apply_rope(q[b], ang, self.H)
                        kk[b] = apply_rope(kk[b], ang, self.H)
            for b in range(B):
                # KV cache: all earlier (possibly pruned) scales plus the rows forwarded now
                self.Kc[l][b] = np.concatenate([self.Kc[l][b][:self.kv_len], kk[b]], axis=0)
                self.Vc[l][b] = np.concatenate([self.Vc[l][b][:self.kv_len], vv[b]], axis=0)
                o = attention(q[b], self.Kc[l][b], self.Vc[l][b], self.H)
                y[b] = linear(o, w["w_o"][l], w["b_o"][l])
            return y
        if sub == "xattn":
            q = linear(a, w["w_q_x"][l])
            y = np.empty_like(xp)
            for b in range(B):
                kv = linear(np.asarray(w["text"][b], dtype=F64), w["w_kv_x"][l])
                o = attention(q[b], kv[:, :self.C], kv[:, self.C:], self.H)
                y[b] = linear(o, w["w_o_x"][l])
            return y
        if sub == "ffn":
            a = modulate(a, mod[:, 3], mod[:, 4])
            hmid = gelu_tanh(linear(a, w["w_fc1"][l], w["b_fc1"][l]))
            return linear(hmid, w["w_fc2"][l], w["b_fc2"][l])
        raise ValueError(sub)

    def var_step(self, x: np.ndarray, scale_idx: int, keep_ratio: float,
                 forced_idx: Optional[Dict] = None, trace: Optional[Dict] = None) -> np.ndarray:
        """One scale step over all L blocks.  x [B,n,C] is the residual stream entering block 0.

        For each block and each wrapped sublayer: PTS (when keep_ratio < 1) -> branch on kept rows
        -> cache write (at the caching step) -> CTR (when keep_ratio < 1) -> gate and residual add.
        `forced_idx[(l,sub)]` overrides the selection; `trace[(l,sub)]` receives idx / score / y."""
        assert scale_idx == self.step, "steps must be taken in order"
        x = np.array(x, dtype=F64, copy=True)
        B, n, C = x.shape
        h, w_ = self.hw[scale_idx]
        assert n == h * w_ and B == self.B and C == self.C
        if keep_ratio == 0.0:
            # Sec. 4.1 "Implementation Details": a 100 % pruning ratio drops every token -- the step is
            # skipped and the intermediate output is interpolated to the target resolution.  Reading: the
            # intermediate output is the output token map of the caching step (the last step that ran in
            # full); nothing enters the KV cache.
            assert self.step_cache is not None and scale_idx > self.cache_step
            hc, wc = self.hw[self.cache_step]
            self.step += 1
            up = {"nearest": ctr_upsample, "bilinear": ctr_upsample_bilinear, "bicubic": ctr_upsample_bicubic}[self.interp_mode]
            return up(self.step_cache, hc, wc, h, w_)
        pruned = keep_ratio < 1.0
        k = kept_count(keep_ratio, h, w_) if pruned else n
        if self.granularity == "step":
            return self._var_step_whole(x, scale_idx, pruned, k, forced_idx, trace)
        for l in range(self.L):
            mod = np.asarray(self.w["mod"][l], dtype=F64)
            for sub in self.subs:
                score = None
                if pruned:
                    score = pts_score(x)
                    if forced_idx is not None:
                        idx = np.asarray(forced_idx[(l, sub)], dtype=np.int64)
                    else:
                        idx = pts_topk(score, k)
                    xp = pts_gather(x, idx)
                else:
                    idx = None
                    xp = x
                tokens = idx if pruned else np.broadcast_to(np.arange(n), (B, n))
                y = self._branch(l, sub, xp, tokens, scale_idx)
                if scale_idx == self.cache_step:
                    assert not pruned, "the caching step is the last unpruned step"
                    self.cache[l][sub] = y.copy()
                if pruned:
                    hc, wc = self.hw[self.cache_step]
                    yfull = cached_token_restoration(y, idx, self.cache[l][sub], hc, wc, h, w_, self.interp_mode)
                else:
                    yfull = y
                if trace is not None:
                    trace[(l, sub)] = {"idx": idx, "score": score, "y": y}
                if sub == "attn":
                    x = x + mod[:, 2][:, None, :] * yfull
                elif sub == "ffn":
                    x = x + mod[:, 5][:, None, :] * yfull
                else:
                    x = x + yfull
        if scale_idx == self.cache_step:
            self.step_cache = x.copy()          # output map of the caching step (used by skipped steps)
        self.kv_len += k
        self.step += 1
        return x

    def _var_step_whole(self, x: np.ndarray, scale_idx: int, pruned: bool, k: int,
                        forced_idx: Optional[Dict], trace: Optional[Dict]) -> np.ndarray:
        """granularity "step": PTS once on the step input, all blocks on the kept rows (compact residual
        stream), CTR once from the cached output map of the caching step.  `forced_idx[("step",)]`
        overrides the selection; `trace[("step",)]` receives idx / score."""
        h, w_ = self.hw[scale_idx]
        idx, score = None, None
        xc = x
        if pruned:
            score = pts_score(x)
            idx = np.asarray(forced_idx[("step",)], dtype=np.int64) if forced_idx is not None else pts_topk(score, k)
            xc = pts_gather(x, idx)
        if trace is not None:
            trace[("step",)] = {"idx": idx, "score": score}
        tokens = idx if pruned else np.broadcast_to(np.arange(x.shape[1]), x.shape[:2])
        for l in range(self.L):
            mod = np.asarray(self.w["mod"][l], dtype=F64)
            for sub in self.subs:
                y = self._branch(l, sub, xc, tokens, scale_idx)
                if sub == "attn":
                    xc = xc + mod[:, 2][:, None, :] * y
                elif sub == "ffn":
                    xc = xc + mod[:, 5][:, None, :] * y
                else:
                    xc = xc + y
        if scale_idx == self.cache_step:
            assert not pruned, "the caching step is the last unpruned step"
            self.step_cache = xc.copy()
        if pruned:
            hc, wc = self.hw[self.cache_step]
            out = cached_token_restoration(xc, idx, self.step_cache, hc, wc, h, w_, self.interp_mode)
        else:
            out = xc
        self.kv_len += k
        self.step += 1
        return out

    def run_schedule(self, inputs: Sequence[np.ndarray], keep: Sequence[float]) -> List[np.ndarray]:
        """All steps 0..K-1 in order; inputs[k] is the token map entering step k."""
        self.reset()
        return [self.var_step(inputs[i], i, keep[i]) for i in range(len(inputs))]
