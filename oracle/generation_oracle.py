"""CPU oracle for the generation loop around the scale step (test infrastructure, NOT a product path).

The paper's preliminary (Sec. 3.1) states the loop a next-scale-prediction model runs: at step k the
transformer turns the token map of scale k into a residual f_k, and the running prediction follows
Eq. 2,  r_k = interpolate(r_{k-1}, (h_k, w_k)) + f_k,  whose unfolded form is Eq. 3.  The paper says
nothing about how f_k is read off the transformer output nor how the next step's token map is made,
so this file takes the plain construction of VAR-style models, stated here as readings:

  * output head: logits = (LN(x) * (1 + sigma_h) + beta_h) @ W_head^T + b_head over a codebook of V entries
    (LN without affine, eps 1e-6, as in the blocks);
  * token choice: id = argmax_v (logits_v + tau * noise_v); noise = 0 is greedy decoding, standard Gumbel
    noise makes it a draw from softmax(logits / tau) (the Gumbel-max identity).  The noise is an INPUT.
    Ties go to the lowest id;
  * f_k = codebook[id]  (a d-vector per token);
  * Eq. 2 with interpolate = nearest neighbour, src = floor(dst * in / out) per axis (the same reading
    as for Eq. 6); r_0 does not exist: r_1 = f_1;
  * the token map entering step k+1 is  interpolate(r_k, (h_{k+1}, w_{k+1})) @ W_in^T + b_in + pos_{k+1}.

Everything is numpy float64, each function the definition written out.  Shares no code with the CUDA
path.  Pins: tests/test_generation_oracle_pins.py (Eq. 2 against Eq. 3 on nested scales, brute-force argmax with
ties, the Gumbel-max identity on a small alphabet, identity / constant special cases of the head and of
the next-input map), and the loop itself by its records: each obeys Eq. 2 against the one before, each
step is fed the map built from the previous record, and with keep ratio 1 the transformer outputs equal a
plain run of the same inputs.  The paper prints no worked example of
the loop.
"""
from __future__ import annotations

from typing import Dict, List, Optional, Sequence, Tuple

import numpy as np

from . import fastvar_oracle as O

F64 = np.float64


def head_logits(x: np.ndarray, sigma_h: np.ndarray, beta_h: np.ndarray, w_head: np.ndarray,
                b_head: Optional[np.ndarray]) -> np.ndarray:
    """x [B,n,C], sigma_h / beta_h [B,C], w_head [V,C] -> logits [B,n,V]."""
    a = O.modulate(O.layernorm(x), np.asarray(sigma_h, dtype=F64), np.asarray(beta_h, dtype=F64))
    return O.linear(a, w_head, b_head)


def choose_tokens(logits: np.ndarray, noise: Optional[np.ndarray] = None, tau: float = 1.0) -> Tuple[np.ndarray, np.ndarray]:
    """id = argmax_v (logits + tau * noise), lowest id on ties.  Returns (ids [B,n] int64, margin [B,n]):
    margin = best minus second-best perturbed logit, the quantity a caller needs to flag decisions that a
    rounding-level change of the logits could flip."""
    z = np.asarray(logits, dtype=F64)
    if noise is not None:
        z = z + float(tau) * np.asarray(noise, dtype=F64)
    ids = np.argmax(z, axis=-1)                      # first occurrence = lowest id
    top2 = np.partition(z, z.shape[-1] - 2, axis=-1)[..., -2:]
    return ids.astype(np.int64), (top2[..., 1] - top2[..., 0])


def interpolate_nearest(r: np.ndarray, hp: int, wp: int, h: int, w: int) -> np.ndarray:
    """[B, hp*wp, d] -> [B, h*w, d], src = floor(dst * in / out) per axis."""
    return np.asarray(r, dtype=F64)[:, O.nearest_source(h, w, hp, wp), :]


def residual_accumulate(r_prev: Optional[np.ndarray], hp: int, wp: int, ids: np.ndarray, codebook: np.ndarray,
                        h: int, w: int) -> np.ndarray:
    """Eq. 2: r_k = interpolate(r_{k-1}, (h_k, w_k)) + f_k with f_k = codebook[ids]; r_1 = f_1."""
    f = np.asarray(codebook, dtype=F64)[np.asarray(ids)]
    if r_prev is None:
        return f
    return interpolate_nearest(r_prev, hp, wp, h, w) + f


def cumulative_form(fs: Sequence[np.ndarray], sizes: Sequence[Tuple[int, int]], k: int) -> np.ndarray:
    """Eq. 3: r_k = sum_{i <= k} interpolate(f_i, (h_k, w_k))  (k zero-based, inclusive)."""
    h, w = sizes[k]
    out = 0.0
    for i in range(k + 1):
        out = out + interpolate_nearest(fs[i], sizes[i][0], sizes[i][1], h, w)
    return out


def next_scale_input(r: np.ndarray, h: int, w: int, h2: int, w2: int, w_in: np.ndarray, b_in: Optional[np.ndarray],
                     pos: Optional[np.ndarray]) -> np.ndarray:
    """x_{k+1} = interpolate(r_k, (h2, w2)) @ W_in^T + b_in + pos.  r [B,h*w,d], w_in [C,d], pos [h2*w2, C]."""
    x = O.linear(interpolate_nearest(r, h, w, h2, w2), w_in, b_in)
    if pos is not None:
        x = x + np.asarray(pos, dtype=F64)[None, :, :]
    return x


class GenerationOracle:
    """The K-step loop: var_step -> head -> token choice -> Eq. 2 -> next token map."""

    def __init__(self, var: "O.VarOracle", sizes: Sequence[Tuple[int, int]], codebook, w_head, b_head, mod_head,
                 w_in, b_in, pos: Sequence[np.ndarray]):
        self.var, self.sizes = var, [tuple(s) for s in sizes]
        self.codebook, self.w_head, self.b_head = codebook, w_head, b_head
        self.mod_head, self.w_in, self.b_in, self.pos = np.asarray(mod_head, dtype=F64), w_in, b_in, list(pos)

    def generate(self, start: np.ndarray, keep: Sequence[float], noise: Optional[Sequence[np.ndarray]] = None,
                 tau: float = 1.0) -> List[Dict[str, np.ndarray]]:
        """start [B, n_0, C] enters step 0.  Returns one record per step: the step's input `x`, the
        transformer output `y`, `logits`, `ids`, `margin`, and the running prediction `r` (Eq. 2)."""
        self.var.reset()
        recs: List[Dict[str, np.ndarray]] = []
        x, r = np.asarray(start, dtype=F64), None
        K = len(self.sizes)
        for k in range(K):
            h, w = self.sizes[k]
            y = self.var.var_step(x, k, keep[k])
            logits = head_logits(y, self.mod_head[:, 0], self.mod_head[:, 1], self.w_head, self.b_head)
            ids, margin = choose_tokens(logits, None if noise is None else noise[k], tau)
            hp, wp = self.sizes[k - 1] if k else (0, 0)
            r = residual_accumulate(r, hp, wp, ids, self.codebook, h, w)
            recs.append({"x": x, "y": y, "logits": logits, "ids": ids, "margin": margin, "r": r})
            if k + 1 < K:
                h2, w2 = self.sizes[k + 1]
                x = next_scale_input(r, h, w, h2, w2, self.w_in, self.b_in, self.pos[k + 1])
        return recs
