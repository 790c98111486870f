"""Seeded synthetic inputs for the pruned VAR scale step.

This module only *draws numbers and lays them out*: token maps, weights, AdaLN
modulation vectors, text tokens and the workload shapes.  It contains none of
the method's arithmetic (no score, top-k, normalisation, GEMM, attention or
restore) and is the one module that both the tests of the CPU oracle and the
CUDA path's tests / benchmark may use, so that both sides see bit-identical
inputs.

Generator: counter based.  Element ``i`` of the tensor with seed ``s`` takes
two 64-bit hashes ``mix(s, 2i)`` and ``mix(s, 2i+1)`` (SplitMix64 finaliser),
turns them into uniforms in (0, 1) and applies Box-Muller.  Values depend only
on ``(seed, flat index)``, never on chunking or thread count.
"""
from __future__ import annotations

import math
from dataclasses import dataclass, field, replace
from typing import Dict, List, Optional, Sequence

import numpy as np

_M64 = np.uint64(0xFFFFFFFFFFFFFFFF)
_GOLD = np.uint64(0x9E3779B97F4A7C15)
_C1 = np.uint64(0xBF58476D1CE4E5B9)
_C2 = np.uint64(0x94D049BB133111EB)


def _mix(seed: int, ctr: np.ndarray) -> np.ndarray:
    """SplitMix64 finaliser of ``seed * GOLD + (ctr + 1) * C1`` (uint64 wrap)."""
    with np.errstate(over="ignore"):
        z = np.uint64(seed & 0xFFFFFFFFFFFFFFFF) * _GOLD + (ctr + np.uint64(1)) * _C1
        z ^= z >> np.uint64(30)
        z *= _C1
        z ^= z >> np.uint64(27)
        z *= _C2
        z ^= z >> np.uint64(31)
    return z


def uniform01(seed: int, count: int, offset: int = 0) -> np.ndarray:
    """``count`` doubles in the open interval (0, 1) for counters offset..offset+count."""
    ctr = np.arange(offset, offset + count, dtype=np.uint64)
    z = _mix(seed, ctr)
    return ((z >> np.uint64(11)).astype(np.float64) + 0.5) * (1.0 / 9007199254740992.0)


def normal(seed: int, shape: Sequence[int], std: float = 1.0, chunk: int = 1 << 22) -> np.ndarray:
    """fp32 N(0, std^2) tensor of ``shape``; element i uses counters 2i and 2i+1."""
    total = int(np.prod(shape)) if len(shape) else 1
    out = np.empty(total, dtype=np.float32)
    for start in range(0, total, chunk):
        m = min(chunk, total - start)
        u = uniform01(seed, 2 * m, 2 * start)
        u1, u2 = u[0::2], u[1::2]
        out[start:start + m] = (np.sqrt(-2.0 * np.log(u1)) * np.cos(2.0 * math.pi * u2) * std).astype(np.float32)
    return out.reshape(tuple(shape))


def to_bf16_bits(a: np.ndarray) -> np.ndarray:
    """Round an fp32 array to bfloat16 (round to nearest even); returns the uint16 bit patterns."""
    u = np.ascontiguousarray(a, dtype=np.float32).view(np.uint32)
    rounded = u + np.uint32(0x7FFF) + ((u >> np.uint32(16)) & np.uint32(1))
    return (rounded >> np.uint32(16)).astype(np.uint16)


def bf16_bits_to_f32(bits: np.ndarray) -> np.ndarray:
    """Widen bfloat16 bit patterns to fp32 (exact)."""
    return (bits.astype(np.uint32) << np.uint32(16)).view(np.float32)


def normal_bf16(seed: int, shape: Sequence[int], std: float = 1.0) -> np.ndarray:
    """N(0, std^2) values rounded to bfloat16, returned as uint16 bit patterns."""
    return to_bf16_bits(normal(seed, shape, std))


# --------------------------------------------------------------------------------------
# Workload shapes
# --------------------------------------------------------------------------------------

@dataclass(frozen=True)
class Workload:
    """One synthetic random-weight model plus its scale and keep-ratio schedule."""
    name: str
    L: int                 # transformer blocks
    C: int                 # width
    H: int                 # attention heads (head dim = C / H)
    B: int                 # images per batch
    sides: tuple           # scale schedule: side of the square token map at every step
    keep: tuple            # keep ratio per step (1.0 = unpruned)
    cross_len: int = 0     # text tokens for cross-attention (0 = no cross-attention sublayer)
    mlp_ratio: int = 4
    seed: int = 0

    @property
    def hd(self) -> int:
        return self.C // self.H

    @property
    def n_sub(self) -> int:
        return 3 if self.cross_len else 2

    @property
    def cache_step(self) -> int:
        """Index of the last unpruned step before the first pruned one (the caching step K-N)."""
        first = next((i for i, r in enumerate(self.keep) if r < 1.0), len(self.keep))
        return first - 1

    def tokens(self, step: int) -> int:
        return self.sides[step] * self.sides[step]

    def with_depth(self, L: int) -> "Workload":
        return replace(self, L=L, name=f"{self.name}-L{L}")


def _keeps(sides, mapping):
    return tuple(float(mapping.get(s, 1.0)) for s in sides)


_VAR256 = (1, 2, 3, 4, 5, 6, 8, 10, 13, 16)
_VAR512 = (1, 2, 3, 4, 6, 9, 13, 18, 24, 32)
_INF1K = (1, 2, 4, 6, 8, 12, 16, 20, 24, 32, 40, 48, 64)
_INF2K = _INF1K + (80, 96, 128)

WORKLOADS: Dict[str, Workload] = {
    "tiny": Workload("tiny", L=2, C=256, H=4, B=1, sides=_VAR256,
                     keep=_keeps(_VAR256, {13: 0.5, 16: 0.5}), seed=1000),
    "var_d16_256": Workload("var_d16_256", L=16, C=1024, H=16, B=8, sides=_VAR256,
                            keep=_keeps(_VAR256, {13: 0.6, 16: 0.5}), seed=2000),
    "var_d30_512": Workload("var_d30_512", L=30, C=1920, H=30, B=4, sides=_VAR512,
                            keep=_keeps(_VAR512, {18: 0.75, 24: 0.5, 32: 0.25}), seed=3000),
    "infinity_2b_1k": Workload("infinity_2b_1k", L=32, C=2048, H=16, B=2, sides=_INF1K,
                               keep=_keeps(_INF1K, {40: 0.6, 48: 0.4, 64: 0.2}),
                               cross_len=512, seed=4000),
    # the paper's own Infinity schedule (Sec. 4.1): pruning ratios {40, 50, 100, 100} % on the last four
    # scale steps, i.e. keep 0.6 / 0.5 and two skipped steps
    "infinity_2b_1k_paper": Workload("infinity_2b_1k_paper", L=32, C=2048, H=16, B=2, sides=_INF1K,
                                     keep=_keeps(_INF1K, {32: 0.6, 40: 0.5, 48: 0.0, 64: 0.0}),
                                     cross_len=512, seed=4000),
    "infinity_2b_2k": Workload("infinity_2b_2k", L=32, C=2048, H=16, B=1, sides=_INF2K,
                               keep=_keeps(_INF2K, {64: 0.2, 80: 0.2, 96: 0.2, 128: 0.2}),
                               cross_len=512, seed=5000),
}


# --------------------------------------------------------------------------------------
# Tensors
# --------------------------------------------------------------------------------------

def token_map(seed: int, B: int, side_h: int, side_w: int, C: int, kind: str = "iid") -> np.ndarray:
    """fp32 token map ``[B, h*w, C]``.

    ``iid``: N(0,1).  ``structured``: a smooth field (bilinear blow-up of a coarse
    N(0,1) grid of side ceil(h/8)) plus 0.1*N(0,1) everywhere plus N(0,1) on a
    random 20 % "edge" subset, so that the deviation-from-mean scores are bimodal
    the way texture / flat regions are.
    """
    n = side_h * side_w
    if kind == "iid":
        return normal(seed, (B, n, C))
    if kind != "structured":
        raise ValueError(kind)
    ch, cw = max(1, -(-side_h // 8)), max(1, -(-side_w // 8))
    coarse = normal(seed, (B, ch, cw, C)).astype(np.float64)
    ys = (np.arange(side_h) + 0.5) * ch / side_h - 0.5
    xs = (np.arange(side_w) + 0.5) * cw / side_w - 0.5
    y0 = np.clip(np.floor(ys).astype(int), 0, ch - 1); y1 = np.clip(y0 + 1, 0, ch - 1)
    x0 = np.clip(np.floor(xs).astype(int), 0, cw - 1); x1 = np.clip(x0 + 1, 0, cw - 1)
    fy = np.clip(ys - np.floor(ys), 0, 1)[None, :, None, None]
    fx = np.clip(xs - np.floor(xs), 0, 1)[None, None, :, None]
    top = coarse[:, y0][:, :, x0] * (1 - fx) + coarse[:, y0][:, :, x1] * fx
    bot = coarse[:, y1][:, :, x0] * (1 - fx) + coarse[:, y1][:, :, x1] * fx
    smooth = (top * (1 - fy) + bot * fy).reshape(B, n, C)
    noise = normal(seed + 1, (B, n, C)).astype(np.float64)
    edge = uniform01(seed + 2, B * n).reshape(B, n, 1) < 0.2
    extra = normal(seed + 3, (B, n, C)).astype(np.float64)
    return (smooth + 0.1 * noise + edge * extra).astype(np.float32)


@dataclass
class ModelTensors:
    """All step-invariant tensors of one synthetic model, as numpy arrays.

    Linear weights are stored ``[out_features, in_features]`` (so y = a @ W.T + b), as
    bfloat16 bit patterns (uint16); biases likewise; ``mod`` is fp32
    ``[L, B, 6, C]`` holding (sigma1, beta1, gamma1, sigma2, beta2, gamma2) per image;
    ``text`` is bfloat16 bits ``[B, cross_len, C]`` or None.
    """
    w_qkv: List[np.ndarray] = field(default_factory=list)
    b_qkv: List[np.ndarray] = field(default_factory=list)
    w_o: List[np.ndarray] = field(default_factory=list)
    b_o: List[np.ndarray] = field(default_factory=list)
    w_fc1: List[np.ndarray] = field(default_factory=list)
    b_fc1: List[np.ndarray] = field(default_factory=list)
    w_fc2: List[np.ndarray] = field(default_factory=list)
    b_fc2: List[np.ndarray] = field(default_factory=list)
    w_q_x: List[np.ndarray] = field(default_factory=list)
    w_kv_x: List[np.ndarray] = field(default_factory=list)
    w_o_x: List[np.ndarray] = field(default_factory=list)
    mod: Optional[np.ndarray] = None
    text: Optional[np.ndarray] = None


def model_tensors(wl: Workload, w_std: float = 0.02, mod_std: float = 0.3) -> ModelTensors:
    """Draw every weight of ``wl``: bf16 N(0, w_std^2) matrices and biases, fp32 N(0, mod_std^2)
    modulation vectors, bf16 N(0,1) text tokens.  Tensor ``t`` of block ``l`` uses seed
    ``wl.seed + 100 + 16*l + t``."""
    C, F = wl.C, wl.C * wl.mlp_ratio
    mt = ModelTensors()
    for l in range(wl.L):
        s = wl.seed + 100 + 16 * l
        mt.w_qkv.append(normal_bf16(s + 0, (3 * C, C), w_std))
        mt.b_qkv.append(normal_bf16(s + 1, (3 * C,), w_std))
        mt.w_o.append(normal_bf16(s + 2, (C, C), w_std))
        mt.b_o.append(normal_bf16(s + 3, (C,), w_std))
        mt.w_fc1.append(normal_bf16(s + 4, (F, C), w_std))
        mt.b_fc1.append(normal_bf16(s + 5, (F,), w_std))
        mt.w_fc2.append(normal_bf16(s + 6, (C, F), w_std))
        mt.b_fc2.append(normal_bf16(s + 7, (C,), w_std))
        if wl.cross_len:
            mt.w_q_x.append(normal_bf16(s + 8, (C, C), w_std))
            mt.w_kv_x.append(normal_bf16(s + 9, (2 * C, C), w_std))
            mt.w_o_x.append(normal_bf16(s + 10, (C, C), w_std))
    mt.mod = normal(wl.seed + 50, (wl.L, wl.B, 6, C), mod_std)
    if wl.cross_len:
        mt.text = normal_bf16(wl.seed + 51, (wl.B, wl.cross_len, C), 1.0)
    return mt


def step_input(wl: Workload, step: int, kind: str = "iid") -> np.ndarray:
    """Token map entering scale step ``step`` of ``wl`` (fp32 ``[B, n, C]``)."""
    s = wl.sides[step]
    return token_map(wl.seed + 10_000 + 10 * step, wl.B, s, s, wl.C, kind)


@dataclass
class GenerationTensors:
    """Step-invariant tensors of the synthetic generation loop around the scale step: the quantiser's
    codebook ``[V, d]`` (fp32), the output head ``w_head [V, C]`` / ``b_head [V]`` (bf16 bits) with its
    AdaLN vectors ``mod_head [B, 2, C]`` (sigma, beta; fp32), the map from accumulated code vectors to the
    next scale's tokens ``w_in [C, d]`` / ``b_in [C]`` (fp32) and one position embedding per scale
    ``pos[k] [n_k, C]`` (fp32)."""
    codebook: Optional[np.ndarray] = None
    w_head: Optional[np.ndarray] = None
    b_head: Optional[np.ndarray] = None
    mod_head: Optional[np.ndarray] = None
    w_in: Optional[np.ndarray] = None
    b_in: Optional[np.ndarray] = None
    pos: List[np.ndarray] = field(default_factory=list)
    start: Optional[np.ndarray] = None   # [B, n_0, C] fp32: the token map entering the first step


def generation_tensors(wl: Workload, V: int = 4096, d: int = 32, w_std: float = 0.02) -> GenerationTensors:
    """Draw the generation-loop tensors of ``wl`` (seeds ``wl.seed + 60 ..``).  The head's weights are larger
    than the blocks' (std ``4 * w_std``) so that its logits spread over a few units, as a trained head's do."""
    g = GenerationTensors()
    g.codebook = normal(wl.seed + 60, (V, d), 1.0)
    g.w_head = normal_bf16(wl.seed + 61, (V, wl.C), 4 * w_std)
    g.b_head = normal_bf16(wl.seed + 62, (V,), w_std)
    g.mod_head = normal(wl.seed + 63, (wl.B, 2, wl.C), 0.3)
    g.w_in = normal(wl.seed + 64, (wl.C, d), 1.0 / math.sqrt(d))
    g.b_in = normal(wl.seed + 65, (wl.C,), w_std)
    g.pos = [normal(wl.seed + 70 + k, (wl.tokens(k), wl.C), 0.5) for k in range(len(wl.sides))]
    g.start = normal(wl.seed + 66, (wl.B, wl.tokens(0), wl.C), 1.0)
    return g


def gumbel_noise(seed: int, shape: Sequence[int]) -> np.ndarray:
    """Standard Gumbel draws -log(-log(u)) from the counter-based uniforms, fp32.  The sampler's random
    numbers are an input of both implementations, so neither has to reproduce a generator."""
    n = int(np.prod(shape))
    u = uniform01(seed, n).astype(np.float64)
    return (-np.log(-np.log(u))).astype(np.float32).reshape(shape)
