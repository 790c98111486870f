"""Shared test plumbing: turns the seeded inputs into what the oracle and the CUDA binding each take.
Holds no arithmetic of the method."""
from __future__ import annotations

import numpy as np

from oracle import fastvar_oracle as O
from paper_2503_23367_b200 import inputs as I

SUB_NAMES = {2: ("attn", "ffn"), 3: ("attn", "xattn", "ffn")}


def oracle_weights(mt: I.ModelTensors) -> dict:
    f = lambda lst: [I.bf16_bits_to_f32(a).astype(np.float64) for a in lst]
    w = {k: f(getattr(mt, k)) for k in ("w_qkv", "b_qkv", "w_o", "b_o", "w_fc1", "b_fc1", "w_fc2", "b_fc2",
                                          "w_q_x", "w_kv_x", "w_o_x")}
    w["mod"] = mt.mod.astype(np.float64)
    w["text"] = None if mt.text is None else I.bf16_bits_to_f32(mt.text).astype(np.float64)
    return w


def make_oracle(wl: I.Workload, mt: I.ModelTensors) -> O.VarOracle:
    return O.VarOracle(wl.L, wl.C, wl.H, [(s, s) for s in wl.sides], cache_step=wl.cache_step,
                       weights=oracle_weights(mt), B=wl.B, cross_len=wl.cross_len)


def run_oracle(wl: I.Workload, mt: I.ModelTensors, xs, forced=None):
    """Whole schedule on the oracle.  Returns (outputs per step, traces per step)."""
    orc = make_oracle(wl, mt)
    outs, traces = [], []
    for i, x in enumerate(xs):
        tr = {}
        kw = {"forced_idx": forced[i]} if (forced is not None and wl.keep[i] < 1.0) else {}
        outs.append(orc.var_step(x, i, wl.keep[i], trace=tr, **kw))
        traces.append(tr)
    return orc, outs, traces


def trace_to_index_tensor(wl: I.Workload, trace: dict) -> np.ndarray:
    """Oracle trace of one pruned step -> int32 [L, n_sub, B, k] in the library's sublayer order."""
    names = SUB_NAMES[wl.n_sub]
    return np.stack([np.stack([trace[(l, s)]["idx"] for s in names]) for l in range(wl.L)]).astype(np.int32)


def per_token_errors(got: np.ndarray, ref: np.ndarray):
    """(max abs error, min cosine over tokens) between [.., C] arrays."""
    got = np.asarray(got, dtype=np.float64).reshape(-1, got.shape[-1])
    ref = np.asarray(ref, dtype=np.float64).reshape(-1, ref.shape[-1])
    max_abs = float(np.abs(got - ref).max())
    num = (got * ref).sum(-1)
    den = np.linalg.norm(got, axis=-1) * np.linalg.norm(ref, axis=-1)
    cos = np.where(den > 0, num / np.maximum(den, 1e-300), 1.0)
    return max_abs, float(cos.min())
