"""Optional backbone pieces through fv_var_step against the oracle with the same options: cosine attention
and 2-D rotary positions (applied in the QKV GEMM's epilogue, by ORIGINAL token index at pruned steps) and
bilinear interpolation of the cache in the restoration.  Forced-index mode, the step tolerances."""
import numpy as np
import pytest
import torch

from oracle import fastvar_oracle as O
from paper_2503_23367_b200 import binding as fv
from paper_2503_23367_b200 import inputs as I
from tests.helpers import oracle_weights, per_token_errors, trace_to_index_tensor

pytestmark = pytest.mark.gpu
DEV = "cuda:0"
MAX_ABS, MIN_COS = 3e-2, 0.999


def sharpen_attention(mt, C, factor=6.0):
    """Input preparation only: the Q and K rows of every QKV weight are drawn `factor` times larger, so that the
    attention is peaked and what happens to q and k shows in the output (with the default N(0, 0.02^2) weights
    the softmax is nearly uniform and rotating q and k changes the result by less than the tolerance)."""
    for l in range(len(mt.w_qkv)):
        w = I.bf16_bits_to_f32(mt.w_qkv[l]).copy()
        w[:2 * C] *= factor
        mt.w_qkv[l] = I.to_bf16_bits(w)


def run_both(wl, granularity=0, rope_base=0.0, qk=False, interp_mode=0, kind="iid"):
    mt = I.model_tensors(wl)
    sharpen_attention(mt, wl.C)
    xs = [I.step_input(wl, i, kind) for i in range(len(wl.sides))]
    qk_scale = (6.0 + 8.0 * I.uniform01(wl.seed + 5, wl.L * wl.H).reshape(wl.L, wl.H)).astype(np.float32) if qk else None
    sizes = [(s, s) for s in wl.sides]
    orc = O.VarOracle(wl.L, wl.C, wl.H, sizes, cache_step=wl.cache_step, weights=oracle_weights(mt), B=wl.B, cross_len=wl.cross_len,
                      granularity="step" if granularity else "sublayer", interp_mode=("nearest", "bilinear", "bicubic")[interp_mode],
                      rope_base=rope_base or None, qk_scale=qk_scale)
    ref, forced = [], []
    for i, x in enumerate(xs):
        tr = {}
        ref.append(orc.var_step(x, i, wl.keep[i], trace=tr))
        if wl.keep[i] < 1.0 and wl.keep[i] > 0.0:
            forced.append(tr[("step",)]["idx"].astype(np.int32) if granularity else trace_to_index_tensor(wl, tr))
        else:
            forced.append(None)
    cap = sum(wl.tokens(i) if wl.keep[i] >= 1.0 else (O.kept_count(wl.keep[i], s, s) if wl.keep[i] > 0 else 0) for i, s in enumerate(wl.sides))
    ctx = fv.FvContext(wl.L, wl.C, wl.H, sizes, wl.cache_step, wl.B, cap, mt, cross_len=wl.cross_len, device=DEV, granularity=granularity,
                       rope_base=rope_base, interp_mode=interp_mode, qk_scale=qk_scale)
    ctx.reset()
    worst = (0.0, 1.0)
    for i, x in enumerate(xs):
        f = None if forced[i] is None else torch.from_numpy(np.ascontiguousarray(forced[i])).to(DEV)
        got = ctx.var_step(torch.from_numpy(x).to(DEV), i, wl.keep[i], forced_idx=f).cpu().numpy()
        err, cos = per_token_errors(got, ref[i])
        worst = (max(worst[0], err), min(worst[1], cos))
        assert err <= MAX_ABS and cos >= MIN_COS, f"step {i} side {wl.sides[i]}: max-abs {err:.4g}, cos {cos:.6f}"
    torch.cuda.synchronize()
    assert ctx.device_status() == 0
    ctx.close()
    # the options must matter at these sizes, or agreeing with the oracle would not show that they ran: the
    # same schedule on a plain oracle (same kept sets) has to sit outside the tolerance of the one with options
    plain = O.VarOracle(wl.L, wl.C, wl.H, sizes, cache_step=wl.cache_step, weights=oracle_weights(mt), B=wl.B, cross_len=wl.cross_len,
                        granularity="step" if granularity else "sublayer")
    far = 0.0
    for i, x in enumerate(xs):
        kw = {}
        if forced[i] is not None:
            if granularity:
                kw["forced_idx"] = {("step",): forced[i]}
            else:
                names = ("attn", "xattn", "ffn") if wl.cross_len else ("attn", "ffn")
                kw["forced_idx"] = {(l, sname): forced[i][l, si] for l in range(wl.L) for si, sname in enumerate(names)}
        far = max(far, float(np.abs(plain.var_step(x, i, wl.keep[i], **kw) - ref[i]).max()))
    assert far > 3 * MAX_ABS, far
    return worst


def wl_small(hd, cross_len=0, B=2, keep_last=(0.5, 0.4)):
    sides = (1, 2, 3, 4, 6, 9, 13, 16)
    keep = (1.0,) * (len(sides) - len(keep_last)) + tuple(keep_last)
    return I.Workload("x", L=2, C=256, H=256 // hd, B=B, sides=sides, keep=keep, cross_len=cross_len, seed=4242 + hd)


@pytest.mark.parametrize("hd", [64, 128])
@pytest.mark.parametrize("rope,qk", [(True, False), (False, True), (True, True)])
def test_rotary_positions_and_cosine_attention(hd, rope, qk):
    run_both(wl_small(hd), rope_base=100.0 if rope else 0.0, qk=qk)


def test_extras_with_cross_attention_and_step_granularity():
    run_both(wl_small(64, cross_len=16), rope_base=10000.0, qk=True)
    run_both(wl_small(128), granularity=1, rope_base=100.0, qk=True)


def test_extras_at_model_width():
    """Infinity-like head count at full width (C = 2048, 16 heads of 128), one block, three scales."""
    wl = I.Workload("w", L=1, C=2048, H=16, B=2, sides=(4, 12, 20), keep=(1.0, 1.0, 0.4), cross_len=0, seed=77)
    run_both(wl, rope_base=10000.0, qk=True)


@pytest.mark.parametrize("mode", [1, 2])
@pytest.mark.parametrize("granularity", [0, 1])
def test_bilinear_restoration_in_the_step(granularity, mode):
    """interp_mode 1 (bilinear) and 2 (bicubic) through the whole step, both granularities (the per-sublayer caches
    and the step-level fp32 cache), structured maps so that neighbouring cached rows differ."""
    run_both(wl_small(64), granularity=granularity, interp_mode=mode, kind="structured")


def test_bilinear_skipped_step_and_all_options_together():
    run_both(wl_small(64, keep_last=(0.5, 0.0)), interp_mode=1, kind="structured")
    run_both(wl_small(128, cross_len=8), rope_base=100.0, qk=True, interp_mode=1)
    run_both(wl_small(64, keep_last=(0.5, 0.0)), interp_mode=2, kind="structured")


def test_all_options_on_non_square_maps_with_a_partial_batch():
    """Rotary coordinates on rectangular maps (rows and columns scale by different factors towards the last map),
    bicubic restoration, cosine attention, cross-attention, and fewer images than the context was built for."""
    hw = [(1, 1), (2, 3), (3, 5), (5, 8), (7, 12), (10, 17)]
    keep = [1.0, 1.0, 1.0, 1.0, 0.5, 0.3]
    L, C, H, B_max, B = 2, 128, 2, 3, 2
    wl = I.Workload("rect", L=L, C=C, H=H, B=B_max, sides=tuple(h for h, _ in hw), keep=tuple(keep), cross_len=8, seed=79)
    mt = I.model_tensors(wl)
    sharpen_attention(mt, C)
    qk_scale = (6.0 + 8.0 * I.uniform01(5, L * H).reshape(L, H)).astype(np.float32)
    w = dict(oracle_weights(mt)); w["mod"] = w["mod"][:, :B]; w["text"] = w["text"][:B]
    orc = O.VarOracle(L, C, H, hw, cache_step=3, weights=w, B=B, cross_len=8, interp_mode="bicubic", rope_base=50.0, qk_scale=qk_scale)
    cap = sum(O.kept_count(r, h, ww) if r < 1 else h * ww for r, (h, ww) in zip(keep, hw))
    ctx = fv.FvContext(L, C, H, hw, 3, B_max, cap, mt, cross_len=8, device=DEV, rope_base=50.0, interp_mode=2, qk_scale=qk_scale)
    names = ("attn", "xattn", "ffn")
    for i, (h, ww) in enumerate(hw):
        x = I.token_map(600 + i, B, h, ww, C, "structured")
        tr = {}
        ref = orc.var_step(x, i, keep[i], trace=tr)
        forced = None
        if keep[i] < 1.0:
            forced = torch.from_numpy(np.stack([np.stack([tr[(l, s)]["idx"] for s in names]) for l in range(L)]).astype(np.int32)).to(DEV)
        got = ctx.var_step(torch.from_numpy(x).to(DEV), i, keep[i], forced_idx=forced).cpu().numpy()
        err, cos = per_token_errors(got, ref)
        assert err <= MAX_ABS and cos >= MIN_COS, (i, err, cos)
    assert ctx.device_status() == 0
    ctx.close()
