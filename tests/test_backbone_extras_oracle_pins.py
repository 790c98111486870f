"""Pins for the optional backbone pieces of the oracle (bilinear restoration, cosine attention, 2-D rotary
positions by original token index): library special cases, closed forms and invariants, none of them a
retyping of the oracle's own formula."""
import numpy as np
import pytest
import torch
import torch.nn.functional as F

from oracle import fastvar_oracle as O
from paper_2503_23367_b200 import inputs as I
from helpers import oracle_weights


@pytest.mark.parametrize("hc,wc,h,w", [(2, 2, 4, 4), (3, 5, 7, 8), (4, 4, 4, 4), (5, 3, 6, 9), (1, 1, 3, 2), (6, 6, 4, 3)])
def test_bilinear_restoration_equals_library_resize(hc, wc, h, w):
    rng = np.random.default_rng(hc * 100 + w)
    cache = rng.standard_normal((2, hc * wc, 5))
    got = O.ctr_upsample_bilinear(cache, hc, wc, h, w)
    t = torch.from_numpy(cache).reshape(2, hc, wc, 5).permute(0, 3, 1, 2)
    lib = F.interpolate(t, size=(h, w), mode="bilinear", align_corners=False).permute(0, 2, 3, 1).reshape(2, h * w, 5).numpy()
    np.testing.assert_allclose(got, lib, rtol=1e-12, atol=1e-12)
    # a map that is linear in (y, x) is reproduced exactly inside the sample hull; constant maps everywhere
    np.testing.assert_allclose(O.ctr_upsample_bilinear(np.full((1, hc * wc, 1), 3.5), hc, wc, h, w), 3.5, atol=1e-12)


@pytest.mark.parametrize("hc,wc,h,w", [(2, 2, 4, 4), (3, 5, 7, 8), (4, 4, 4, 4), (5, 3, 6, 9), (1, 1, 3, 2), (6, 6, 4, 3), (8, 8, 16, 12)])
def test_bicubic_restoration_equals_library_resize(hc, wc, h, w):
    rng = np.random.default_rng(hc * 10 + w)
    cache = rng.standard_normal((2, hc * wc, 3))
    got = O.ctr_upsample_bicubic(cache, hc, wc, h, w)
    t = torch.from_numpy(cache).reshape(2, hc, wc, 3).permute(0, 3, 1, 2)
    lib = F.interpolate(t, size=(h, w), mode="bicubic", align_corners=False).permute(0, 2, 3, 1).reshape(2, h * w, 3).numpy()
    np.testing.assert_allclose(got, lib, rtol=1e-11, atol=1e-11)
    # the four weights of a tap set sum to one: a constant map stays constant
    np.testing.assert_allclose(O.ctr_upsample_bicubic(np.full((1, hc * wc, 1), -2.25), hc, wc, h, w), -2.25, atol=1e-12)
    idx, wt = O.bicubic_taps(h, hc)
    np.testing.assert_allclose(wt.sum(1), 1.0, atol=1e-12)


def test_bilinear_restoration_keeps_pivots_and_blends_elsewhere():
    rng = np.random.default_rng(3)
    cache = rng.standard_normal((1, 4, 3)); piv = rng.standard_normal((1, 2, 3)); idx = np.array([[1, 14]])
    out = O.cached_token_restoration(piv, idx, cache, 2, 2, 4, 4, "bilinear")
    np.testing.assert_array_equal(out[0, [1, 14]], piv[0])
    up = O.ctr_upsample_bilinear(cache, 2, 2, 4, 4)
    rest = np.setdiff1d(np.arange(16), idx[0])
    np.testing.assert_array_equal(out[0, rest], up[0, rest])


def test_qk_normalise_is_cosine_similarity():
    rng = np.random.default_rng(4)
    H, hd, k = 3, 8, 5
    q, kk = rng.standard_normal((k, H * hd)) * 4, rng.standard_normal((k, H * hd)) * 0.1
    s = np.array([2.0, 0.5, 7.0])
    qn, kn = O.qk_normalise(q, H, s), O.qk_normalise(kk, H)
    for h in range(H):
        sl = slice(h * hd, (h + 1) * hd)
        np.testing.assert_allclose(np.linalg.norm(kn[:, sl], axis=1), 1.0, atol=1e-12)
        cos = F.cosine_similarity(torch.from_numpy(q[:, None, sl]), torch.from_numpy(kk[None, :, sl]), dim=-1).numpy()
        np.testing.assert_allclose(qn[:, sl] @ kn[:, sl].T, s[h] * cos, atol=1e-12)
    assert np.all(np.isfinite(O.qk_normalise(np.zeros((1, H * hd)), H)))       # zero vector: floored norm


def test_rope_is_complex_multiplication_and_keeps_norms():
    rng = np.random.default_rng(5)
    H, hd, k = 2, 16, 7
    v = rng.standard_normal((k, H * hd))
    tok = np.array([0, 1, 5, 6, 11, 17, 19])
    ang = O.rope_angles(tok, 4, 5, 8, 10, hd, 100.0)
    assert ang.shape == (k, hd // 2)
    got = O.apply_rope(v, ang, H)
    z = v.reshape(k, H, hd // 2, 2)
    zc = (z[..., 0] + 1j * z[..., 1]) * np.exp(1j * ang)[:, None, :]
    np.testing.assert_allclose(got.reshape(k, H, hd // 2, 2)[..., 0], zc.real, atol=1e-12)
    np.testing.assert_allclose(got.reshape(k, H, hd // 2, 2)[..., 1], zc.imag, atol=1e-12)
    np.testing.assert_allclose(np.linalg.norm(got, axis=1), np.linalg.norm(v, axis=1), atol=1e-12)
    np.testing.assert_array_equal(got[0], v[0])                                  # token (0,0): no rotation
    # coordinates live in the last scale's frame: token (y,x) of a 4x5 map sits at (2y, 2x) of the 8x10 map
    a2 = O.rope_angles(np.array([2 * 1 * 10 + 2 * 3]), 8, 10, 8, 10, hd, 100.0)  # (y,x) = (2,6) of the last scale
    a1 = O.rope_angles(np.array([1 * 5 + 3]), 4, 5, 8, 10, hd, 100.0)            # (1,3) of the 4x5 map
    np.testing.assert_allclose(a1, a2, atol=1e-12)
    # first half turns with the row, second half with the column, frequencies base^(-j/(hd/4))
    a = O.rope_angles(np.array([3 * 10 + 0, 7]), 8, 10, 8, 10, hd, 100.0)
    np.testing.assert_allclose(a[0, :hd // 4], 3 * 100.0 ** (-np.arange(4) / 4)); np.testing.assert_allclose(a[0, hd // 4:], 0)
    np.testing.assert_allclose(a[1, hd // 4:], 7 * 100.0 ** (-np.arange(4) / 4)); np.testing.assert_allclose(a[1, :hd // 4], 0)


def test_rope_scores_depend_on_position_differences_only():
    rng = np.random.default_rng(6)
    H, hd = 1, 16
    q, kk = rng.standard_normal((1, hd)), rng.standard_normal((1, hd))
    def score(tq, tk):
        aq = O.rope_angles(np.array([tq]), 8, 8, 8, 8, hd, 50.0); ak = O.rope_angles(np.array([tk]), 8, 8, 8, 8, hd, 50.0)
        return (O.apply_rope(q, aq, H) @ O.apply_rope(kk, ak, H).T)[0, 0]
    base = score(1 * 8 + 2, 3 * 8 + 1)
    for dy, dx in ((1, 1), (4, 0), (0, 5), (3, 4)):
        np.testing.assert_allclose(score((1 + dy) * 8 + 2 + dx, (3 + dy) * 8 + 1 + dx), base, atol=1e-12)
    assert abs(score(1 * 8 + 2, 3 * 8 + 2) - base) > 1e-6


def _model(**kw):
    wl = I.Workload("x", L=2, C=32, H=2, B=2, sides=(1, 2, 4, 6), keep=(1.0, 1.0, 1.0, 0.5), cross_len=0, seed=17)
    mt = I.model_tensors(wl, w_std=0.15)
    mk = lambda **k2: O.VarOracle(wl.L, wl.C, wl.H, [(s, s) for s in wl.sides], cache_step=wl.cache_step, weights=oracle_weights(mt),
                                  B=wl.B, **{**kw, **k2})
    xs = [I.step_input(wl, i) for i in range(4)]
    return wl, mk, xs


@pytest.mark.parametrize("granularity", ["sublayer", "step"])
def test_extras_keep_the_method_invariants(granularity):
    """With all three pieces on: keeping every token through the selection / restoration path equals the
    unpruned forward (so the rotation really is by original slot: forcing a permuted kept order must not
    change anything either), and the restored map equals the interpolated cache outside the pivot slots."""
    qk = np.array([[1.5, 0.7], [2.0, 1.0]])
    wl, mk, xs = _model(interp_mode="bilinear", rope_base=100.0, qk_scale=qk, granularity=granularity)
    ref = mk().run_schedule(xs, (1.0, 1.0, 1.0, 1.0))
    all_idx = np.broadcast_to(np.arange(36), (2, 36))
    key = lambda l, s: (("step",) if granularity == "step" else (l, s))
    forced = {key(l, s): all_idx for l in range(2) for s in ("attn", "ffn")}
    o = mk()
    for i in range(3):
        o.var_step(xs[i], i, 1.0)
    np.testing.assert_allclose(o.var_step(xs[3], 3, 0.999999, forced_idx=forced), ref[3], atol=1e-10)
    # the rotary position follows the token, not the row of the compact tensor: a kept set given in another
    # order yields the same map
    idx = np.stack([np.sort(np.random.default_rng(b).permutation(36)[:18]) for b in range(2)])
    perm = np.random.default_rng(9).permutation(18)
    outs = []
    for ix in (idx, idx[:, perm]):
        o = mk()
        for i in range(3):
            o.var_step(xs[i], i, 1.0)
        outs.append(o.var_step(xs[3], 3, 0.5, forced_idx={key(l, s): ix for l in range(2) for s in ("attn", "ffn")}))
    np.testing.assert_allclose(outs[0], outs[1], atol=1e-10)


def test_rope_changes_attention_only_through_positions():
    """rope on, every position at the origin (a 1x1 schedule step) equals rope off; on a real map it differs."""
    wl, mk, xs = _model()
    a = mk().var_step(xs[0], 0, 1.0)
    b = mk(rope_base=100.0).var_step(xs[0], 0, 1.0)
    np.testing.assert_allclose(a, b, atol=1e-12)
    o1, o2 = mk(), mk(rope_base=100.0)
    o1.var_step(xs[0], 0, 1.0); o2.var_step(xs[0], 0, 1.0)
    assert np.abs(o1.var_step(xs[1], 1, 1.0) - o2.var_step(xs[1], 1, 1.0)).max() > 1e-6
