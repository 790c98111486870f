"""Pins for the CPU oracle: each oracle function is checked against something other than itself
(closed forms, brute force on tiny inputs, invariants the paper states, a different library's
routine for the special cases that reduce to one).  CPU only."""
import itertools
import math
import os
from fractions import Fraction

import numpy as np
import pytest
import torch
import torch.nn.functional as F

from oracle import fastvar_oracle as O
from paper_2503_23367_b200 import inputs as I
from tests.helpers import oracle_weights

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")
rng = np.random.default_rng(1234)


# ------------------------------------------------------------------ kept count
def test_kept_count_golden_table():
    rows = [l.split() for l in open(os.path.join(GOLDEN, "kept_counts.txt")) if l.strip() and l[0] != "#"]
    assert len(rows) == 13
    for side, num, den, k in rows:
        side, num, den, k = int(side), int(num), int(den), int(k)
        assert O.kept_count(num / den, side, side) == k
        # exact rational ceil, independent of floating point
        assert math.ceil(Fraction(num, den) * side * side) == k


def test_kept_count_edges():
    assert O.kept_count(1.0, 7, 5) == 35
    assert O.kept_count(1e-6, 7, 5) == 1          # never empty
    assert O.kept_count(0.5, 1, 1) == 1
    for n_side in range(1, 40):
        for r in (0.1, 0.2, 0.25, 0.4, 0.5, 0.6, 0.75, 0.9):
            k = O.kept_count(r, n_side, n_side + 1)
            n = n_side * (n_side + 1)
            assert 1 <= k <= n
            assert k == max(1, math.ceil(Fraction(str(r)) * n))


# ------------------------------------------------------------------ PTS mean / score
def test_pts_mean_is_spatial_global_average_pool():
    # Algorithm 1: rearrange 'b (h w) c -> b c h w', adaptive_avg_pool2d(., (1,1))
    B, h, w, C = 2, 5, 7, 6
    x = rng.standard_normal((B, h * w, C))
    xt = torch.from_numpy(x).reshape(B, h, w, C).permute(0, 3, 1, 2)
    pooled = F.adaptive_avg_pool2d(xt, (1, 1)).reshape(B, C).numpy()
    np.testing.assert_allclose(O.pts_mean(x), pooled, rtol=1e-13, atol=1e-13)


def test_pts_score_brute_force_tiny():
    B, n, C = 2, 9, 4
    x = rng.standard_normal((B, n, C))
    s = O.pts_score(x)
    for b in range(B):
        mean = [sum(x[b, t, c] for t in range(n)) / n for c in range(C)]
        for t in range(n):
            ref = sum((x[b, t, c] - mean[c]) ** 2 for c in range(C))
            assert abs(s[b, t] - ref) < 1e-12


def test_pts_score_closed_forms():
    B, n, C = 3, 64, 16
    x = rng.standard_normal((B, n, C))
    s = O.pts_score(x)
    assert (s >= 0).all()
    # translation invariance: adding a constant token to every token changes nothing
    shift = rng.standard_normal((B, 1, C)) * 5
    np.testing.assert_allclose(O.pts_score(x + shift), s, rtol=1e-10, atol=1e-10)
    # sum_n s_n = sum_n |x_n|^2 - n |mean|^2
    lhs = s.sum(axis=1)
    rhs = (x ** 2).sum(axis=(1, 2)) - n * (x.mean(axis=1) ** 2).sum(axis=1)
    np.testing.assert_allclose(lhs, rhs, rtol=1e-11)
    # images are independent: scoring image 1 alone gives the same scores
    np.testing.assert_allclose(O.pts_score(x[1:2]), s[1:2], rtol=1e-13)
    # square of the Eq. 5 L2 norm
    l2 = np.linalg.norm(x - x.mean(axis=1, keepdims=True), axis=2)
    np.testing.assert_allclose(np.sqrt(s), l2, rtol=1e-12)


def test_pts_score_single_outlier_ranks_first():
    x = np.ones((1, 25, 8))
    x[0, 17, 3] = 4.0
    s = O.pts_score(x)
    assert int(np.argmax(s[0])) == 17
    assert O.pts_topk(s, 1)[0, 0] == 17
    # the flat tokens all share one (small) score
    others = np.delete(s[0], 17)
    assert np.allclose(others, others[0]) and others[0] < s[0, 17]


# ------------------------------------------------------------------ top-k
def _brute_topk(scores, k):
    order = sorted(range(len(scores)), key=lambda i: (-scores[i], i))
    return sorted(order[:k])


@pytest.mark.parametrize("kind", ["random", "all_equal", "two_valued", "one_outlier", "many_ties"])
def test_pts_topk_vs_brute_force(kind):
    for n in (1, 2, 7, 16, 33, 64):
        if kind == "random":
            s = rng.standard_normal((2, n)) ** 2
        elif kind == "all_equal":
            s = np.full((2, n), 3.25)
        elif kind == "two_valued":
            s = rng.integers(0, 2, size=(2, n)).astype(np.float64)
        elif kind == "one_outlier":
            s = np.zeros((2, n)); s[:, n // 2] = 9.0
        else:
            s = rng.integers(0, 4, size=(2, n)).astype(np.float64)
        for k in sorted({1, max(1, n // 3), max(1, n // 2), n}):
            got = O.pts_topk(s, k)
            for b in range(2):
                assert list(got[b]) == _brute_topk(list(s[b]), k)
                assert len(set(got[b])) == k
                assert all(got[b][i] < got[b][i + 1] for i in range(k - 1))


def test_pts_topk_constant_map_takes_lowest_indices():
    x = np.full((2, 36, 8), 0.7)
    idx, s, kept = O.pivotal_token_selection(x, 6, 6, 0.5)
    assert idx.shape == (2, 18)
    assert (idx == np.arange(18)[None, :]).all()
    assert np.array_equal(kept, x[:, :18])


def test_pts_topk_matches_library_topk_without_ties():
    s = rng.standard_normal((3, 200)) ** 2
    got = O.pts_topk(s, 50)
    lib = torch.topk(torch.from_numpy(s), 50, dim=1).indices.numpy()
    for b in range(3):
        assert set(got[b]) == set(lib[b])


def test_inverse_map_properties():
    s = rng.standard_normal((2, 40)) ** 2
    idx = O.pts_topk(s, 13)
    inv = O.inverse_map(idx, 40)
    for b in range(2):
        assert (inv[b] >= 0).sum() == 13
        for j, t in enumerate(idx[b]):
            assert inv[b, t] == j
        assert (inv[b][np.setdiff1d(np.arange(40), idx[b])] == -1).all()


def test_selection_count_and_gather():
    x = rng.standard_normal((2, 13 * 13, 8))
    idx, s, kept = O.pivotal_token_selection(x, 13, 13, 0.6)
    assert idx.shape == (2, 102)                      # ceil(0.6 * 169)
    for b in range(2):
        assert np.array_equal(kept[b], x[b, idx[b]])  # bit-exact rows
        assert s[b, idx[b]].min() >= np.delete(s[b], idx[b]).max()


# ------------------------------------------------------------------ CTR
@pytest.mark.parametrize("hc,wc,h,w", [(3, 3, 3, 3), (2, 3, 4, 6), (10, 10, 13, 13), (10, 10, 16, 16),
                                       (5, 7, 9, 8), (1, 1, 4, 5), (13, 13, 32, 32), (4, 4, 3, 2)])
def test_upsample_vs_library_nearest(hc, wc, h, w):
    B, C = 2, 3
    cache = rng.standard_normal((B, hc * wc, C))
    got = O.ctr_upsample(cache, hc, wc, h, w)
    t = torch.from_numpy(cache).reshape(B, hc, wc, C).permute(0, 3, 1, 2)
    lib = F.interpolate(t, size=(h, w), mode="nearest").permute(0, 2, 3, 1).reshape(B, h * w, C).numpy()
    assert np.array_equal(got, lib)


def test_upsample_identity_and_integer_factor():
    B, hc, wc, C = 1, 3, 4, 2
    cache = rng.standard_normal((B, hc * wc, C))
    assert np.array_equal(O.ctr_upsample(cache, hc, wc, hc, wc), cache)
    f = 3
    grid = cache.reshape(B, hc, wc, C)
    rep = np.repeat(np.repeat(grid, f, axis=1), f, axis=2).reshape(B, hc * f * wc * f, C)
    assert np.array_equal(O.ctr_upsample(cache, hc, wc, hc * f, wc * f), rep)


def test_restoration_invariants_and_scatter_form():
    B, hc, wc, h, w, C, k = 2, 4, 4, 6, 6, 5, 11
    cache = rng.standard_normal((B, hc * wc, C))
    piv = rng.standard_normal((B, k, C))
    idx = np.stack([np.sort(rng.choice(h * w, k, replace=False)) for _ in range(B)])
    out = O.cached_token_restoration(piv, idx, cache, hc, wc, h, w)
    assert out.shape == (B, h * w, C)                               # token-count invariance
    up = O.ctr_upsample(cache, hc, wc, h, w)
    for b in range(B):
        rest = np.setdiff1d(np.arange(h * w), idx[b])
        assert np.array_equal(out[b, rest], up[b, rest])            # cache outside the pivot slots
        assert np.array_equal(out[b, idx[b]], piv[b])               # forwarded rows in their slots
    # Algorithm 1 written with the library's interpolate + scatter_
    t = torch.from_numpy(cache).reshape(B, hc, wc, C).permute(0, 3, 1, 2)
    restored = F.interpolate(t, size=(h, w), mode="nearest").permute(0, 2, 3, 1).reshape(B, h * w, C).clone()
    restored.scatter_(1, torch.from_numpy(idx)[:, :, None].expand(B, k, C), torch.from_numpy(piv))
    assert np.array_equal(out, restored.numpy())
    # k = n: nothing is taken from the cache
    full = np.tile(np.arange(h * w), (B, 1))
    y = rng.standard_normal((B, h * w, C))
    assert np.array_equal(O.cached_token_restoration(y, full, cache, hc, wc, h, w), y)


# ------------------------------------------------------------------ block pieces
def test_layernorm_vs_library_and_moments():
    x = rng.standard_normal((4, 7, 32)) * 3 + 1.5
    got = O.layernorm(x)
    lib = F.layer_norm(torch.from_numpy(x), (32,), eps=1e-6).numpy()
    np.testing.assert_allclose(got, lib, rtol=1e-12, atol=1e-12)
    np.testing.assert_allclose(got.mean(-1), 0, atol=1e-12)
    np.testing.assert_allclose(got.var(-1), 1, atol=1e-5)


def test_modulate_identity_and_values():
    a = rng.standard_normal((2, 3, 4))
    z = np.zeros((2, 4))
    assert np.array_equal(O.modulate(a, z, z), a)
    sig, beta = rng.standard_normal((2, 4)), rng.standard_normal((2, 4))
    got = O.modulate(a, sig, beta)
    for b, j, c in itertools.product(range(2), range(3), range(4)):
        assert abs(got[b, j, c] - (a[b, j, c] * (1 + sig[b, c]) + beta[b, c])) < 1e-15


def test_gelu_tanh_vs_library_and_identities():
    x = np.linspace(-6, 6, 241)
    got = O.gelu_tanh(x)
    lib = F.gelu(torch.from_numpy(x), approximate="tanh").numpy()
    np.testing.assert_allclose(got, lib, rtol=1e-12, atol=1e-14)
    assert O.gelu_tanh(np.array([0.0]))[0] == 0.0
    np.testing.assert_allclose(got - O.gelu_tanh(-x), x, atol=1e-12)   # gelu(x) - gelu(-x) = x


def test_linear_brute_force_and_orientation():
    a = rng.standard_normal((3, 5)); W = rng.standard_normal((4, 5)); b = rng.standard_normal(4)
    got = O.linear(a, W, b)
    assert got.shape == (3, 4)                                          # W is [out, in]
    for i, o in itertools.product(range(3), range(4)):
        assert abs(got[i, o] - (sum(a[i, c] * W[o, c] for c in range(5)) + b[o])) < 1e-13
    np.testing.assert_allclose(O.linear(a, np.eye(5)), a, atol=0)
    np.testing.assert_allclose(got, F.linear(torch.from_numpy(a), torch.from_numpy(W), torch.from_numpy(b)).numpy(),
                               rtol=1e-13, atol=1e-13)


def test_attention_special_cases_and_library():
    H, hd, k, Lkv = 3, 8, 5, 11
    C = H * hd
    q = rng.standard_normal((k, C)); K = rng.standard_normal((Lkv, C)); V = rng.standard_normal((Lkv, C))
    got = O.attention(q, K, V, H)
    # one key: output is that key's value
    np.testing.assert_allclose(O.attention(q, K[:1], V[:1], H), np.tile(V[:1], (k, 1)), atol=1e-13)
    # identical keys: uniform weights -> mean of V
    Ksame = np.tile(K[:1], (Lkv, 1))
    np.testing.assert_allclose(O.attention(q, Ksame, V, H), np.tile(V.mean(0), (k, 1)), atol=1e-12)
    # key order does not matter
    perm = rng.permutation(Lkv)
    np.testing.assert_allclose(O.attention(q, K[perm], V[perm], H), got, atol=1e-12)
    # library scaled-dot-product attention, head by head (default scale 1/sqrt(hd))
    qt = torch.from_numpy(q).reshape(k, H, hd).transpose(0, 1)
    Kt = torch.from_numpy(K).reshape(Lkv, H, hd).transpose(0, 1)
    Vt = torch.from_numpy(V).reshape(Lkv, H, hd).transpose(0, 1)
    lib = F.scaled_dot_product_attention(qt, Kt, Vt).transpose(0, 1).reshape(k, C).numpy()
    np.testing.assert_allclose(got, lib, rtol=1e-11, atol=1e-12)


# ------------------------------------------------------------------ whole step
def _tiny_model(L=2, C=32, H=4, B=2, sides=(1, 2, 3, 4, 6), cross_len=0, seed=7):
    wl = I.Workload("t", L=L, C=C, H=H, B=B, sides=tuple(sides), keep=(1.0,) * len(sides),
                    cross_len=cross_len, seed=seed)
    mt = I.model_tensors(wl, w_std=0.15)
    return wl, mt, oracle_weights(mt)


def _torch_block_causal_forward(wl, w, xs):
    """Unpruned multi-scale forward as ONE sequence with a block-causal mask, from library ops
    (F.layer_norm, F.linear, F.scaled_dot_product_attention, F.gelu): what a KV cache must reproduce."""
    T = lambda a: torch.from_numpy(np.asarray(a, dtype=np.float64))
    x = torch.cat([T(a) for a in xs], dim=1)                    # [B, N, C]
    B, N, C = x.shape
    lens = [a.shape[1] for a in xs]
    scale_of = torch.repeat_interleave(torch.arange(len(lens)), torch.tensor(lens))
    mask = scale_of[:, None] >= scale_of[None, :]               # query may see keys of its own and earlier scales
    H, hd = wl.H, wl.C // wl.H
    for l in range(wl.L):
        mod = T(w["mod"][l])
        a = F.layer_norm(x, (C,), eps=1e-6) * (1 + mod[:, 0:1]) + mod[:, 1:2]
        qkv = F.linear(a, T(w["w_qkv"][l]), T(w["b_qkv"][l]))
        q, k, v = [t.reshape(B, N, H, hd).transpose(1, 2) for t in qkv.split(C, dim=-1)]
        o = F.scaled_dot_product_attention(q, k, v, attn_mask=mask).transpose(1, 2).reshape(B, N, C)
        x = x + mod[:, 2:3] * F.linear(o, T(w["w_o"][l]), T(w["b_o"][l]))
        if wl.cross_len:
            a = F.layer_norm(x, (C,), eps=1e-6)
            q = F.linear(a, T(w["w_q_x"][l])).reshape(B, N, H, hd).transpose(1, 2)
            kv = F.linear(T(w["text"]), T(w["w_kv_x"][l]))
            kx = kv[..., :C].reshape(B, -1, H, hd).transpose(1, 2)
            vx = kv[..., C:].reshape(B, -1, H, hd).transpose(1, 2)
            o = F.scaled_dot_product_attention(q, kx, vx).transpose(1, 2).reshape(B, N, C)
            x = x + F.linear(o, T(w["w_o_x"][l]))
        a = F.layer_norm(x, (C,), eps=1e-6) * (1 + mod[:, 3:4]) + mod[:, 4:5]
        hmid = F.gelu(F.linear(a, T(w["w_fc1"][l]), T(w["b_fc1"][l])), approximate="tanh")
        x = x + mod[:, 5:6] * F.linear(hmid, T(w["w_fc2"][l]), T(w["b_fc2"][l]))
    return [t.numpy() for t in x.split(lens, dim=1)]


@pytest.mark.parametrize("cross_len", [0, 5])
def test_unpruned_schedule_equals_block_causal_sequence_forward(cross_len):
    wl, mt, w = _tiny_model(cross_len=cross_len)
    xs = [I.step_input(wl, s) for s in range(len(wl.sides))]
    orc = O.VarOracle(wl.L, wl.C, wl.H, [(s, s) for s in wl.sides], cache_step=2, weights=w, B=wl.B,
                      cross_len=cross_len)
    outs = orc.run_schedule(xs, wl.keep)
    ref = _torch_block_causal_forward(wl, w, xs)
    for a, b in zip(outs, ref):
        np.testing.assert_allclose(a, b, rtol=1e-9, atol=1e-10)
    assert orc.kv_len == sum(s * s for s in wl.sides)


def _run(wl, w, xs, keep, cache_step, granularity="sublayer", **kw):
    orc = O.VarOracle(wl.L, wl.C, wl.H, [(s, s) for s in wl.sides], cache_step=cache_step, weights=w,
                      B=wl.B, cross_len=wl.cross_len, granularity=granularity)
    outs, traces = [], []
    for i, x in enumerate(xs):
        tr = {}
        outs.append(orc.var_step(x, i, keep[i], trace=tr, **(kw if keep[i] < 1 else {})))
        traces.append(tr)
    return orc, outs, traces


@pytest.mark.parametrize("cross_len", [0, 4])
def test_keeping_every_token_through_pts_ctr_equals_unpruned(cross_len):
    """keep_ratio -> 1: selection keeps all n tokens, gather is the identity, restoration takes
    nothing from the cache; the pruned code path must reproduce the unpruned forward."""
    wl, mt, w = _tiny_model(cross_len=cross_len)
    xs = [I.step_input(wl, s) for s in range(len(wl.sides))]
    _, ref, _ = _run(wl, w, xs, [1.0] * 5, cache_step=2)
    almost = 1.0 - 1e-7                                            # < 1 so PTS/CTR run; ceil gives k = n
    assert O.kept_count(almost, 6, 6) == 36
    _, got, tr = _run(wl, w, xs, [1.0, 1.0, 1.0, almost, almost], cache_step=2)
    for a, b in zip(got, ref):
        np.testing.assert_allclose(a, b, rtol=1e-11, atol=1e-12)
    assert (tr[4][(0, "attn")]["idx"] == np.arange(36)).all()


def test_pruned_step_bookkeeping_and_cache_outside_pivots():
    wl, mt, w = _tiny_model(L=1)
    xs = [I.step_input(wl, s) for s in range(len(wl.sides))]
    keep = [1.0, 1.0, 1.0, 0.5, 0.25]
    orc, outs, tr = _run(wl, w, xs, keep, cache_step=2)
    ks = [1, 4, 9, 8, 9]
    assert orc.kv_len == sum(ks)                                   # only pivotal K/V enter the cache
    for b in range(wl.B):
        assert orc.Kc[0][b].shape[0] == sum(ks)
    assert outs[4].shape == xs[4].shape                            # token-count invariance
    # rows pruned in BOTH sublayers moved by exactly gamma1*cache_attn[src] + gamma2*cache_ffn[src]
    h = wl.sides[4]; hc = wl.sides[2]
    src = O.nearest_source(h, h, hc, hc)
    mod = w["mod"][0]
    ia, iff = tr[4][(0, "attn")]["idx"], tr[4][(0, "ffn")]["idx"]
    assert ia.shape == (wl.B, 9)
    for b in range(wl.B):
        rest = np.setdiff1d(np.arange(h * h), np.union1d(ia[b], iff[b]))
        assert len(rest) > 0
        want = xs[4][b, rest].astype(np.float64) + mod[b, 2] * orc.cache[0]["attn"][b, src[rest]] \
            + mod[b, 5] * orc.cache[0]["ffn"][b, src[rest]]
        np.testing.assert_allclose(outs[4][b, rest], want, rtol=1e-12, atol=1e-12)
    # the cache is the unpruned step-2 branch output and is never refreshed
    _, _, tr_ref = _run(wl, w, xs[:3], [1.0] * 3, cache_step=2)
    np.testing.assert_array_equal(orc.cache[0]["attn"], tr_ref[2][(0, "attn")]["y"])


def test_emission_order_of_the_index_set_does_not_matter():
    wl, mt, w = _tiny_model(L=2)
    xs = [I.step_input(wl, s) for s in range(len(wl.sides))]
    keep = [1.0, 1.0, 1.0, 1.0, 0.5]
    _, ref, tr = _run(wl, w, xs, keep, cache_step=3)
    forced = {}
    for key, t in tr[4].items():                                   # same sets, in descending-score order
        forced[key] = np.stack([t["idx"][b][np.argsort(-t["score"][b][t["idx"][b]], kind="stable")]
                                for b in range(wl.B)])
    _, got, _ = _run(wl, w, xs, keep, cache_step=3, forced_idx=forced)
    np.testing.assert_allclose(got[4], ref[4], rtol=1e-10, atol=1e-11)


@pytest.mark.parametrize("cross_len", [0, 4])
def test_pruned_steps_with_one_kept_set_equal_a_sequence_forward_over_the_kept_tokens(cross_len):
    """With the same kept set at every sublayer of a pruned step the kept tokens never meet the others: they
    see the keys of the earlier scales (at a pruned earlier step: of its kept tokens only, Sec. 3.3) and their
    own, so their outputs are those of a library block-causal forward over the sequence
    [x_1 ... x_{K-N} ; kept tokens of every pruned step].  Every other token moves by the gated sum of the
    cached sublayer outputs of its source token (Eq. 6)."""
    wl, mt, w = _tiny_model(cross_len=cross_len)
    xs = [I.step_input(wl, s) for s in range(len(wl.sides))]
    keep = [1.0, 1.0, 1.0, 0.5, 0.25]
    orc = O.VarOracle(wl.L, wl.C, wl.H, [(s, s) for s in wl.sides], cache_step=2, weights=w, B=wl.B,
                      cross_len=cross_len)
    pick = np.random.default_rng(77)
    kept, outs = {}, []
    for i, x in enumerate(xs):
        if keep[i] < 1:
            n = wl.sides[i] ** 2
            k = O.kept_count(keep[i], wl.sides[i], wl.sides[i])
            kept[i] = np.stack([np.sort(pick.choice(n, size=k, replace=False)) for _ in range(wl.B)])
            outs.append(orc.var_step(x, i, keep[i], forced_idx={(l, sub): kept[i] for l in range(wl.L) for sub in orc.subs}))
        else:
            outs.append(orc.var_step(x, i, 1.0))
    compact = [x if i not in kept else np.stack([x[b, kept[i][b]] for b in range(wl.B)]) for i, x in enumerate(xs)]
    ref = _torch_block_causal_forward(wl, w, compact)
    gate = {"attn": 2, "ffn": 5}
    for i in kept:
        side, side_c = wl.sides[i], wl.sides[2]
        src = O.nearest_source(side, side, side_c, side_c)
        for b in range(wl.B):
            np.testing.assert_allclose(outs[i][b, kept[i][b]], ref[i][b], rtol=1e-9, atol=1e-10)
            rest = np.setdiff1d(np.arange(side * side), kept[i][b])
            want = xs[i][b, rest].astype(np.float64)
            for l in range(wl.L):
                for sub in orc.subs:
                    g = w["mod"][l][b, gate[sub]] if sub in gate else 1.0
                    want = want + g * orc.cache[l][sub][b, src[rest]]
            np.testing.assert_allclose(outs[i][b, rest], want, rtol=1e-12, atol=1e-12)
    assert orc.kv_len == 1 + 4 + 9 + kept[3].shape[1] + kept[4].shape[1]


def test_free_running_selections_are_taken_on_the_current_stream():
    """Every wrapped sublayer selects on the token map as the sublayers before it left it (Sec. 3.3
    "Implementation"): replaying the trace -- brute-force ranking of the deviation from the mean token by a
    stable sort, the branch output scattered over the interpolated cache -- reproduces each recorded kept set
    and the step's output."""
    wl, mt, w = _tiny_model(L=2, cross_len=3)
    xs = [I.step_input(wl, s) for s in range(len(wl.sides))]
    keep = [1.0, 1.0, 1.0, 0.5, 0.25]
    orc, outs, tr = _run(wl, w, xs, keep, cache_step=2)
    gate = {"attn": 2, "ffn": 5}
    for i in (3, 4):
        side, side_c = wl.sides[i], wl.sides[2]
        k = O.kept_count(keep[i], side, side)
        src = O.nearest_source(side, side, side_c, side_c)
        x = xs[i].astype(np.float64).copy()
        for l in range(wl.L):
            for sub in orc.subs:
                t = tr[i][(l, sub)]
                for b in range(wl.B):
                    dev = x[b] - x[b].sum(axis=0) / x.shape[1]
                    order = sorted(range(x.shape[1]), key=lambda j: -float((dev[j] * dev[j]).sum()))   # stable: ties keep index order
                    assert sorted(order[:k]) == list(t["idx"][b])
                    full = orc.cache[l][sub][b, src].copy()
                    full[t["idx"][b]] = t["y"][b]
                    g = w["mod"][l][b, gate[sub]] if sub in gate else 1.0
                    x[b] = x[b] + g * full
        np.testing.assert_allclose(outs[i], x, rtol=1e-12, atol=1e-12)


def test_images_are_independent():
    wl, mt, w = _tiny_model(L=1, B=2)
    xs = [I.step_input(wl, s) for s in range(len(wl.sides))]
    keep = [1.0, 1.0, 1.0, 0.5, 0.5]
    _, both, _ = _run(wl, w, xs, keep, cache_step=2)
    wl1 = I.Workload("t1", L=1, C=wl.C, H=wl.H, B=1, sides=wl.sides, keep=wl.keep, seed=wl.seed)
    w1 = dict(w); w1["mod"] = w["mod"][:, 1:2]
    _, one, _ = _run(wl1, w1, [x[1:2] for x in xs], keep, cache_step=2)
    np.testing.assert_allclose(both[4][1:2], one[4], rtol=1e-12, atol=1e-13)


# ------------------------------------------------------------------ per-step granularity (the coarser variant)
@pytest.mark.parametrize("cross_len", [0, 4])
def test_step_granularity_unpruned_and_keep_all_equal_the_unpruned_forward(cross_len):
    wl, mt, w = _tiny_model(cross_len=cross_len)
    xs = [I.step_input(wl, s) for s in range(len(wl.sides))]
    _, ref, _ = _run(wl, w, xs, [1.0] * 5, cache_step=2)                      # paper granularity, unpruned
    _, got, _ = _run(wl, w, xs, [1.0] * 5, cache_step=2, granularity="step")
    for a, b in zip(got, ref):
        np.testing.assert_array_equal(a, b)                                   # no pruning: the same arithmetic
    almost = 1.0 - 1e-7                                                       # PTS / CTR run, k = n
    _, got, tr = _run(wl, w, xs, [1.0, 1.0, 1.0, almost, almost], cache_step=2, granularity="step")
    for a, b in zip(got, ref):
        np.testing.assert_allclose(a, b, rtol=1e-11, atol=1e-12)
    assert (tr[4][("step",)]["idx"] == np.arange(36)).all()


def test_step_granularity_pivot_rows_and_restored_rows():
    """Kept rows: the blocks only ever see the compact rows, so with the SAME index set forced on every
    sublayer the paper-granularity oracle must give the same values on those rows.  Other rows: exactly
    the cached output map of step K-N, nearest-upsampled.  KV cache: k rows per pruned step."""
    wl, mt, w = _tiny_model(L=2, cross_len=3)
    xs = [I.step_input(wl, s) for s in range(len(wl.sides))]
    keep = [1.0, 1.0, 1.0, 0.5, 0.25]
    orc, outs, tr = _run(wl, w, xs, keep, cache_step=2, granularity="step")
    assert orc.kv_len == 1 + 4 + 9 + 8 + 9
    np.testing.assert_array_equal(orc.step_cache, outs[2])                    # the cache is step 2's output map
    h, hc = wl.sides[4], wl.sides[2]
    src = O.nearest_source(h, h, hc, hc)
    idx = tr[4][("step",)]["idx"]
    assert idx.shape == (wl.B, 9) and (np.diff(idx, axis=1) > 0).all()
    np.testing.assert_array_equal(idx, O.pts_topk(O.pts_score(xs[4]), 9))     # selected on the step input
    for b in range(wl.B):
        rest = np.setdiff1d(np.arange(h * h), idx[b])
        np.testing.assert_array_equal(outs[4][b, rest], outs[2][b, src[rest]])
    # same sets forced on every sublayer of the paper-granularity oracle, steps 3 and 4
    forced3 = {(l, s): tr[3][("step",)]["idx"] for l in range(wl.L) for s in ("attn", "xattn", "ffn")}
    forced4 = {(l, s): idx for l in range(wl.L) for s in ("attn", "xattn", "ffn")}
    ref = O.VarOracle(wl.L, wl.C, wl.H, [(s, s) for s in wl.sides], cache_step=2, weights=w, B=wl.B, cross_len=wl.cross_len)
    for i in range(3):
        ref.var_step(xs[i], i, 1.0)
    ref.var_step(xs[3], 3, keep[3], forced_idx=forced3)
    out4 = ref.var_step(xs[4], 4, keep[4], forced_idx=forced4)
    for b in range(wl.B):
        np.testing.assert_allclose(outs[4][b, idx[b]], out4[b, idx[b]], rtol=1e-11, atol=1e-12)


@pytest.mark.parametrize("granularity", ["sublayer", "step"])
def test_skipped_step_is_the_interpolated_output_of_the_caching_step(granularity):
    """keep_ratio = 0 (the paper's 100 % pruning ratio): no token is forwarded, the step's output is the
    nearest-neighbour interpolation of the caching step's output map (checked against the library's
    interpolate), the KV cache does not grow, and a later step still runs."""
    wl, mt, w = _tiny_model(L=1)
    xs = [I.step_input(wl, s) for s in range(len(wl.sides))]
    orc, outs, _ = _run(wl, w, xs, [1.0, 1.0, 1.0, 0.0, 0.5], cache_step=2, granularity=granularity)
    hc, h = wl.sides[2], wl.sides[3]
    t = torch.from_numpy(outs[2]).reshape(wl.B, hc, hc, wl.C).permute(0, 3, 1, 2)
    up = F.interpolate(t, size=(h, h), mode="nearest").permute(0, 2, 3, 1).reshape(wl.B, h * h, wl.C).numpy()
    np.testing.assert_array_equal(outs[3], up)
    assert orc.kv_len == 1 + 4 + 9 + 0 + 18 and orc.step == 5
    assert outs[4].shape == xs[4].shape


def test_step_granularity_images_are_independent():
    wl, mt, w = _tiny_model(L=1, B=2)
    xs = [I.step_input(wl, s) for s in range(len(wl.sides))]
    keep = [1.0, 1.0, 1.0, 0.5, 0.5]
    _, both, _ = _run(wl, w, xs, keep, cache_step=2, granularity="step")
    wl1 = I.Workload("t1", L=1, C=wl.C, H=wl.H, B=1, sides=wl.sides, keep=wl.keep, seed=wl.seed)
    w1 = dict(w); w1["mod"] = w["mod"][:, 1:2]
    _, one, _ = _run(wl1, w1, [x[1:2] for x in xs], keep, cache_step=2, granularity="step")
    np.testing.assert_allclose(both[4][1:2], one[4], rtol=1e-12, atol=1e-13)


# ------------------------------------------------------------------ input generator
def test_generator_is_counter_based_and_normal():
    a = I.normal(11, (1000, 33))
    b = I.normal(11, (1000, 33), chunk=977)
    assert np.array_equal(a, b)                                    # independent of chunking
    assert abs(a.mean()) < 0.02 and abs(a.std() - 1) < 0.02
    assert not np.array_equal(a, I.normal(12, (1000, 33)))


def test_bf16_rounding_matches_library():
    a = I.normal(5, (4096,), 3.0)
    bits = I.to_bf16_bits(a)
    lib = torch.from_numpy(a).to(torch.bfloat16)
    assert np.array_equal(bits, lib.view(torch.int16).numpy().view(np.uint16))
    assert np.array_equal(I.bf16_bits_to_f32(bits), lib.to(torch.float32).numpy())
