"""Pins for the generation-loop oracle (Sec. 3.1, Eq. 2-3): each function is checked against something
other than itself -- the unfolded form Eq. 3, brute force, a textbook identity, or a special case with a
known answer."""
import numpy as np
import pytest

from oracle import fastvar_oracle as O
from oracle import generation_oracle as G
from paper_2503_23367_b200 import inputs as I


def test_eq2_recursion_equals_eq3_on_nested_scales():
    """Eq. 3 is Eq. 2 unfolded.  With nearest-neighbour interpolation the unfolding is exact when every
    scale divides the next (the floor maps then compose); a wrong interpolation index, a dropped term or an
    accumulation at the wrong scale breaks the equality."""
    rng = np.random.default_rng(0)
    sizes = [(1, 1), (2, 2), (4, 4), (8, 8), (16, 8)]
    V, d, B = 11, 5, 2
    cb = rng.standard_normal((V, d))
    ids = [rng.integers(0, V, size=(B, h * w)) for h, w in sizes]
    fs = [cb[i] for i in ids]
    r = None
    for k, (h, w) in enumerate(sizes):
        hp, wp = sizes[k - 1] if k else (0, 0)
        r = G.residual_accumulate(r, hp, wp, ids[k], cb, h, w)
        np.testing.assert_allclose(r, G.cumulative_form(fs, sizes, k), rtol=0, atol=1e-12)


def test_eq2_is_the_recursive_form_where_the_two_differ():
    """On scales that do not divide each other (1, 2, 3) the floor maps do not compose, so the two forms
    differ; the oracle follows Eq. 2 literally: each step interpolates the previous running map."""
    sizes = [(1, 1), (2, 2), (3, 3)]
    cb = np.eye(4)[:, :3] + np.arange(4)[:, None]
    ids = [np.array([[1]]), np.array([[0, 1, 2, 3]]), np.zeros((1, 9), dtype=np.int64)]
    r1 = G.residual_accumulate(None, 0, 0, ids[0], cb, 1, 1)
    r2 = G.residual_accumulate(r1, 1, 1, ids[1], cb, 2, 2)
    r3 = G.residual_accumulate(r2, 2, 2, ids[2], cb, 3, 3)
    # by hand: token (y, x) of the 3x3 map reads token (floor(2y/3), floor(2x/3)) of the 2x2 map
    for y in range(3):
        for x in range(3):
            src = (2 * y // 3) * 2 + (2 * x // 3)
            np.testing.assert_allclose(r3[0, y * 3 + x], cb[1] + cb[ids[1][0, src]] + cb[0], atol=1e-12)


def test_choose_tokens_brute_force_and_ties():
    rng = np.random.default_rng(1)
    z = rng.integers(-3, 4, size=(2, 7, 9)).astype(np.float64)      # many exact ties
    noise = rng.integers(-1, 2, size=z.shape).astype(np.float64)
    for nz, tau in ((None, 1.0), (noise, 1.0), (noise, 2.0)):
        ids, margin = G.choose_tokens(z, nz, tau)
        for b in range(2):
            for t in range(7):
                row = z[b, t] + (0 if nz is None else tau * nz[b, t])
                best = max(range(9), key=lambda v: (row[v], -v))     # highest value, then lowest id
                assert ids[b, t] == best
                srt = np.sort(row)
                assert margin[b, t] == srt[-1] - srt[-2]


def test_gumbel_noise_makes_the_choice_a_softmax_draw():
    """Gumbel-max identity: argmax(l + tau*g) with standard Gumbel g is distributed as softmax(l / tau)."""
    logits = np.array([1.0, 0.0, -1.0, 2.0])
    tau, n = 1.7, 40000
    g = I.gumbel_noise(123, (1, n, 4)).astype(np.float64)
    ids, _ = G.choose_tokens(np.broadcast_to(logits, (1, n, 4)), g, tau)
    freq = np.bincount(ids[0], minlength=4) / n
    p = np.exp(logits / tau) / np.exp(logits / tau).sum()
    assert np.all(np.abs(freq - p) < 4 * np.sqrt(p * (1 - p) / n))


def test_head_logits_special_cases():
    rng = np.random.default_rng(2)
    B, n, C = 2, 5, 16
    x = rng.standard_normal((B, n, C)) * 3 + 1
    z = np.zeros((B, C))
    # identity head, no modulation: logits are the normalised rows (mean 0, variance 1 up to eps)
    lg = G.head_logits(x, z, z, np.eye(C), None)
    np.testing.assert_allclose(lg.mean(-1), 0, atol=1e-12)
    np.testing.assert_allclose((lg ** 2).mean(-1), 1, atol=1e-5)
    # against library ops
    import torch, torch.nn.functional as F
    W, b = rng.standard_normal((7, C)), rng.standard_normal(7)
    sg, bt = rng.standard_normal((B, C)), rng.standard_normal((B, C))
    T = lambda a: torch.from_numpy(np.asarray(a, dtype=np.float64))
    lib = F.linear(F.layer_norm(T(x), (C,), eps=1e-6) * (1 + T(sg)[:, None]) + T(bt)[:, None], T(W), T(b)).numpy()
    np.testing.assert_allclose(G.head_logits(x, sg, bt, W, b), lib, rtol=1e-11, atol=1e-11)


def test_next_scale_input_special_cases():
    rng = np.random.default_rng(3)
    B, d = 2, 6
    r = rng.standard_normal((B, 1, d))
    # identity map, 1x1 -> 2x3: every token of the next scale is the single source token
    x = G.next_scale_input(r, 1, 1, 2, 3, np.eye(d), None, None)
    assert x.shape == (B, 6, d)
    np.testing.assert_allclose(x, np.broadcast_to(r, (B, 6, d)), atol=0)
    # bias and position embedding are added once each; the map is linear in r
    W, b, pos = rng.standard_normal((4, d)), rng.standard_normal(4), rng.standard_normal((6, 4))
    r22 = rng.standard_normal((B, 4, d))
    full = G.next_scale_input(r22, 2, 2, 2, 3, W, b, pos)
    lin = G.next_scale_input(2 * r22, 2, 2, 2, 3, W, None, None)
    np.testing.assert_allclose(2 * (full - b - pos[None]), lin, atol=1e-12)
    # columns 0,1,2 of the 2x3 map read columns 0,0,1 of the 2x2 map (floor(x*2/3))
    src = [0, 0, 1, 2, 2, 3]
    np.testing.assert_allclose(full, r22[:, src] @ W.T + b + pos[None], atol=1e-12)


def test_generation_loop_is_the_steps_chained():
    """The loop's records obey Eq. 2 step by step and feed each step the map built from the previous record;
    with keep ratio 1 everywhere its transformer outputs equal a plain run of the same inputs."""
    wl = I.Workload("g", L=1, C=32, H=4, B=2, sides=(1, 2, 4), keep=(1.0, 1.0, 1.0), cross_len=0, seed=5)
    mt = I.model_tensors(wl, w_std=0.15)
    gt = I.generation_tensors(wl, V=13, d=6)
    from helpers import oracle_weights
    w = oracle_weights(mt)
    sizes = [(s, s) for s in wl.sides]
    mk = lambda: O.VarOracle(wl.L, wl.C, wl.H, sizes, cache_step=wl.cache_step, weights=w, B=wl.B, cross_len=0)
    gen = G.GenerationOracle(mk(), sizes, gt.codebook, I.bf16_bits_to_f32(gt.w_head), I.bf16_bits_to_f32(gt.b_head),
                             gt.mod_head, gt.w_in, gt.b_in, gt.pos)
    recs = gen.generate(gt.start, wl.keep)
    plain = mk().run_schedule([r["x"] for r in recs], wl.keep)
    for k, rec in enumerate(recs):
        np.testing.assert_allclose(rec["y"], plain[k], atol=1e-12)
        assert rec["ids"].shape == (wl.B, wl.tokens(k)) and rec["ids"].min() >= 0 and rec["ids"].max() < 13
        f = gt.codebook.astype(np.float64)[rec["ids"]]
        prev = 0 if k == 0 else G.interpolate_nearest(recs[k - 1]["r"], *sizes[k - 1], *sizes[k])
        np.testing.assert_allclose(rec["r"], prev + f, atol=1e-12)
