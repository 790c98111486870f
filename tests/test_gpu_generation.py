"""Generation loop around the scale step (Sec. 3.1, Eq. 2-3) through the C ABI against its CPU oracle.

Integer decisions (token ids) are compared where the oracle's own margin (best minus second-best
perturbed logit) exceeds what fp32 / bf16 rounding can move; decisions inside that margin are counted as
near-ties and must stay rare.  Kernel-level tests feed both sides the same seeded inputs; the loop test is
teacher-forced: every GPU stage takes the ORACLE's record of the previous stage as its input."""
import numpy as np
import pytest
import torch

from oracle import fastvar_oracle as O
from oracle import generation_oracle as G
from paper_2503_23367_b200 import binding as fv
from paper_2503_23367_b200 import inputs as I
from tests.helpers import make_oracle, per_token_errors

pytestmark = pytest.mark.gpu
DEV = "cuda:0"
T = lambda a, dt=torch.float32: torch.from_numpy(np.ascontiguousarray(a)).to(DEV, dt)
BF = lambda bits: torch.from_numpy(bits.view("int16")).to(DEV).view(torch.bfloat16).contiguous()


@pytest.mark.parametrize("rows,V", [(1, 4), (7, 64), (300, 4096), (5, 100), (2050, 1000), (8192, 4096)])
@pytest.mark.parametrize("with_noise", [False, True])
def test_argmax_rows_bit_exact(rows, V, with_noise):
    """Same fp32 logits on both sides: ids are bit-exact without noise (pure comparisons, ties to the lowest
    id -- the integer-valued logits below tie often); with noise the perturbed value is one fp32 fma on the GPU
    and exact in the oracle, so a row may differ only if its margin is at rounding level."""
    lg = np.round(I.normal(11 + rows, (rows, V), 2.0)).astype(np.float32) if not with_noise else I.normal(12 + rows, (rows, V), 2.0)
    nz = I.gumbel_noise(13 + V, (rows, V)) if with_noise else None
    ref, margin = G.choose_tokens(lg[None], None if nz is None else nz[None], 0.7)
    got = fv.fv_argmax_rows(T(lg), None if nz is None else T(nz), 0.7).cpu().numpy()
    if not with_noise:
        assert (lg == lg.max(-1, keepdims=True)).sum(-1).max() > 1 or V <= 4     # the case has real ties
        np.testing.assert_array_equal(got, ref[0])
    else:
        flagged = margin[0] < 1e-5
        np.testing.assert_array_equal(got[~flagged], ref[0][~flagged])
        assert flagged.mean() <= 0.01


def test_residual_accumulate_matches_eq2():
    B, V, d = 3, 50, 32
    cb = I.normal(21, (V, d), 1.0)
    sizes = [(1, 1), (2, 3), (5, 4), (12, 12), (40, 33)]
    r_ref, r_gpu = None, None
    for k, (h, w) in enumerate(sizes):
        ids = (I.uniform01(30 + k, B * h * w) * V).astype(np.int32).reshape(B, h * w)
        hp, wp = sizes[k - 1] if k else (0, 0)
        r_ref = G.residual_accumulate(r_ref, hp, wp, ids, cb, h, w)
        # the GPU takes the oracle-side previous map (rounded to fp32), so each step is compared on its own
        prev = None if k == 0 else T(prev_ref32)
        r_gpu = fv.fv_residual_accumulate(T(ids, torch.int32), h, w, T(cb), prev, hp, wp).cpu().numpy()
        np.testing.assert_allclose(r_gpu, r_ref, rtol=0, atol=1e-6)
        prev_ref32 = r_ref.astype(np.float32)
        r_ref = prev_ref32.astype(np.float64)


def test_residual_accumulate_flags_bad_ids():
    cb = T(I.normal(22, (8, 4), 1.0))
    st = torch.zeros(1, dtype=torch.int32, device=DEV)
    ids = torch.tensor([[0, 9, -1, 7]], dtype=torch.int32, device=DEV)
    out = fv.fv_residual_accumulate(ids, 2, 2, cb, status=st).cpu().numpy()
    assert int(st.item()) == 40
    np.testing.assert_array_equal(out[0, 1], cb[7].cpu().numpy())   # clamped, not read out of bounds
    np.testing.assert_array_equal(out[0, 2], cb[0].cpu().numpy())


@pytest.mark.parametrize("d,C,h,w,h2,w2,B", [(32, 256, 3, 3, 4, 4, 2), (8, 64, 1, 1, 2, 2, 1), (16, 1920, 12, 12, 16, 16, 2),
                                              (64, 2048, 16, 16, 20, 20, 1), (32, 2048, 5, 7, 9, 4, 3)])
def test_next_scale_input_matches_oracle(d, C, h, w, h2, w2, B):
    r = I.normal(41, (B, h * w, d), 2.0)
    w_in, b_in, pos = I.normal(42, (C, d), 1 / np.sqrt(d)), I.normal(43, (C,), 0.1), I.normal(44, (h2 * w2, C), 0.5)
    ref = G.next_scale_input(r, h, w, h2, w2, w_in, b_in, pos)
    got = fv.fv_next_scale_input(T(r), h, w, h2, w2, T(w_in), T(b_in), T(pos)).cpu().numpy()
    np.testing.assert_allclose(got, ref, rtol=1e-5, atol=2e-5)      # fp32 dot products of d terms
    got0 = fv.fv_next_scale_input(T(r), h, w, h2, w2, T(w_in), None, None).cpu().numpy()
    np.testing.assert_allclose(got0, G.next_scale_input(r, h, w, h2, w2, w_in, None, None), rtol=1e-5, atol=2e-5)


# margin below which a token choice may legitimately differ: the logits come out of a bf16 GEMM (K = C terms,
# inputs rounded to bf16, |logit| of a few units) against the fp64 oracle
LOGIT_TOL = 3e-2


@pytest.mark.parametrize("B,n,C,V", [(2, 16, 256, 512), (1, 300, 1024, 4096), (2, 1, 64, 64)])
def test_head_tokens_matches_oracle(B, n, C, V):
    y = I.normal(51, (B, n, C), 1.5) + 0.3
    wl = I.Workload("h", L=1, C=C, H=C // 64, B=B, sides=(1,), keep=(1.0,), cross_len=0, seed=9)
    gt = I.generation_tensors(wl, V=V, d=8)
    wh, bh = I.bf16_bits_to_f32(gt.w_head), I.bf16_bits_to_f32(gt.b_head)
    ref_logits = G.head_logits(y, gt.mod_head[:, 0], gt.mod_head[:, 1], wh, bh)
    noise = I.gumbel_noise(52, (B * n, V))
    for nz, tau in ((None, 1.0), (noise, 0.8)):
        ref_ids, margin = G.choose_tokens(ref_logits, None if nz is None else nz.reshape(B, n, V), tau)
        st = torch.zeros(1, dtype=torch.int32, device=DEV)
        ids, logits = fv.fv_head_tokens(T(y), T(gt.mod_head), BF(gt.w_head), BF(gt.b_head), None if nz is None else T(nz), tau,
                                        want_logits=True, status=st)
        torch.cuda.synchronize()
        assert int(st.item()) == 0
        lg = logits.cpu().numpy().reshape(B, n, V)
        assert np.abs(lg - ref_logits).max() <= LOGIT_TOL
        ids = ids.cpu().numpy()
        clear = margin > 2 * LOGIT_TOL
        np.testing.assert_array_equal(ids[clear], ref_ids[clear])
        # a disputed id must still be a near-best entry of the oracle's own perturbed logits
        z = ref_logits + (0 if nz is None else tau * nz.reshape(B, n, V).astype(np.float64))
        chosen = np.take_along_axis(z, ids[..., None].astype(np.int64), -1)[..., 0]
        assert np.all(z.max(-1) - chosen <= 2 * LOGIT_TOL)
        assert clear.size < 50 or clear.mean() >= 0.8
        # the GPU's own ids are the exact argmax of the GPU's own fp32 logits (ties to the lowest id)
        own, _ = G.choose_tokens(lg.astype(np.float32), None if nz is None else nz.reshape(B, n, V), tau)
        own_flag = _ < 1e-5
        np.testing.assert_array_equal(ids[~own_flag], own[~own_flag])


def _gen_setup(keep, sides=(1, 2, 3, 4, 6, 8), L=2, C=128, H=2, B=2, V=256, d=16, cross_len=0):
    wl = I.Workload("gen", L=L, C=C, H=H, B=B, sides=tuple(sides), keep=tuple(keep), cross_len=cross_len, seed=31)
    mt = I.model_tensors(wl)
    gt = I.generation_tensors(wl, V=V, d=d)
    sizes = [(s, s) for s in wl.sides]
    gen = G.GenerationOracle(make_oracle(wl, mt), sizes, gt.codebook, I.bf16_bits_to_f32(gt.w_head), I.bf16_bits_to_f32(gt.b_head),
                             gt.mod_head, gt.w_in, gt.b_in, gt.pos)
    cap = sum(wl.tokens(i) if wl.keep[i] >= 1.0 else O.kept_count(wl.keep[i], s, s) for i, s in enumerate(wl.sides))
    ctx = fv.FvContext(wl.L, wl.C, wl.H, sizes, wl.cache_step, wl.B, cap, mt, cross_len=wl.cross_len, device=DEV)
    return wl, gt, sizes, gen, ctx


def test_generation_loop_teacher_forced_against_oracle():
    """Each GPU stage of every step takes the oracle's record as input: the transformer output is within the
    step tolerance, the ids agree outside the margin, Eq. 2 and the next token map agree to fp32 rounding."""
    keep = (1.0, 1.0, 1.0, 1.0, 1.0, 1.0)
    wl, gt, sizes, gen, ctx = _gen_setup(keep)
    noise = [I.gumbel_noise(700 + k, (wl.B, wl.tokens(k), 256)) for k in range(len(sizes))]
    recs = gen.generate(gt.start, keep, noise, tau=0.5)
    ctx.reset()
    cb, w_in, b_in = T(gt.codebook), T(gt.w_in), T(gt.b_in)
    for k, rec in enumerate(recs):
        h, w = sizes[k]
        y = ctx.var_step(T(rec["x"].astype(np.float32)), k, keep[k])
        err, cos = per_token_errors(y.cpu().numpy(), rec["y"])
        assert err <= 3e-2 and cos >= 0.999
        ids = fv.fv_head_tokens(T(rec["y"].astype(np.float32)), T(gt.mod_head), BF(gt.w_head), BF(gt.b_head),
                                T(noise[k].reshape(-1, 256)), 0.5).cpu().numpy()
        clear = rec["margin"] > 2 * LOGIT_TOL
        np.testing.assert_array_equal(ids[clear], rec["ids"][clear])
        prev = None if k == 0 else T(recs[k - 1]["r"].astype(np.float32))
        hp, wp = sizes[k - 1] if k else (0, 0)
        r = fv.fv_residual_accumulate(T(rec["ids"].astype(np.int32), torch.int32), h, w, cb, prev, hp, wp)
        np.testing.assert_allclose(r.cpu().numpy(), rec["r"], rtol=0, atol=1e-5)
        if k + 1 < len(recs):
            h2, w2 = sizes[k + 1]
            x2 = fv.fv_next_scale_input(T(rec["r"].astype(np.float32)), h, w, h2, w2, w_in, b_in, T(gt.pos[k + 1]))
            np.testing.assert_allclose(x2.cpu().numpy(), recs[k + 1]["x"], rtol=1e-5, atol=5e-5)
    assert ctx.device_status() == 0
    ctx.close()


@pytest.mark.parametrize("keep", [(1.0,) * 6, (1.0, 1.0, 1.0, 1.0, 0.5, 0.4), (1.0, 1.0, 1.0, 1.0, 0.5, 0.0)])
def test_fv_generate_equals_its_stages_and_follows_the_oracle(keep):
    """The one-call loop gives exactly what chaining the exported stages on the GPU gives (bit for bit), twice
    in a row; against the free-running oracle the ids agree up to the first near-tie (after a legitimately
    different choice the two sequences are different samples and are no longer comparable)."""
    wl, gt, sizes, gen, ctx = _gen_setup(keep)
    noise = [I.gumbel_noise(800 + k, (wl.B * wl.tokens(k), 256)) for k in range(len(sizes))]
    g = fv.FvGenerator(ctx, gt, tau=0.5)
    nz = [T(a) for a in noise]
    ids_a, r_a = g.generate(T(gt.start), keep, nz)
    ids_a = [t.clone() for t in ids_a]; r_a = r_a.clone()
    ids_b, r_b = g.generate(T(gt.start), keep, nz)
    torch.cuda.synchronize()
    assert ctx.device_status() == 0
    for a, b in zip(ids_a, ids_b):
        assert torch.equal(a, b)
    assert torch.equal(r_a, r_b)
    # chained stages
    ctx.reset()
    x, r = T(gt.start), None
    for k, (h, w) in enumerate(sizes):
        y = ctx.var_step(x, k, keep[k])
        ids = fv.fv_head_tokens(y, g.mod_head, g.w_head, g.b_head, nz[k], 0.5)
        assert torch.equal(ids, ids_a[k])
        hp, wp = sizes[k - 1] if k else (0, 0)
        r = fv.fv_residual_accumulate(ids, h, w, g.codebook, r, hp, wp)
        if k + 1 < len(sizes):
            x = fv.fv_next_scale_input(r, h, w, *sizes[k + 1], g.w_in, g.b_in, g.pos[k + 1])
    assert torch.equal(r, r_a)
    # free-running oracle
    recs = gen.generate(gt.start, keep, [a.reshape(wl.B, -1, 256) for a in noise], tau=0.5)
    compared = 0
    for k, rec in enumerate(recs):
        got = ids_a[k].cpu().numpy()
        if np.array_equal(got, rec["ids"]):
            compared += 1
            continue
        diff = got != rec["ids"]
        assert np.all(rec["margin"][diff] <= 2 * LOGIT_TOL), f"step {k}: ids differ outside the margin"
        break
    assert compared >= 2
    if compared == len(recs):
        np.testing.assert_allclose(r_a.cpu().numpy(), recs[-1]["r"], rtol=0, atol=1e-5)
    ctx.close()


def test_head_tokens_at_the_last_scale_of_the_bench_workload_sampled_rows():
    """The head at full size (B = 2, 64x64 tokens, C = 2048, V = 4096: the launch configuration the bench times);
    the oracle computes a sample of rows (rows are independent), every sampled logit and id is checked."""
    B, n, C, V = 2, 4096, 2048, 4096
    y = I.normal(61, (B, n, C), 1.5) + 0.3
    wl = I.Workload("h", L=1, C=C, H=16, B=B, sides=(1,), keep=(1.0,), cross_len=0, seed=19)
    # head weights at the blocks' scale (std 0.02): |logits| stays below ~7, where one bf16 rounding of the
    # normalised activations keeps a K = 2048 dot product inside the 3e-2 bar
    gt = I.generation_tensors(wl, V=V, d=32, w_std=0.005)
    st = torch.zeros(1, dtype=torch.int32, device=DEV)
    ids, logits = fv.fv_head_tokens(T(y), T(gt.mod_head), BF(gt.w_head), BF(gt.b_head), want_logits=True, status=st)
    torch.cuda.synchronize()
    assert int(st.item()) == 0
    ids = ids.cpu().numpy(); lg = logits.cpu().numpy().reshape(B, n, V)
    rows = np.unique((I.uniform01(62, 96) * n).astype(np.int64))
    rows = np.concatenate([rows, [0, 127, 128, n - 1]])             # tile edges of the GEMM too
    wh, bh = I.bf16_bits_to_f32(gt.w_head), I.bf16_bits_to_f32(gt.b_head)
    ref = G.head_logits(y[:, rows], gt.mod_head[:, 0], gt.mod_head[:, 1], wh, bh)
    assert np.abs(lg[:, rows] - ref).max() <= LOGIT_TOL
    ref_ids, margin = G.choose_tokens(ref)
    clear = margin > 2 * LOGIT_TOL
    np.testing.assert_array_equal(ids[:, rows][clear], ref_ids[clear])
    # every id (all 8192 rows) is the exact argmax of the GPU's own fp32 logits
    np.testing.assert_array_equal(ids, lg.argmax(-1))


def test_head_tokens_of_the_bench_s_own_head_within_one_bf16_rounding():
    """The head bench.py times (generation_tensors' default: weights of std 0.08, logits of +-15), at full size.  Its
    logits are too large for the absolute 3e-2 bar, so the bound is the arithmetic's own: the normalised, modulated
    activations are rounded to bf16 once before the tensor-core GEMM (<= 2^-9 relative per element, fp32 accumulation),
    hence |logit - oracle| <= 2^-9 * sum_c |a_c * w_vc| (+ 1e-4 for the fp32 sums) for every sampled logit; ids may
    differ from the oracle's only where its margin is inside twice that bound."""
    B, n, C, V = 2, 4096, 2048, 4096
    y = I.normal(61, (B, n, C), 1.5) + 0.3
    wl = I.Workload("h", L=1, C=C, H=16, B=B, sides=(1,), keep=(1.0,), cross_len=0, seed=19)
    gt = I.generation_tensors(wl, V=V, d=32)                          # the bench's head
    st = torch.zeros(1, dtype=torch.int32, device=DEV)
    ids, logits = fv.fv_head_tokens(T(y), T(gt.mod_head), BF(gt.w_head), BF(gt.b_head), want_logits=True, status=st)
    torch.cuda.synchronize()
    assert int(st.item()) == 0
    ids = ids.cpu().numpy(); lg = logits.cpu().numpy().reshape(B, n, V)
    rows = np.unique(np.concatenate([(I.uniform01(63, 64) * n).astype(np.int64), [0, 127, 128, n - 1]]))
    wh, bh = I.bf16_bits_to_f32(gt.w_head).astype(np.float64), I.bf16_bits_to_f32(gt.b_head).astype(np.float64)
    ref = G.head_logits(y[:, rows], gt.mod_head[:, 0], gt.mod_head[:, 1], wh, bh)
    a = O.modulate(O.layernorm(y[:, rows].astype(np.float64)), gt.mod_head[:, 0].astype(np.float64), gt.mod_head[:, 1].astype(np.float64))
    bound = 2.0 ** -9 * (np.abs(a) @ np.abs(wh).T) + 1e-4             # [B, rows, V]
    err = np.abs(lg[:, rows] - ref)
    assert np.all(err <= bound), float((err / bound).max())
    assert np.abs(ref).max() > 7.0                                     # the case the absolute bar does not cover
    ref_ids, margin = G.choose_tokens(ref)
    clear = margin > 2 * bound.max(axis=-1)
    assert clear.mean() > 0.5
    np.testing.assert_array_equal(ids[:, rows][clear], ref_ids[clear])
    np.testing.assert_array_equal(ids, lg.argmax(-1))
