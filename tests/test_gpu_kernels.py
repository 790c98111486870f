"""Kernel-level parity: each CUDA kernel, called through the C ABI, against the CPU oracle on the same
seeded inputs.  Integer results (indices, inverse map, restored copies) must be bit-exact; floating
point within max-abs 3e-2 and per-token cosine >= 0.999 (bf16 tensor-core path vs fp64 oracle)."""
import numpy as np
import pytest
import torch

from oracle import fastvar_oracle as O
from paper_2503_23367_b200 import binding as fv
from paper_2503_23367_b200 import inputs as I
from tests.helpers import per_token_errors

pytestmark = pytest.mark.gpu
DEV = "cuda:0"
MAX_ABS, MIN_COS = 3e-2, 0.999


def dev(a, dtype=None):
    t = torch.from_numpy(np.ascontiguousarray(a)).to(DEV)
    return t if dtype is None else t.to(dtype)


def bf16_dev(bits):
    return torch.from_numpy(bits.view(np.int16)).to(DEV).view(torch.bfloat16)


def bf16_host(t):
    return t.detach().to(torch.float32).cpu().numpy().astype(np.float64)


# ------------------------------------------------------------------ Pivotal Token Selection
SELECT_CASES = [  # B, h, w, C, keep, kind
    (1, 13, 13, 256, 0.5, "iid"), (8, 16, 16, 1024, 0.5, "iid"), (4, 18, 18, 1920, 0.75, "iid"),
    (2, 64, 64, 2048, 0.2, "structured"), (1, 1, 1, 256, 0.5, "iid"), (3, 5, 7, 260, 0.3, "iid"),
    (2, 40, 40, 2048, 0.6, "structured"), (1, 3, 2, 8, 1.0, "iid"), (2, 33, 31, 128, 0.01, "iid"),
    (1, 128, 128, 2048, 0.2, "iid"),        # 2K zero-shot step: 16384 tokens, map larger than L2
    (1, 192, 256, 64, 0.1, "iid"),          # 49152 tokens: the largest map the top-k CTA holds in shared memory
]


@pytest.mark.parametrize("B,h,w,C,keep,kind", SELECT_CASES)
def test_prune_select_matches_oracle(B, h, w, C, keep, kind):
    x = I.token_map(77 + B + h, B, h, w, C, kind)
    r = fv.fv_prune_select(dev(x), h, w, keep, want_inv=True, want_score=True, want_near_tie=True)
    torch.cuda.synchronize()
    k = O.kept_count(keep, h, w)
    assert r["k"] == k
    score_g = r["score"].cpu().numpy()
    idx_g = r["idx"].cpu().numpy().astype(np.int64)
    inv_g = r["inv"].cpu().numpy().astype(np.int64)
    score_o = O.pts_score(x)
    np.testing.assert_allclose(score_g, score_o, rtol=2e-5, atol=1e-4)
    # integer work is exact GIVEN the scores: oracle top-k on the very scores the kernel ranked
    assert np.array_equal(idx_g, O.pts_topk(score_g, k))
    assert np.array_equal(inv_g, O.inverse_map(idx_g, h * w))
    # against the oracle's own fp64 scores: any difference must sit on a near-tie at the threshold
    idx_o = O.pts_topk(score_o, k)
    for b in range(B):
        diff = np.setxor1d(idx_g[b], idx_o[b])
        if len(diff):
            tau = np.sort(score_o[b])[::-1][k - 1]
            assert np.all(np.abs(score_o[b, diff] - tau) <= 1e-5 * tau), "index mismatch away from a near-tie"
    assert (r["near_tie"].cpu().numpy() >= 1).all()


def test_prune_select_ties_go_to_lowest_index():
    B, h, w, C = 2, 12, 12, 64
    n = h * w
    # constant map: every score is 0 -> the first k tokens
    x = np.full((B, n, C), 0.37, dtype=np.float32)
    r = fv.fv_prune_select(dev(x), h, w, 0.5, want_near_tie=True)
    assert np.array_equal(r["idx"].cpu().numpy(), np.tile(np.arange(72, dtype=np.int32), (B, 1)))
    # rows drawn from 3 prototype tokens: exact ties in bulk
    protos = I.normal(5, (3, C))
    pick = (I.uniform01(6, B * n) * 3).astype(np.int64).reshape(B, n)
    x = protos[pick]
    r = fv.fv_prune_select(dev(x), h, w, 0.4, want_score=True, want_near_tie=True)
    torch.cuda.synchronize()
    s = r["score"].cpu().numpy()
    assert len(np.unique(s[0])) <= 3
    assert np.array_equal(r["idx"].cpu().numpy().astype(np.int64), O.pts_topk(s, r["k"]))
    assert (r["near_tie"].cpu().numpy() > 1).all()


@pytest.mark.parametrize("crowd,levels,keep", [(3000, 3000, 0.3), (3000, 300, 0.3), (600, 600, 0.1), (200, 40, 0.02),
                                               (4000, 1, 0.5), (1100, 1100, 0.2)])
def test_prune_select_scores_crowded_at_the_threshold(crowd, levels, keep):
    """A few far outliers stretch the range of the scores while `crowd` tokens sit within a few hundred ulps of one
    another (on `levels` distinct values) right where the k-th largest falls: the threshold's first-digit bin holds
    the whole crowd, so the ranking has to refine it with further digits -- over all keys while the bin is too full
    for the candidate list, over the list afterwards -- before it can finish by counting.  Exact given the scores."""
    B, h, w, C = 2, 64, 64, 8
    n = h * w
    k = O.kept_count(keep, h, w)
    above = max(2, k - crowd // 2)             # tokens far above the crowd: the k-th largest falls inside the crowd
    assert above < k <= above + crowd <= n
    a = np.zeros((B, n), dtype=np.float64)
    for b in range(B):
        perm = np.argsort(I.uniform01(90 + b, n), kind="stable")
        a[b, perm[:crowd]] = 1.0 + (np.arange(crowd) % levels) * 2.0 ** -22 * (1 + b)
        a[b, perm[crowd:crowd + above]] = 2.0 + 30.0 * I.uniform01(290 + b, above)
        a[b, perm[crowd + above:]] = 0.25 + 0.5 * I.uniform01(190 + b, n - crowd - above)
    x = np.zeros((B, n, C), dtype=np.float32)
    x[:, :, 0] = a
    x[:, 1::2, 0] *= -1.0                      # alternating signs keep the mean token near zero
    r = fv.fv_prune_select(dev(x), h, w, keep, want_inv=True, want_score=True, want_near_tie=True)
    torch.cuda.synchronize()
    score_g = r["score"].cpu().numpy()
    np.testing.assert_allclose(score_g, O.pts_score(x), rtol=2e-5, atol=1e-6)
    idx_g = r["idx"].cpu().numpy().astype(np.int64)
    assert np.array_equal(idx_g, O.pts_topk(score_g, k))
    assert np.array_equal(r["inv"].cpu().numpy().astype(np.int64), O.inverse_map(idx_g, n))


def test_prune_select_argument_errors():
    big = torch.zeros((1, 193 * 256, 8), device=DEV)                      # one row of tokens beyond the largest map
    with pytest.raises(fv.FvError) as e:
        fv.fv_prune_select(big, 193, 256, 0.5)
    assert e.value.code == 4
    x = torch.zeros((1, 4, 8), device=DEV)
    with pytest.raises(fv.FvError) as e:
        fv.fv_prune_select(x, 2, 2, 0.0)
    assert e.value.code == 1
    with pytest.raises(fv.FvError) as e:
        fv.fv_prune_select(x, 2, 2, 0.5, workspace=torch.empty(16, dtype=torch.uint8, device=DEV))
    assert e.value.code == 3


# ------------------------------------------------------------------ gather + LayerNorm + modulate
@pytest.mark.parametrize("B,n,k,C,with_mod", [(1, 169, 85, 256, True), (4, 324, 243, 1920, True),
                                             (2, 1024, 205, 2048, False), (2, 50, 50, 128, True), (2, 4096, 820, 2048, True)])
def test_gather_ln(B, n, k, C, with_mod):
    x = I.normal(3, (B, n, C)) * 2.0 + 0.5
    idx = np.stack([np.sort(np.argsort(I.uniform01(9 + b, n))[:k]) for b in range(B)]).astype(np.int32)
    mod = I.normal(4, (B, 6, C), 0.3)
    modt = dev(mod)                      # sigma at +0, beta at +C floats, images 6*C floats apart
    sig, bet = (modt.data_ptr(), modt.data_ptr() + 4 * C) if with_mod else (None, None)
    out = fv.fv_gather_ln(dev(x), dev(idx) if k != n else None, sig, bet, 6 * C)
    torch.cuda.synchronize()
    ref = O.layernorm(O.pts_gather(x.astype(np.float64), idx) if k != n else x.astype(np.float64))
    if with_mod:
        ref = O.modulate(ref, mod[:, 0].astype(np.float64), mod[:, 1].astype(np.float64))
    err, cos = per_token_errors(bf16_host(out), ref)
    assert err <= MAX_ABS and cos >= MIN_COS
    assert np.abs(bf16_host(out) - ref).max() <= np.abs(ref).max() * 2 ** -8 + 1e-6   # one bf16 rounding


# ------------------------------------------------------------------ Cached Token Restoration
@pytest.mark.parametrize("B,hc,wc,h,w,C,k", [(1, 10, 10, 13, 13, 256, 85), (2, 32, 32, 64, 64, 2048, 820),
                                             (2, 3, 5, 7, 4, 64, 1), (1, 4, 4, 4, 4, 8, 16), (3, 13, 13, 32, 32, 1920, 256)])
def test_restore_is_bit_exact(B, hc, wc, h, w, C, k):
    n = h * w
    cache = I.normal_bf16(21, (B, hc * wc, C))
    piv = I.normal_bf16(22, (B, k, C))
    idx = np.stack([np.sort(np.argsort(I.uniform01(30 + b, n))[:k]) for b in range(B)]).astype(np.int32)
    out = fv.fv_restore(bf16_dev(cache), hc, wc, bf16_dev(piv), dev(idx), h, w)
    torch.cuda.synchronize()
    ref = O.cached_token_restoration(I.bf16_bits_to_f32(piv).astype(np.float64), idx.astype(np.int64),
                                     I.bf16_bits_to_f32(cache).astype(np.float64), hc, wc, h, w)
    got = out.view(torch.int16).cpu().numpy().view(np.uint16)
    assert np.array_equal(got, I.to_bf16_bits(ref.astype(np.float32)))           # a copy: exact bits
    # unsorted index order gives the same map
    perm = np.stack([np.argsort(I.uniform01(40 + b, k)) for b in range(B)])
    idx_p = np.take_along_axis(idx, perm, axis=1)
    piv_p = np.stack([piv[b][perm[b]] for b in range(B)])
    out2 = fv.fv_restore(bf16_dev(cache), hc, wc, bf16_dev(piv_p), dev(idx_p), h, w)
    assert torch.equal(out2, out)


@pytest.mark.parametrize("with_gamma", [True, False])
def test_restore_residual(with_gamma):
    B, hc, wc, h, w, C, k = 2, 10, 10, 16, 16, 1024, 128
    n = h * w
    x = I.normal(50, (B, n, C))
    y = I.normal_bf16(51, (B, k, C))
    cache = I.normal_bf16(52, (B, hc * wc, C))
    mod = I.normal(53, (B, 6, C), 0.3)
    idx = np.stack([np.sort(np.argsort(I.uniform01(60 + b, n))[:k]) for b in range(B)])
    inv = O.inverse_map(idx, n).astype(np.int32)
    xd, modd = dev(x), dev(mod)
    fv.fv_restore_residual(xd, bf16_dev(y), bf16_dev(cache), dev(inv), modd.data_ptr() + 2 * 4 * C if with_gamma else None,
                           6 * C, h, w, hc, wc)
    torch.cuda.synchronize()
    yfull = O.cached_token_restoration(I.bf16_bits_to_f32(y).astype(np.float64), idx,
                                       I.bf16_bits_to_f32(cache).astype(np.float64), hc, wc, h, w)
    g = mod[:, 2].astype(np.float64)[:, None, :] if with_gamma else 1.0
    ref = x.astype(np.float64) + g * yfull
    np.testing.assert_allclose(xd.cpu().numpy(), ref, rtol=1e-6, atol=2e-6)


@pytest.mark.parametrize("B,hc,wc,h,w,C,k", [(1, 10, 10, 13, 13, 256, 85), (2, 32, 32, 64, 64, 2048, 820), (2, 3, 5, 7, 4, 64, 1),
                                             (1, 4, 4, 4, 4, 8, 3), (2, 6, 6, 4, 3, 64, 5), (1, 1, 1, 5, 5, 32, 2)])
@pytest.mark.parametrize("mode", [1, 2])
def test_restore_bilinear(B, hc, wc, h, w, C, k, mode):
    """interp_mode 1 / 2: unkept tokens are the bilinear (four cached rows) or bicubic (sixteen) blend at half-pixel
    centres, computed in fp32 and rounded to bf16 once; kept tokens are still exact copies."""
    n = h * w
    cache = I.normal_bf16(23, (B, hc * wc, C))
    piv = I.normal_bf16(24, (B, k, C))
    idx = np.stack([np.sort(np.argsort(I.uniform01(33 + b, n))[:k]) for b in range(B)]).astype(np.int32)
    out = fv.fv_restore(bf16_dev(cache), hc, wc, bf16_dev(piv), dev(idx), h, w, interp_mode=mode)
    torch.cuda.synchronize()
    ref = O.cached_token_restoration(I.bf16_bits_to_f32(piv).astype(np.float64), idx.astype(np.int64),
                                     I.bf16_bits_to_f32(cache).astype(np.float64), hc, wc, h, w, ("bilinear", "bicubic")[mode - 1])
    got = bf16_host(out)
    assert np.abs(got - ref).max() <= np.abs(ref).max() * 2 ** -8 + 1e-5        # one bf16 rounding of the fp32 blend
    for b in range(B):
        np.testing.assert_array_equal(got[b, idx[b]], I.bf16_bits_to_f32(piv[b]))


@pytest.mark.parametrize("B,hc,wc,h,w,C,k", [(2, 10, 10, 16, 16, 1024, 128), (2, 32, 32, 64, 64, 2048, 820), (1, 5, 7, 9, 6, 64, 11)])
@pytest.mark.parametrize("mode", [1, 2])
def test_restore_residual_bilinear(B, hc, wc, h, w, C, k, mode):
    n = h * w
    x = I.normal(58, (B, n, C)); y = I.normal_bf16(59, (B, k, C)); cache = I.normal_bf16(60, (B, hc * wc, C))
    mod = I.normal(61, (B, 6, C), 0.3)
    idx = np.stack([np.sort(np.argsort(I.uniform01(62 + b, n))[:k]) for b in range(B)])
    inv = O.inverse_map(idx, n).astype(np.int32)
    xd, modd = dev(x), dev(mod)
    fv.fv_restore_residual(xd, bf16_dev(y), bf16_dev(cache), dev(inv), modd.data_ptr() + 2 * 4 * C, 6 * C, h, w, hc, wc, interp_mode=mode)
    torch.cuda.synchronize()
    yfull = O.cached_token_restoration(I.bf16_bits_to_f32(y).astype(np.float64), idx, I.bf16_bits_to_f32(cache).astype(np.float64),
                                       hc, wc, h, w, ("bilinear", "bicubic")[mode - 1])
    ref = x.astype(np.float64) + mod[:, 2].astype(np.float64)[:, None, :] * yfull
    np.testing.assert_allclose(xd.cpu().numpy(), ref, rtol=2e-6, atol=1e-5)      # fp32 blend of 4 / 16 rows, then one fma


def _restore_case(B, hc, wc, h, w, C, k, seed=54):
    n = h * w
    x = I.normal(seed, (B, n, C))
    y = I.normal_bf16(seed + 1, (B, k, C))
    cache = I.normal_bf16(seed + 2, (B, hc * wc, C))
    mod = I.normal(seed + 3, (B, 6, C), 0.3)
    idx = np.stack([np.sort(np.argsort(I.uniform01(seed + 7 + b, n))[:k]) for b in range(B)])
    inv = O.inverse_map(idx, n).astype(np.int32)
    yfull = O.cached_token_restoration(I.bf16_bits_to_f32(y).astype(np.float64), idx,
                                       I.bf16_bits_to_f32(cache).astype(np.float64), hc, wc, h, w)
    ref = x.astype(np.float64) + mod[:, 2].astype(np.float64)[:, None, :] * yfull
    return x, y, cache, mod, inv, ref


def test_restore_residual_large():
    """The 64x64 pruned step's restore (67 MB map, 820 kept rows per image, cache of the 32x32 step): every element
    of the updated map against the oracle."""
    B, hc, wc, h, w, C, k = 2, 32, 32, 64, 64, 2048, 820
    x, y, cache, mod, inv, ref = _restore_case(B, hc, wc, h, w, C, k)
    xd, modd = dev(x), dev(mod)
    fv.fv_restore_residual(xd, bf16_dev(y), bf16_dev(cache), dev(inv), modd.data_ptr() + 2 * 4 * C, 6 * C, h, w, hc, wc)
    torch.cuda.synchronize()
    np.testing.assert_allclose(xd.cpu().numpy(), ref, rtol=1e-6, atol=2e-6)


# Maps whose chunks of 32 tokens fold in groups of 1 / 2 / 4 / 5 / 8 (one thread-block cluster per group), with a
# ragged last chunk (33 x 31, 50 x 50), a ragged last group (50 x 50: 79 chunks in groups of 5), and groups too
# large for a cluster (96 x 96, 128 x 128: 18 and 32 chunks per group, folded through global memory).
COLSUM_CASES = [  # B, hc, wc, h, w, C, k
    (1, 10, 10, 13, 13, 256, 85), (3, 10, 10, 33, 31, 256, 205), (2, 32, 32, 40, 40, 2048, 960), (2, 32, 32, 48, 48, 2048, 922),
    (2, 32, 32, 64, 64, 2048, 820), (1, 13, 13, 50, 50, 1920, 625), (1, 48, 48, 96, 96, 2048, 1844), (1, 48, 48, 128, 128, 2048, 3277),
]


@pytest.mark.parametrize("B,hc,wc,h,w,C,k", COLSUM_CASES)
@pytest.mark.parametrize("fold", [0, 1])
def test_restore_leaves_the_column_sums_of_the_updated_map(B, hc, wc, h, w, C, k, fold):
    """Eq. 4 for the NEXT selection comes from the restoration: the partial sums it leaves in the selection
    workspace, added up per image, are the column sums of the map it has just updated -- for the one-pass form
    (part 0), for the two-pass form a scale step uses (part 1: rows that were not kept, part 2: kept rows + fold),
    with the fold inside thread-block clusters (fold 0, where the shape allows) and through global memory (fold 1).
    The two forms must give the same bits in the map (their sums add the rows in a different order)."""
    n = h * w
    x, y, cache, mod, inv, ref = _restore_case(B, hc, wc, h, w, C, k, seed=154)
    yd, cd, invd, modd = bf16_dev(y), bf16_dev(cache), dev(inv), dev(mod)
    gamma = modd.data_ptr() + 2 * 4 * C
    colsum_ref = ref.sum(axis=1)                                            # fp64 [B, C]
    scale = np.abs(ref).sum(axis=1).max()                                   # fp32 sums of n terms in a fixed order
    fv.fv_restore_force_fold(fold)
    try:
        results = []
        for parts in ((0,), (1, 2)):
            xd = dev(x)
            ws = fv.fv_prune_select_workspace(B, n, C, DEV)
            ws.fill_(0xFF)                                                  # stale contents must not matter (NaN patterns)
            for part in parts:
                fv.fv_restore_residual(xd, yd, cd, invd, gamma, 6 * C, h, w, hc, wc, colsum_ws=ws, part=part)
            torch.cuda.synchronize()
            got = fv.fv_colsum_partials(ws, B, n, C).cpu().numpy().astype(np.float64).sum(axis=1)
            assert np.abs(got - colsum_ref).max() <= 1e-5 * scale, (parts, np.abs(got - colsum_ref).max(), scale)
            np.testing.assert_allclose(xd.cpu().numpy(), ref, rtol=1e-6, atol=2e-6)
            results.append(xd.cpu().numpy())
        assert np.array_equal(results[0], results[1])
    finally:
        fv.fv_restore_force_fold(0)


@pytest.mark.parametrize("B,hc,wc,h,w,C,k", COLSUM_CASES)
def test_selection_from_the_restoration_s_column_sums(B, hc, wc, h, w, C, k):
    """The selection that follows a restoration inside a scale step: it takes Eq. 4's mean token from the sums the
    restoration left behind instead of summing the map again.  Scores and kept set against the oracle applied to
    the updated map, and the same kept set as the stand-alone selection of the same map up to near-ties."""
    n = h * w
    keep = k / n
    assert O.kept_count(keep, h, w) == k
    x, y, cache, mod, inv, ref = _restore_case(B, hc, wc, h, w, C, k, seed=254)
    xd, modd = dev(x), dev(mod)
    ws = fv.fv_prune_select_workspace(B, n, C, DEV)
    for part in (1, 2):
        fv.fv_restore_residual(xd, bf16_dev(y), bf16_dev(cache), dev(inv), modd.data_ptr() + 2 * 4 * C, 6 * C, h, w, hc, wc,
                               colsum_ws=ws, part=part)
    r = fv.fv_prune_select_after_restore(xd, h, w, keep, ws, want_score=True)
    alone = fv.fv_prune_select(xd, h, w, keep, want_score=True)
    torch.cuda.synchronize()
    x_new = xd.cpu().numpy()
    score_o = O.pts_score(x_new)                                            # oracle on the map the GPU holds
    score_g = r["score"].cpu().numpy()
    np.testing.assert_allclose(score_g, score_o, rtol=2e-5, atol=1e-4)
    idx_g = r["idx"].cpu().numpy().astype(np.int64)
    assert np.array_equal(idx_g, O.pts_topk(score_g, k))
    assert np.array_equal(r["inv"].cpu().numpy(), O.inverse_map(idx_g, n))
    idx_o = O.pts_topk(score_o, k)
    for b in range(B):
        diff = np.setxor1d(idx_g[b], idx_o[b])
        if len(diff):
            tau = np.sort(score_o[b])[::-1][k - 1]
            assert np.all(np.abs(score_o[b, diff] - tau) <= 1e-5 * tau), "index mismatch away from a near-tie"
    # the stand-alone selection sums the rows of a chunk in another order: same scores up to fp32 rounding
    np.testing.assert_allclose(alone["score"].cpu().numpy(), score_g, rtol=2e-6, atol=1e-5)
    assert np.array_equal(alone["idx"].cpu().numpy(), O.pts_topk(alone["score"].cpu().numpy(), k))


# ------------------------------------------------------------------ tcgen05 GEMM
GEMM_CASES = [(128, 128, 64), (85, 768, 256), (1000, 1024, 1024), (1640, 6144, 2048), (300, 4096, 1024),
              (130, 1920, 1920), (7, 136, 72), (2048, 2048, 8192)]


@pytest.mark.parametrize("M,N,K", GEMM_CASES)
@pytest.mark.parametrize("epilogue", [0, 1])
def test_gemm_bf16(M, N, K, epilogue):
    # activations ~ LayerNorm outputs (unit scale); the K = 8192 case is the MLP's second GEMM, whose
    # input is GELU output (rms ~0.5), which keeps |y| where one bf16 rounding stays below 3e-2
    a = I.normal_bf16(70, (M, K), 1.0 if K <= 2048 else 0.5)
    w = I.normal_bf16(71, (N, K), 0.02)
    b = I.normal_bf16(72, (N,), 0.02)
    status = torch.zeros(1, dtype=torch.int32, device=DEV)
    out = fv.fv_gemm_bf16(bf16_dev(a), bf16_dev(w), bf16_dev(b), epilogue=epilogue, status=status)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    ref = O.linear(I.bf16_bits_to_f32(a), I.bf16_bits_to_f32(w), I.bf16_bits_to_f32(b))
    if epilogue == 1:
        ref = O.gelu_tanh(ref)
    err, cos = per_token_errors(bf16_host(out), ref)
    assert err <= MAX_ABS and cos >= MIN_COS, (err, cos)


@pytest.mark.parametrize("N,K", [(6144, 2048), (2048, 2048), (8192, 2048), (2048, 8192)])
def test_gemm_bf16_at_the_2k_step_s_row_count(N, K):
    """The four projection shapes of a block at the 128x128 zero-shot step (3277 kept rows: 25 full row tiles and a
    ragged one of 77), bias + GELU epilogue; the oracle runs on a sample of rows that covers every row tile."""
    M = 3277
    a = I.normal_bf16(170, (M, K), 1.0 if K <= 2048 else 0.5); w = I.normal_bf16(171, (N, K), 0.02); b = I.normal_bf16(172, (N,), 0.02)
    status = torch.zeros(1, dtype=torch.int32, device=DEV)
    out = fv.fv_gemm_bf16(bf16_dev(a), bf16_dev(w), bf16_dev(b), epilogue=1, status=status)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    rows = np.unique(np.concatenate([np.arange(0, M, 11), np.arange(M - 80, M)]))
    ref = O.gelu_tanh(O.linear(I.bf16_bits_to_f32(a[rows]), I.bf16_bits_to_f32(w), I.bf16_bits_to_f32(b)))
    err, cos = per_token_errors(bf16_host(out)[rows], ref)
    assert err <= MAX_ABS and cos >= MIN_COS, (err, cos)


SPLITK_CASES = [(2, 2048, 8192), (2, 6144, 2048), (85, 768, 256), (128, 8192, 2048), (288, 2048, 2048), (300, 1024, 4096), (7, 136, 1024),
                (1640, 6144, 2048)]   # the last shape has enough tiles: the scratch is passed but no split is taken


@pytest.mark.parametrize("M,N,K", SPLITK_CASES)
@pytest.mark.parametrize("epilogue", [0, 1])
def test_gemm_bf16_split_along_k(M, N, K, epilogue):
    """Few rows against a large weight matrix: K slices on different CTAs, partial sums added in slice order."""
    a = I.normal_bf16(73, (M, K), 1.0 if K <= 2048 else 0.5)
    w = I.normal_bf16(74, (N, K), 0.02)
    b = I.normal_bf16(75, (N,), 0.02)
    status = torch.zeros(1, dtype=torch.int32, device=DEV)
    ws = torch.zeros(fv.lib().fv_gemm_splitk_workspace_bytes(), dtype=torch.uint8, device=DEV)
    ad, wd, bd = bf16_dev(a), bf16_dev(w), bf16_dev(b)
    out = fv.fv_gemm_bf16(ad, wd, bd, epilogue=epilogue, status=status, splitk_ws=ws)
    out2 = fv.fv_gemm_bf16(ad, wd, bd, epilogue=epilogue, status=status, splitk_ws=ws)   # counters were left at zero
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    assert torch.equal(out, out2)                       # arrival order does not change the sum
    assert int(ws[:4096].to(torch.int32).sum().item()) == 0
    ref = O.linear(I.bf16_bits_to_f32(a), I.bf16_bits_to_f32(w), I.bf16_bits_to_f32(b))
    if epilogue == 1:
        ref = O.gelu_tanh(ref)
    err, cos = per_token_errors(bf16_host(out), ref)
    assert err <= MAX_ABS and cos >= MIN_COS, (err, cos)


def test_gemm_split_along_k_refuses_small_scratch():
    a = torch.zeros((2, 256), dtype=torch.bfloat16, device=DEV); w = torch.zeros((256, 256), dtype=torch.bfloat16, device=DEV)
    with pytest.raises(fv.FvError) as e:
        fv.fv_gemm_bf16(a, w, None, splitk_ws=torch.zeros(4096, dtype=torch.uint8, device=DEV))
    assert e.value.code == 3


@pytest.mark.parametrize("path", [2, 3])
@pytest.mark.parametrize("M,N,K", [(128, 128, 64), (300, 512, 256), (7, 136, 72), (1000, 1024, 1024), (130, 1920, 1920),
                                   (1640, 6144, 2048), (1844, 2048, 8192)])
def test_gemm_bf16_on_cta_pairs(M, N, K, path):
    """The CTA-pair kernel (two CTAs share a 256-row tile, tcgen05 cta_group::2), forced for every shape,
    ragged M / N tails included; both tile widths."""
    a = I.normal_bf16(76, (M, K), 1.0 if K <= 2048 else 0.5)
    w = I.normal_bf16(77, (N, K), 0.02)
    b = I.normal_bf16(78, (N,), 0.02)
    status = torch.zeros(1, dtype=torch.int32, device=DEV)
    assert fv.lib().fv_gemm_force_path(path) == 0
    try:
        out = fv.fv_gemm_bf16(bf16_dev(a), bf16_dev(w), bf16_dev(b), epilogue=1, status=status)
        torch.cuda.synchronize()
    finally:
        fv.lib().fv_gemm_force_path(0)
    assert int(status.item()) == 0
    ref = O.gelu_tanh(O.linear(I.bf16_bits_to_f32(a), I.bf16_bits_to_f32(w), I.bf16_bits_to_f32(b)))
    err, cos = per_token_errors(bf16_host(out), ref)
    assert err <= MAX_ABS and cos >= MIN_COS, (err, cos)


@pytest.mark.parametrize("epilogue", [0, 1])
@pytest.mark.parametrize("M,N,K,splitk", [(128, 128, 64, False), (7, 136, 72, False), (300, 1024, 4096, True), (32, 2048, 2048, True),
                                          (128, 2048, 8192, True), (1000, 1032, 1024, False), (2, 2048, 8192, True)])
def test_gemm_bf16_width_64_tiles(M, N, K, splitk, epilogue):
    """The 64-wide tile (chosen by itself for few rows against a narrow output), forced for every shape, with
    and without the K split."""
    a = I.normal_bf16(93, (M, K), 1.0 if K <= 2048 else 0.5); w = I.normal_bf16(94, (N, K), 0.02); b = I.normal_bf16(95, (N,), 0.02)
    status = torch.zeros(1, dtype=torch.int32, device=DEV)
    ws = torch.zeros(fv.lib().fv_gemm_splitk_workspace_bytes(), dtype=torch.uint8, device=DEV) if splitk else None
    assert fv.lib().fv_gemm_force_path(7) == 0
    try:
        out = fv.fv_gemm_bf16(bf16_dev(a), bf16_dev(w), bf16_dev(b), epilogue=epilogue, status=status, splitk_ws=ws)
        torch.cuda.synchronize()
    finally:
        fv.lib().fv_gemm_force_path(0)
    assert int(status.item()) == 0
    ref = O.linear(I.bf16_bits_to_f32(a), I.bf16_bits_to_f32(w), I.bf16_bits_to_f32(b))
    if epilogue == 1:
        ref = O.gelu_tanh(ref)
    err, cos = per_token_errors(bf16_host(out), ref)
    assert err <= MAX_ABS and cos >= MIN_COS, (err, cos)


@pytest.mark.parametrize("path", [8, 9, 10, 11])
@pytest.mark.parametrize("epilogue", [0, 1])
@pytest.mark.parametrize("M,N,K", [(128, 128, 64), (7, 136, 72), (300, 1024, 4096), (32, 2048, 2048), (128, 2048, 8192), (2, 6144, 2048),
                                   (200, 1032, 1024), (2, 2048, 8192), (130, 192, 128)])
def test_gemm_bf16_split_inside_a_cluster(M, N, K, epilogue, path):
    """K split over the 2 or 4 CTAs of a cluster (partials reduced through distributed shared memory), 128- and
    64-wide tiles, forced for every shape: ragged rows and columns, fewer k-blocks than CTAs (K = 64, 72, 128: some
    CTAs of the cluster then have nothing to add), and twice in a row with identical bits."""
    a = I.normal_bf16(96, (M, K), 1.0 if K <= 2048 else 0.5); w = I.normal_bf16(97, (N, K), 0.02); b = I.normal_bf16(98, (N,), 0.02)
    status = torch.zeros(1, dtype=torch.int32, device=DEV)
    ad, wd, bd = bf16_dev(a), bf16_dev(w), bf16_dev(b)
    assert fv.lib().fv_gemm_force_path(path) == 0
    try:
        out = fv.fv_gemm_bf16(ad, wd, bd, epilogue=epilogue, status=status)
        out2 = fv.fv_gemm_bf16(ad, wd, bd, epilogue=epilogue, status=status)
        torch.cuda.synchronize()
    finally:
        fv.lib().fv_gemm_force_path(0)
    assert int(status.item()) == 0
    assert torch.equal(out, out2)
    ref = O.linear(I.bf16_bits_to_f32(a), I.bf16_bits_to_f32(w), I.bf16_bits_to_f32(b))
    if epilogue == 1:
        ref = O.gelu_tanh(ref)
    err, cos = per_token_errors(bf16_host(out), ref)
    assert err <= MAX_ABS and cos >= MIN_COS, (err, cos)


def test_gemm_residual_epilogue_with_cache_copy():
    B, rows, N, K = 2, 100, 256, 512
    M = B * rows
    a = I.normal_bf16(80, (M, K)); w = I.normal_bf16(81, (N, K), 0.03); b = I.normal_bf16(82, (N,), 0.02)
    x = I.normal(83, (M, N)); mod = I.normal(84, (B, 6, N), 0.3)
    xd, modd = dev(x), dev(mod)
    aux = torch.zeros((M, N), dtype=torch.bfloat16, device=DEV)
    gamma = modd.data_ptr() + 5 * 4 * N      # gamma2 of image 0; images are 6*N floats apart
    fv.fv_gemm_bf16(bf16_dev(a), bf16_dev(w), bf16_dev(b), epilogue=2, out=xd, aux=aux, gamma=gamma, mod_stride=6 * N,
                    rows_per_image=rows)
    torch.cuda.synchronize()
    y = O.linear(I.bf16_bits_to_f32(a), I.bf16_bits_to_f32(w), I.bf16_bits_to_f32(b))
    g = np.repeat(mod[:, 5].astype(np.float64), rows, axis=0)
    ref = x.astype(np.float64) + g * y
    assert np.abs(xd.cpu().numpy() - ref).max() <= 2e-3
    err, cos = per_token_errors(bf16_host(aux), y)
    assert err <= MAX_ABS and cos >= MIN_COS


@pytest.mark.parametrize("path", [0, 2, 3, 4, 5, 6, 7])
@pytest.mark.parametrize("M,N,K,rows_per_image,splitk", [(300, 512, 256, 300, False), (7, 136, 72, 7, False), (1000, 1032, 1024, 500, False),
                                                          (2, 2048, 2048, 1, True), (130, 1920, 1920, 20, False)])
def test_gemm_fp32_epilogue(M, N, K, rows_per_image, splitk, path):
    """Epilogue 4: the fp32 value of acc + bias itself, on every kernel (one-CTA widths, CTA pairs, K split) and
    with images shorter than a warp's 32 rows (the row-per-thread store path)."""
    a = I.normal_bf16(85, (M, K)); w = I.normal_bf16(86, (N, K), 0.03); b = I.normal_bf16(87, (N,), 0.02)
    out = torch.full((M, N), 7.0, dtype=torch.float32, device=DEV)          # must be overwritten, not added to
    status = torch.zeros(1, dtype=torch.int32, device=DEV)
    ws = torch.zeros(fv.lib().fv_gemm_splitk_workspace_bytes(), dtype=torch.uint8, device=DEV) if splitk else None
    assert fv.lib().fv_gemm_force_path(path) == 0
    try:
        fv.fv_gemm_bf16(bf16_dev(a), bf16_dev(w), bf16_dev(b), epilogue=4, out=out, rows_per_image=rows_per_image, status=status,
                        splitk_ws=ws)
        torch.cuda.synchronize()
    finally:
        fv.lib().fv_gemm_force_path(0)
    assert int(status.item()) == 0
    ref = O.linear(I.bf16_bits_to_f32(a), I.bf16_bits_to_f32(w), I.bf16_bits_to_f32(b))
    assert np.abs(out.cpu().numpy() - ref).max() <= 2e-3      # fp32 accumulation of K bf16 x bf16 products


@pytest.mark.parametrize("rows,N,K", [(960, 2048, 2048), (820, 2048, 8192)])
def test_gemm_residual_epilogue_at_step_shapes(rows, N, K):
    """The out-projection and second MLP GEMM of the unpruned 32x32 / pruned 64x64 steps of the bench workload
    (B = 2), gate + residual into the fp32 stream, rows of two images inside one warp's 32 rows."""
    B = 2
    M = B * rows
    a = I.normal_bf16(88, (M, K), 1.0 if K <= 2048 else 0.5); w = I.normal_bf16(89, (N, K), 0.02); b = I.normal_bf16(90, (N,), 0.02)
    x = I.normal(91, (M, N)); mod = I.normal(92, (B, 6, N), 0.3)
    xd, modd = dev(x), dev(mod)
    status = torch.zeros(1, dtype=torch.int32, device=DEV)
    fv.fv_gemm_bf16(bf16_dev(a), bf16_dev(w), bf16_dev(b), epilogue=2, out=xd, gamma=modd.data_ptr() + 2 * 4 * N, mod_stride=6 * N,
                    rows_per_image=rows, status=status)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    y = O.linear(I.bf16_bits_to_f32(a), I.bf16_bits_to_f32(w), I.bf16_bits_to_f32(b))
    ref = x.astype(np.float64) + np.repeat(mod[:, 2].astype(np.float64), rows, axis=0) * y
    assert np.abs(xd.cpu().numpy() - ref).max() <= 2e-3


# ------------------------------------------------------------------ attention over the KV cache
ATTN_CASES = [  # B, rows, H, C, kv_len, cap
    (2, 85, 4, 256, 340, 344), (1, 300, 2, 256, 1000, 1024), (2, 128, 16, 1024, 485, 488), (1, 1, 4, 256, 1, 8),
    (1, 130, 2, 256, 129, 136), (2, 820, 16, 2048, 5223, 5224), (1, 37, 30, 1920, 640, 640),
    (1, 3277, 16, 2048, 13646, 13648),      # the 128x128 zero-shot step: 13 query-tile pairs x 107 key tiles per head
    (1, 1280, 16, 2048, 8525, 8528), (2, 260, 4, 256, 700, 704), (1, 52, 16, 2048, 6000, 6000),
    (1, 820, 16, 2048, 7245, 7248),         # the 64x64 step of the 2K workload: 64 query blocks, cut into one piece per SM
]


def _attention_reference_check(got, q, kk, vv, B, rows, H, C, kv_len):
    qf, kf, vf = (I.bf16_bits_to_f32(t).astype(np.float64) for t in (q, kk, vv))
    heads = range(H) if B * rows * kv_len * C < 3e9 else (0, H - 1)    # bound the oracle's time on the big cases
    hd = C // H
    for b in range(B):
        if len(heads) == H:
            ref = O.attention(qf[b * rows:(b + 1) * rows], kf[b, :kv_len], vf[b, :kv_len], H)
            err, cos = per_token_errors(got[b * rows:(b + 1) * rows], ref)
            assert err <= MAX_ABS and cos >= MIN_COS, (err, cos)
        else:
            for hh in heads:
                sl = slice(hh * hd, (hh + 1) * hd)
                ref = O.attention(qf[b * rows:(b + 1) * rows, sl], kf[b, :kv_len, sl], vf[b, :kv_len, sl], 1)
                err, cos = per_token_errors(got[b * rows:(b + 1) * rows, sl], ref)
                assert err <= MAX_ABS and cos >= MIN_COS, (err, cos)


@pytest.mark.parametrize("B,rows,H,C,kv_len,cap", ATTN_CASES)
def test_attention_over_kv_cache(B, rows, H, C, kv_len, cap):
    """Without scratch (one CTA per block of 256 queries of a head) and with it (the work cut into one piece per SM,
    the pieces of a query block merged in key order): both against the oracle, the split twice with identical bits,
    its arrival counters left at zero."""
    q = I.normal_bf16(90, (B * rows, C)); kk = I.normal_bf16(91, (B, cap, C)); vv = I.normal_bf16(92, (B, cap, C))
    vt = np.ascontiguousarray(vv.transpose(0, 2, 1))
    status = torch.zeros(1, dtype=torch.int32, device=DEV)
    qd, kd, vd = bf16_dev(q), bf16_dev(kk), bf16_dev(vt)
    out = fv.fv_attention(qd, kd, vd, B, rows, H, kv_len, status=status)
    ws = fv.fv_attention_workspace(DEV)
    out_s = fv.fv_attention(qd, kd, vd, B, rows, H, kv_len, status=status, workspace=ws)
    out_s2 = fv.fv_attention(qd, kd, vd, B, rows, H, kv_len, status=status, workspace=ws)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    assert torch.equal(out_s, out_s2)
    assert int(ws[:65536].view(torch.int32).abs().sum().item()) == 0
    _attention_reference_check(bf16_host(out), q, kk, vv, B, rows, H, C, kv_len)
    _attention_reference_check(bf16_host(out_s), q, kk, vv, B, rows, H, C, kv_len)


@pytest.mark.parametrize("ctas", [1, 2, 3, 5, 7, 16, 37, 97, 160])
@pytest.mark.parametrize("B,rows,H,C,kv_len,cap", [(2, 300, 2, 256, 1000, 1024), (1, 130, 2, 256, 129, 136), (2, 260, 4, 256, 700, 704),
                                                   (1, 820, 2, 256, 2000, 2000), (3, 37, 4, 256, 333, 336), (1, 1, 4, 256, 1, 8)])
def test_attention_split_into_any_number_of_pieces(B, rows, H, C, kv_len, cap, ctas):
    """The split with a forced piece count: pieces that end inside a query block, that hold the end of one block, whole
    blocks and the start of another, blocks merged from many parts, single-tile blocks, a ragged last key tile, and
    more pieces asked for than the work allows.  Every output row against the oracle."""
    q = I.normal_bf16(190, (B * rows, C)); kk = I.normal_bf16(191, (B, cap, C)); vv = I.normal_bf16(192, (B, cap, C))
    vt = np.ascontiguousarray(vv.transpose(0, 2, 1))
    status = torch.zeros(1, dtype=torch.int32, device=DEV)
    ws = fv.fv_attention_workspace(DEV)
    assert fv.lib().fv_attention_force_ctas(ctas) == 0
    try:
        out = fv.fv_attention(bf16_dev(q), bf16_dev(kk), bf16_dev(vt), B, rows, H, kv_len, status=status, workspace=ws)
        torch.cuda.synchronize()
    finally:
        fv.lib().fv_attention_force_ctas(0)
    assert int(status.item()) == 0
    assert int(ws[:65536].view(torch.int32).abs().sum().item()) == 0
    _attention_reference_check(bf16_host(out), q, kk, vv, B, rows, H, C, kv_len)


def test_attention_refuses_small_scratch():
    q = torch.zeros((8, 256), dtype=torch.bfloat16, device=DEV); k = torch.zeros((1, 8, 256), dtype=torch.bfloat16, device=DEV)
    with pytest.raises(fv.FvError) as e:
        fv.fv_attention(q, k, k.transpose(1, 2).contiguous(), 1, 8, 4, 8, workspace=torch.zeros(4096, dtype=torch.uint8, device=DEV))
    assert e.value.code == 3
