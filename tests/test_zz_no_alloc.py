"""fv_prune_select_static -- the selection entry point for callers that cannot allocate device memory
(its scratch is a fixed array inside the library) -- must give exactly what fv_prune_select gives with a
caller-provided workspace.  Collected last on purpose: a run that stops at the first failure has
then already run every other test.  Two calls in a row with different shapes check that whatever the
shared scratch still holds from the previous call does not leak into the next."""
import numpy as np
import pytest
import torch

from paper_2503_23367_b200 import binding as fv
from paper_2503_23367_b200 import inputs as I

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def _both(B, h, w, C, keep, seed):
    x = torch.from_numpy(I.token_map(seed, B, h, w, C, "structured")).to(DEV)
    ref = fv.fv_prune_select(x, h, w, keep, want_inv=True, want_score=True, want_near_tie=True)
    n, k = h * w, ref["k"]
    out = {"idx": torch.full((B, k), -7, dtype=torch.int32, device=DEV),
           "inv": torch.full((B, n), -7, dtype=torch.int32, device=DEV),
           "score": torch.full((B, n), float("nan"), dtype=torch.float32, device=DEV),
           "near_tie": torch.full((B,), -7, dtype=torch.int32, device=DEV)}
    assert fv.fv_prune_select_static(x, h, w, keep, out) == k
    torch.cuda.synchronize()
    # same kernels, same arithmetic order: integers exact, and the scores bit-identical
    assert torch.equal(out["idx"], ref["idx"])
    assert torch.equal(out["inv"], ref["inv"])
    assert torch.equal(out["near_tie"], ref["near_tie"])
    assert np.array_equal(out["score"].cpu().numpy().view(np.uint32), ref["score"].cpu().numpy().view(np.uint32))


def test_static_scratch_selection_matches_workspace_selection_twice_in_a_row():
    _both(2, 64, 64, 2048, 0.2, seed=11)      # 2.2 MiB of scratch
    _both(3, 13, 13, 256, 0.6, seed=12)       # a smaller call right after: stale scratch must not matter
    _both(2, 64, 64, 2048, 0.2, seed=13)      # and the large shape again over the small call's leftovers


def test_static_scratch_refuses_what_does_not_fit_and_bad_arguments():
    cap = fv.lib().fv_prune_select_static_capacity()
    assert cap == 8 << 20
    B, h, w, C = 4, 128, 128, 2048            # needs 16.5 MiB of scratch
    assert fv.lib().fv_prune_select_workspace_bytes(B, h * w, C) > cap
    x = torch.zeros((B, h * w, C), dtype=torch.float32, device=DEV)
    out = {"idx": torch.zeros((B, fv.fv_k_for(0.2, h, w)), dtype=torch.int32, device=DEV)}
    with pytest.raises(fv.FvError) as e:
        fv.fv_prune_select_static(x, h, w, 0.2, out)
    assert e.value.code == 3                  # FV_ERR_CAPACITY
    with pytest.raises(fv.FvError) as e:
        fv.fv_prune_select_static(x, h, w, 1.5, out)
    assert e.value.code == 1                  # FV_ERR_INVALID_ARG
