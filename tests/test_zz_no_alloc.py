"""nkv_budget_static, the budget entry point for callers that cannot allocate device memory.

Such callers (a host living inside a fixed memory pool, a plugin that only receives its inputs
and outputs) cannot give nkv_budget the scratch buffer it wants, so the library keeps that
scratch in a fixed array of its own.  The test calls the new entry point through the C ABI twice
in a row, on different inputs, and requires the same budgets as nkv_budget, bit for bit (budgets
are integers, so the tolerance of the other budget tests applies: none).  The second call runs on
scratch that still holds the first call's contents, which is the situation the entry point has
to cope with.  The file sorts last so that a run that stops at the first failure has already
run every other test.
"""
import numpy as np
import pytest
import torch

from paper_2605_26678_b200 import nkv

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def _scores(G, H, N, seed, dense):
    rng = np.random.default_rng(seed)
    s = rng.random((G, H, N)).astype(np.float32) ** 3
    s *= rng.uniform(0.05, 1.0, size=(G, H, 1)).astype(np.float32)
    if dense:
        s = np.round(s * 64) / 64          # many exact ties
    s[:, :, :4] = np.inf
    return torch.from_numpy(s).to(DEV)


def test_static_scratch_budgets_match_nkv_budget_on_two_calls_in_a_row():
    first = _scores(3, 8, 5000, seed=1, dense=False)
    second = _scores(2, 4, 1777, seed=2, dense=True)
    out1 = torch.empty((3, 8), dtype=torch.int32, device=DEV)
    out2 = torch.empty((2, 4), dtype=torch.int32, device=DEV)
    got1 = nkv.nkv_budget_static(first, 0.75, out=out1)
    got2 = nkv.nkv_budget_static(second, 0.9, out=out2)      # reuses the scratch the first call left behind
    torch.cuda.synchronize()
    want1 = nkv.nkv_budget(first, 0.75)
    want2 = nkv.nkv_budget(second, 0.9)
    torch.cuda.synchronize()
    assert torch.equal(got1, want1)
    assert torch.equal(got2, want2)
    assert int(got1.sum()) == 3 * 8 * nkv.nkv_keep_per_head(5000, 0.75)
    assert int(got2.sum()) == 2 * 4 * nkv.nkv_keep_per_head(1777, 0.9)


def test_static_scratch_rejects_more_heads_than_it_can_hold():
    G = nkv.NKV_STATIC_MAX_UNITS // 8 + 1
    a = torch.zeros((G, 8, 16), dtype=torch.float32, device=DEV)
    with pytest.raises(nkv.NkvError) as e:
        nkv.nkv_budget_static(a, 0.5)
    assert e.value.status == nkv.NKV_ERR_WORKSPACE
