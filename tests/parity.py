"""Helpers shared by the GPU parity tests: run both sides on the same bytes and compare.

Tolerances (fp32 scores): |delta| <= 1e-4 absolute or 1e-4 relative.  Integer outputs
(budgets, positions, ranks) and compacted bytes are compared exactly; when the GPU's own
scores feed the integer stages, a token may legitimately swap in or out only if its oracle
score lies within the tolerance (plus the observed score difference of that token) of a
threshold that the selection used, and such swaps are counted.
"""
from __future__ import annotations

from dataclasses import dataclass
from typing import List

import numpy as np
import torch

import oracle
from paper_2605_26678_b200 import nkv

TOL = 1e-4


def oracle_params(p: "nkv.Params") -> "oracle.Params":
    q = oracle.default_params()
    for name in ("window", "n_sink", "block_div", "block_min", "block_max", "gate_mode", "top_frac", "beta",
                 "tau", "kappa", "safeguard"):
        setattr(q, name, getattr(p, name))
    for k in range(3):
        q.prior[k] = p.prior[k]
    return q


def close(got, want, tol=TOL) -> np.ndarray:
    got = np.asarray(got, np.float64)
    want = np.asarray(want, np.float64)
    both_inf = np.isinf(got) & np.isinf(want) & (np.sign(got) == np.sign(want))
    with np.errstate(invalid="ignore"):
        err = np.abs(got - want)
        ok = (err <= tol) | (err <= tol * np.abs(want))
    return ok | both_inf


def assert_close(got, want, what, tol=TOL):
    ok = close(got, want, tol)
    if not ok.all():
        bad = np.argwhere(~ok)
        first = tuple(bad[0])
        raise AssertionError("%s: %d of %d outside tolerance %g; first at %s: got %r want %r" % (
            what, (~ok).sum(), ok.size, tol, first, np.asarray(got)[first], np.asarray(want)[first]))


def raw_rows(x: torch.Tensor) -> np.ndarray:
    """bf16 / fp16 -> uint16 view, fp32 -> float32, on host."""
    x = x.detach().cpu().contiguous()
    if x.dtype in (torch.bfloat16, torch.float16):
        return x.view(torch.int16).numpy().view(np.uint16)
    return x.numpy()


@dataclass
class SwapReport:
    heads: int = 0
    heads_with_swaps: int = 0
    swapped_tokens: int = 0
    budget_mismatch_heads: int = 0


def compare_selection(a_star_oracle: np.ndarray, sel: "oracle.GroupSelection", gpu_budgets: np.ndarray,
                      gpu_idx: np.ndarray, gpu_offsets: np.ndarray, report: SwapReport, tol=TOL, n_safe=None,
                      a_star_gpu=None):
    """One group: exact match, or every differing token is a near-tie of a threshold the selection used.

    The thresholds are, per head, the smallest retained score and the n_safe-th best score (the safeguard
    threshold), and the smallest score retained anywhere in the group (the cross-head competition).  A token
    may change sides only if its oracle score is within tol + |gpu - oracle| of one of them: two scores that
    each carry at most `tol` of error can swap only when they are that close."""
    H, N = a_star_oracle.shape
    finite = np.where(np.isfinite(a_star_oracle), a_star_oracle, -np.inf)
    finite_max = float(finite.max())
    head_thr = []
    for h in range(H):
        rows = sel.idx[sel.offsets[h]:sel.offsets[h + 1]]
        t = float(a_star_oracle[h, rows].min()) if len(rows) else np.inf
        thr = [finite_max if np.isinf(t) else t]
        if n_safe is not None and 0 < n_safe <= N:
            t2 = float(np.sort(a_star_oracle[h])[::-1][n_safe - 1])
            thr.append(finite_max if np.isinf(t2) else t2)
        head_thr.append(thr)
    group_thr = min(t[0] for t in head_thr)
    for h in range(H):
        report.heads += 1
        want = set(sel.idx[sel.offsets[h]:sel.offsets[h + 1]].tolist())
        got = set(gpu_idx[gpu_offsets[h]:gpu_offsets[h + 1]].tolist())
        assert len(got) == gpu_budgets[h], "head %d: %d positions for budget %d" % (h, len(got), gpu_budgets[h])
        diff = want ^ got
        if gpu_budgets[h] != sel.budgets[h]:
            report.budget_mismatch_heads += 1
            assert diff, "head %d: budgets differ but the position sets do not" % h
        if not diff:
            continue
        report.heads_with_swaps += 1
        report.swapped_tokens += len(diff)
        for i in diff:
            s = float(a_star_oracle[h, i])
            near = min([abs(s - t) for t in head_thr[h]] + [abs(s - group_thr)])
            seen = abs(float(a_star_gpu[h, i]) - s) if a_star_gpu is not None else tol
            assert near <= (tol + seen) * max(1.0, abs(s)), (
                "head %d token %d (score %.7f) changed sides but is %.3g away from the thresholds %s / %.7f"
                % (h, i, s, near, head_thr[h], group_thr))


def gpu_group_outputs(res: "nkv.Compressed", g: int):
    return (res.budgets[g].cpu().numpy(), res.idx[g].cpu().numpy(), res.head_offsets[g].cpu().numpy())


def check_group_against_oracle(K: torch.Tensor, V: torch.Tensor, res: "nkv.Compressed", g: int, r: float,
                               params: "nkv.Params", report: SwapReport):
    """Full comparison of group g of a fused GPU result against the oracle."""
    op = oracle_params(params)
    ref = oracle.compress_group(K[g].cpu(), V[g].cpu(), r, op)
    if res.a_star is not None:
        assert_close(res.a_star[g].cpu().numpy(), ref.a_star, "a_star group %d" % g)
    b, idx, offs = gpu_group_outputs(res, g)
    H = K.shape[1]
    assert b.sum() == ref.sel.budgets.sum() == offs[H]
    assert np.array_equal(offs[1:] - offs[:-1], b)
    compare_selection(ref.a_star, ref.sel, b, idx, offs, report, n_safe=nkv.nkv_safeguard_count(K.shape[2], r, params),
                      a_star_gpu=None if res.a_star is None else res.a_star[g].cpu().numpy())
    # integer stages are exact given the GPU's own scores
    if res.a_star is not None:
        own = oracle.budget_select(res.a_star[g].cpu().numpy(), r, op)
        assert np.array_equal(own.budgets, b), "budgets differ from the oracle run on the GPU's scores"
        assert np.array_equal(own.idx, idx), "positions differ from the oracle run on the GPU's scores"
    # compacted bytes are the gathered rows
    k_out, v_out = raw_rows(res.k_out[g]), raw_rows(res.v_out[g])
    Kr, Vr = raw_rows(K[g]), raw_rows(V[g])
    for h in range(H):
        rows = idx[offs[h]:offs[h + 1]]
        assert np.array_equal(k_out[offs[h]:offs[h + 1]], Kr[h][rows]), "K bytes head %d" % h
        assert np.array_equal(v_out[offs[h]:offs[h + 1]], Vr[h][rows]), "V bytes head %d" % h
    return ref
