"""Brute-force numpy restatement of the method for tiny inputs (test helper).

It is written differently from the C oracle on purpose: window means come from
prefix sums, block means from reshaped slices, ranks from Python's sort of
explicit tuples, and the budget from a greedy walk over one merged list.  The
tests compare the oracle with it on small random inputs.
"""
from __future__ import annotations

import math
from typing import List, Tuple

import numpy as np


def unit_rows(K: np.ndarray) -> np.ndarray:
    K = K.astype(np.float64)
    n = np.sqrt((K * K).sum(1, keepdims=True))
    return K / np.maximum(n, 1e-12)


def block_size(N: int, div=32, lo=128, hi=256) -> int:
    return min(max(N // div, lo), hi)


def anchors(K: np.ndarray, W=64, div=32, lo=128, hi=256):
    X = unit_rows(K)
    N, d = X.shape
    mu_s = X.sum(0) / N
    b = block_size(N, div, lo, hi)
    nb = -(-N // b)
    mu_e = np.stack([X[t * b:(t + 1) * b].mean(0) for t in range(nb)])
    P = np.concatenate([np.zeros((1, d)), np.cumsum(X, 0)], 0)   # P[i] = sum of rows < i
    mu_c = np.empty_like(X)
    for i in range(N):
        l = max(0, i - W + 1)
        mu_c[i] = (P[i + 1] - P[l]) / (i + 1 - l)
    return X, mu_s, mu_e, mu_c, b


def cosines(X, mu_s, mu_e, mu_c, b):
    def cos_rows(A, B):
        num = (A * B).sum(1)
        den = np.maximum(np.sqrt((A * A).sum(1)), 1e-12) * np.maximum(np.sqrt((B * B).sum(1)), 1e-12)
        return num / den
    N = X.shape[0]
    blk = np.arange(N) // b
    return np.stack([-cos_rows(X, np.broadcast_to(mu_s, X.shape)),
                     -cos_rows(X, mu_e[blk]),
                     -cos_rows(X, mu_c)])


def minmax(v: np.ndarray) -> np.ndarray:
    lo, hi = v.min(), v.max()
    return (v - lo) / (hi - lo) if hi > lo else np.zeros_like(v)


def final_score(K: np.ndarray, prior=(0.4, 0.4, 0.2), beta=3.0, tau=0.6, kappa=10.0, p=0.10,
                n_sink=4, W=64, gate="surprise", ddof=0):
    X, mu_s, mu_e, mu_c, b = anchors(K, W=W)
    a = cosines(X, mu_s, mu_e, mu_c, b)
    an = np.stack([minmax(a[k]) for k in range(3)])
    N = K.shape[0]
    m = max(1, int(math.floor(p * N)))
    delta = np.array([np.sort(an[k])[::-1][:m].mean() - np.sort(an[k])[:m].mean() for k in range(3)])
    z = np.log(np.array(prior)) + beta * delta
    w = np.exp(z - z.max())
    w = w / w.sum()
    blend = (w[:, None] * an).sum(0)
    win = an.max(0)
    s = an.std(0, ddof=ddof)
    sn = minmax(s)
    sp = np.maximum(0.0, sn - sn.mean())
    if gate == "average":
        alpha = np.zeros(N)
    elif gate == "max":
        alpha = np.ones(N)
    else:
        alpha = 1.0 / (1.0 + np.exp(-kappa * (sp - tau)))
    star = ((1 - alpha) * blend + alpha * win).astype(np.float32)
    star[:min(n_sink, N)] = np.inf
    return dict(a=a, an=an, delta=delta, w=w, blend=blend, win=win, s=s, sn=sn, alpha=alpha,
                star=star, mu_s=mu_s, mu_e=mu_e, mu_c=mu_c, b=b, m=m)


def budgets_and_sets(star: np.ndarray, r: float, safeguard=0.20) -> Tuple[np.ndarray, List[List[int]], np.ndarray]:
    """star [H, N] -> (B_h, retained positions per head ascending, ranks [H, N])."""
    H, N = star.shape
    k = int(math.floor((1.0 - r) * N))
    n_safe = min(k, int(math.floor(safeguard * k)))
    triples = sorted(((-float(star[h, i]), h, i) for h in range(H) for i in range(N)))
    # greedy walk over the single merged order: a pair is kept if it is among its
    # head's first n_safe, or while free slots remain
    free = H * k - H * n_safe
    seen = [0] * H
    kept = [[] for _ in range(H)]
    # first find each head's safeguard members
    per_head = [[t for t in triples if t[1] == h] for h in range(H)]
    safe = [set(t[2] for t in per_head[h][:n_safe]) for h in range(H)]
    for neg, h, i in triples:
        if i in safe[h]:
            kept[h].append(i)
        elif free > 0:
            kept[h].append(i)
            free -= 1
        seen[h] += 1
    ranks = np.empty((H, N), np.int64)
    for h in range(H):
        for j, t in enumerate(per_head[h]):
            ranks[h, t[2]] = j
    return np.array([len(x) for x in kept]), [sorted(x) for x in kept], ranks
