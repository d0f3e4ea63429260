"""The two identities the tensor-core key passes rest on, checked on the CPU against the oracle.

1. Section 2.2-2.3, current memory: with g_ij = k_hat_i . k_hat_j, the window sum S_i satisfies
   k_hat_i . S_i = sum of g over the band j in window(i), and ||S_i||^2 follows tile by tile from an exact
   restart value (the Gram block of the previous tile's last W rows) plus the prefix sum of
   (2 c_i - g_ii) - (2 f_{i-W} - g_{i-W,i-W}), c and f being the backward and forward band sums.
2. An fp32 number is the exact sum of three bf16 numbers (hi, mid, lo), so a dot product with fp32
   anchors can be taken as three dot products with bf16 anchors.
"""
import numpy as np
import pytest
import torch

import oracle

W, TILE = 64, 128


def _window_anomaly_from_gram(K):
    """a_c of one head from band sums of the Gram matrix, organised as the kernel organises it."""
    K = np.asarray(K, np.float64)
    N = K.shape[0]
    norm = np.linalg.norm(K, axis=1)
    w = 1.0 / np.maximum(norm, 1e-12)
    G = (K @ K.T) * w[:, None] * w[None, :]
    g = np.diag(G).copy()
    c = np.array([G[i, max(0, i - W + 1):i + 1].sum() for i in range(N)])   # backward band
    f = np.array([G[i, i:min(N, i + W)].sum() for i in range(N)])           # forward band
    T = np.empty(N)
    anchor = 0.0
    for i0 in range(0, N, TILE):
        rows = np.arange(i0, min(N, i0 + TILE))
        add = 2.0 * c[rows] - g[rows]
        rem = np.array([2.0 * f[i - W] - g[i - W] if i - W >= 0 else 0.0 for i in rows])
        T[rows] = anchor + np.cumsum(add - rem)
        last = i0 + TILE - 1
        if last < N:   # exact restart value: the Gram block of the tile's last W rows
            anchor = G[last - W + 1:last + 1, last - W + 1:last + 1].sum()
    return -c / np.maximum(np.sqrt(np.maximum(T, 0.0)), 1e-12)


@pytest.mark.parametrize("N,d,seed", [(5, 16, 0), (64, 32, 1), (65, 32, 2), (300, 64, 3), (777, 128, 4)])
def test_band_sums_of_the_gram_matrix_give_the_window_anomaly(N, d, seed):
    rng = np.random.default_rng(seed)
    K = (rng.standard_normal((N, d)) + 0.5 * rng.standard_normal((1, d))).astype(np.float32)
    if N > 10:
        K[N // 3] = 0.0   # a zero key scores 0 and adds nothing to any window
    ref = oracle.score_head(K).a_raw[2]
    got = _window_anomaly_from_gram(K)
    assert np.allclose(got, ref, rtol=0, atol=1e-9)


def test_restart_value_equals_the_running_value():
    """The per-tile restart is not a correction: in exact arithmetic it equals the prefix sum's last value."""
    rng = np.random.default_rng(7)
    K = rng.standard_normal((3 * TILE, 48))
    w = 1.0 / np.linalg.norm(K, axis=1)
    G = (K @ K.T) * w[:, None] * w[None, :]
    kh = K * w[:, None]
    for last in (TILE - 1, 2 * TILE - 1):
        S = kh[last - W + 1:last + 1].sum(axis=0)
        assert abs(G[last - W + 1:last + 1, last - W + 1:last + 1].sum() - S @ S) < 1e-9


def test_three_bf16_parts_carry_an_fp32_number_exactly():
    g = torch.Generator().manual_seed(3)
    x = torch.randn(4096, generator=g) * torch.logspace(-6, 3, 4096)
    hi = x.to(torch.bfloat16)
    r1 = x - hi.float()
    mid = r1.to(torch.bfloat16)
    lo = (r1 - mid.float()).to(torch.bfloat16)
    assert torch.equal(hi.float() + mid.float() + lo.float(), x)
    # the parts are what they are meant to be: each a bf16 rounding of what is left
    assert torch.all((r1.abs() <= x.abs() * 2.0 ** -8) | (x == 0))
