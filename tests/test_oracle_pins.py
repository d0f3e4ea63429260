"""Pins of the CPU oracle against what the paper and the mathematics fix.

None of these tests touches the CUDA path.  They use: the constants the paper
prints (tests/golden), closed forms on constructed inputs, invariants the paper
states, named ablation variants that reduce to textbook computations, and brute
force on tiny inputs (tests/bruteforce.py).
"""
import math
import os

import numpy as np
import pytest

import oracle
from tests import bruteforce as bf

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def _read_table(name):
    rows = []
    with open(os.path.join(GOLDEN, name)) as f:
        for line in f:
            line = line.strip()
            if line and not line.startswith("#"):
                rows.append(line.split())
    return rows


def _rand_keys(rng, N, d, structured=True):
    K = rng.standard_normal((N, d)).astype(np.float32)
    if structured:
        K += 2.0 * rng.standard_normal((1, d)).astype(np.float32)
        seg = np.repeat(rng.standard_normal((max(1, N // 37) + 1, d)).astype(np.float32), 37, 0)[:N]
        K += 0.5 * seg
    return K


# --------------------------------------------------------------------------- constants
def test_defaults_match_paper_hyperparameters():
    p = oracle.default_params()
    want = {k: float(v) for k, v in _read_table("hyperparameters.txt")}
    assert (p.prior[0], p.prior[1], p.prior[2]) == (want["prior_s"], want["prior_e"], want["prior_c"])
    assert p.block_div == want["block_div"] and p.block_min == want["block_min"]
    assert p.block_max == want["block_max"] and p.window == want["window"]
    assert p.n_sink == want["n_sink"] and p.beta == want["beta"] and p.tau == want["tau"]
    assert p.kappa == want["kappa"] and p.safeguard == want["safeguard"] and p.top_frac == want["top_frac"]
    assert p.gate_mode == oracle.GATE_SURPRISE


def test_block_size_table():
    for N, b, nb in _read_table("block_size.txt"):
        assert oracle.block_size(int(N)) == int(b)
        assert oracle.num_blocks(int(N)) == int(nb)


def test_budget_count_table():
    for N, r, k, ns in _read_table("budget_counts.txt"):
        assert oracle.keep_per_head(int(N), float(r)) == int(k)
        assert oracle.safeguard_count(int(N), float(r)) == int(ns)


def test_top_count():
    assert oracle.top_count(4096) == 409 and oracle.top_count(5) == 1 and oracle.top_count(32768) == 3276


# --------------------------------------------------------------------------- closed forms
def test_identical_keys_degenerate():
    """Every key equal to every anchor: a = -1 everywhere, normalised scores 0,
    gaps 0, weights = prior (Section 2.4, 'fall back on the prior'), surprise 0."""
    K = np.tile(np.array([[0.0, -4.0, 0.0, 0.0]], np.float32), (200, 1))   # exact arithmetic
    h = oracle.score_head(K)
    assert np.all(h.a_raw == -1.0)
    assert np.all(h.delta == 0.0)
    assert np.allclose(h.w, [0.4, 0.4, 0.2], atol=1e-15)
    assert h.s_min == 0.0 and h.s_max == 0.0 and h.s_mean == 0.0
    assert np.all(np.isinf(h.a_star[:4])) and np.all(h.a_star[4:] == 0.0)
    assert np.all(h.inv_norm == 0.25)


def test_first_token_current_anchor_is_itself():
    rng = np.random.default_rng(1)
    h = oracle.score_head(_rand_keys(rng, 150, 16), want_mu_c=True)
    assert abs(h.a_raw[2, 0] + 1.0) < 1e-12


def test_two_direction_closed_form():
    """Keys alternate e1, e2 (N even, one block): mu_s = mu_e = (e1+e2)/2, so
    cos = 1/sqrt(2) for every token on both scales; the window ending at token i
    holds p keys of i's own direction and q of the other, so cos = p/sqrt(p^2+q^2)."""
    N, d = 100, 8
    K = np.zeros((N, d), np.float32)
    K[0::2, 0] = 5.0   # scale must not matter
    K[1::2, 1] = 0.25
    h = oracle.score_head(K, want_mu_c=True)
    assert np.allclose(h.a_raw[0], -1 / math.sqrt(2), atol=1e-12)
    assert np.allclose(h.a_raw[1], -1 / math.sqrt(2), atol=1e-12)
    for i in range(N):
        n = min(i + 1, 64)
        p_own = (n + 1) // 2
        q = n - p_own
        assert abs(h.a_raw[2, i] + p_own / math.sqrt(p_own ** 2 + q ** 2)) < 1e-12
    assert np.allclose(h.mu_s[:2], 0.5) and np.allclose(h.mu_s[2:], 0.0)


def test_window_length_and_partial_block():
    """Orthonormal keys e_i: mu_c(i) averages min(i+1, W) distinct unit vectors,
    so cos = 1/sqrt(min(i+1, W)); block t has |B| members, cos = 1/sqrt(|B|);
    global cos = 1/sqrt(N).  N is not a multiple of b, so the last block is short."""
    N = 300
    K = np.eye(N, dtype=np.float32)
    h = oracle.score_head(K)
    i = np.arange(N)
    assert np.allclose(h.a_raw[2], -1 / np.sqrt(np.minimum(i + 1, 64)), atol=1e-12)
    b = 128
    size = np.where(i // b == 2, N - 2 * b, b)
    assert np.allclose(h.a_raw[1], -1 / np.sqrt(size), atol=1e-12)
    assert np.allclose(h.a_raw[0], -1 / math.sqrt(N), atol=1e-12)


def test_zero_key_gives_zero_cosine():
    rng = np.random.default_rng(5)
    K = _rand_keys(rng, 90, 8)
    K[17] = 0.0
    h = oracle.score_head(K)
    assert np.all(h.a_raw[:, 17] == 0.0)
    assert np.all(np.isfinite(h.a_star[4:]))


# --------------------------------------------------------------------------- invariants
@pytest.mark.parametrize("N,d", [(64, 8), (257, 16), (300, 64)])
def test_positive_rescaling_invariance(N, d):
    rng = np.random.default_rng(N)
    K = _rand_keys(rng, N, d)
    scale = rng.uniform(0.25, 8.0, size=(N, 1)).astype(np.float32)
    scale = 2.0 ** np.round(np.log2(scale))      # powers of two: products are exact in fp32
    h1, h2 = oracle.score_head(K), oracle.score_head(K * scale)
    assert np.allclose(h1.a_raw, h2.a_raw, atol=1e-13)
    assert np.array_equal(h1.a_star, h2.a_star)


def test_minmax_uses_the_heads_own_extremes():
    """The oracle's lo / hi are the extremes of its own raw anomalies, every normalised scale
    attains 0 and 1, and the head statistics are consistent with them (Section 2.3)."""
    rng = np.random.default_rng(11)
    K = _rand_keys(rng, 200, 16)
    h = oracle.score_head(K)
    assert np.array_equal(h.lo, h.a_raw.min(1)) and np.array_equal(h.hi, h.a_raw.max(1))
    an = (h.a_raw - h.lo[:, None]) / (h.hi - h.lo)[:, None]
    for k in range(3):
        assert an[k].min() == 0.0 and an[k].max() == 1.0
    # the reliability gap of a scale is a difference of means of values in [0, 1]
    assert np.all(h.delta >= 0.0) and np.all(h.delta <= 1.0)


def _two_direction_case():
    """Keys alternate between two orthogonal directions (N = 100, one block, W = 64).  Then a_s and a_e are
    constant (their normalised scales are identically 0) and the window anomaly is known in closed form:
    a_c(i) = -p / sqrt(p^2 + q^2) with p keys of i's own direction and q of the other in the window."""
    N, d = 100, 8
    K = np.zeros((N, d), np.float32)
    K[0::2, 0] = 5.0
    K[1::2, 1] = 0.25
    i = np.arange(N)
    n = np.minimum(i + 1, 64)
    p_own = (n + 1) // 2
    q = n - p_own
    a_c = -p_own / np.sqrt(p_own.astype(np.float64) ** 2 + q ** 2)
    return K, a_c


def test_surprise_gate_chain_closed_form():
    """Section 2.4 and Appendix A on an input where every quantity follows by hand.

    With a_tilde_s = a_tilde_e = 0 and x = a_tilde_c: the population std of (0, 0, x) is x sqrt(2)/3, so the
    surprise is proportional to x and its per-head min-max is x itself; centring and rectifying give
    s' = max(0, x - mean x); the gate is sigma(kappa (s' - tau)); Delta_s = Delta_e = 0 and Delta_c is the
    gap of x; the blend is w_c x, the winner is x, so a_star = (1 - alpha) w_c x + alpha x."""
    K, a_c = _two_direction_case()
    N = len(a_c)
    x = (a_c - a_c.min()) / (a_c.max() - a_c.min())
    m = 10                                              # max(1, floor(0.10 * 100))
    srt = np.sort(x)
    delta_c = srt[-m:].mean() - srt[:m].mean()
    z = np.log(np.array([0.4, 0.4, 0.2])) + 3.0 * np.array([0.0, 0.0, delta_c])
    w = np.exp(z - z.max())
    w /= w.sum()
    s_prime = np.maximum(0.0, x - x.mean())
    alpha = 1.0 / (1.0 + np.exp(-10.0 * (s_prime - 0.60)))
    want = (1.0 - alpha) * w[2] * x + alpha * x

    h = oracle.score_head(K)
    assert np.allclose(h.delta, [0.0, 0.0, delta_c], atol=1e-12)
    assert np.allclose(h.w, w, atol=1e-12)
    # surprise statistics: min 0, max sqrt(2)/3 (at x = 1), mean of the normalised surprise = mean x
    assert abs(h.s_min) < 1e-12 and abs(h.s_max - math.sqrt(2.0) / 3.0) < 1e-12
    assert abs(h.s_mean - x.mean()) < 1e-12
    assert np.all(np.isinf(h.a_star[:4]))
    assert np.allclose(h.a_star[4:], want[4:].astype(np.float32), atol=1e-7)

    # the gate grows with the surprise: alpha = (a_star - w_c x) / (x - w_c x) where x > 0
    pos = np.arange(N)[4:][x[4:] > 1e-6]
    a64 = h.a_star.astype(np.float64)
    alpha_seen = (a64[pos] - w[2] * x[pos]) / (x[pos] - w[2] * x[pos])
    order = np.argsort(x[pos], kind="stable")
    assert np.all(np.diff(alpha_seen[order]) >= -1e-6)

    # plausible misreadings of Appendix A give visibly different scores on this input, so the
    # comparison above would catch them: threshold applied to the normalised surprise before
    # centring, and rectifying before centring
    alt1 = 1.0 / (1.0 + np.exp(-10.0 * (x - 0.60)))
    alt2 = 1.0 / (1.0 + np.exp(-10.0 * ((np.maximum(0.0, x) - x.mean()) - 0.60)))
    for alt in (alt1, alt2):
        other = (1.0 - alt) * w[2] * x + alt * x
        assert np.max(np.abs(other[4:] - want[4:])) > 5e-4    # 5000 times the tolerance of the comparison


def test_gate_parameters_move_the_closed_form():
    """The same input with other (beta, tau, kappa, priors): every constant enters where Section 2.4 puts it."""
    K, a_c = _two_direction_case()
    x = (a_c - a_c.min()) / (a_c.max() - a_c.min())
    p = oracle.default_params()
    p.beta, p.tau, p.kappa = 1.5, 0.2, 4.0
    p.prior[0], p.prior[1], p.prior[2] = 0.5, 0.2, 0.3
    srt = np.sort(x)
    delta_c = srt[-10:].mean() - srt[:10].mean()
    z = np.log(np.array([0.5, 0.2, 0.3])) + 1.5 * np.array([0.0, 0.0, delta_c])
    w = np.exp(z - z.max())
    w /= w.sum()
    alpha = 1.0 / (1.0 + np.exp(-4.0 * (np.maximum(0.0, x - x.mean()) - 0.2)))
    want = (1.0 - alpha) * w[2] * x + alpha * x
    h = oracle.score_head(K, p)
    assert np.allclose(h.w, w, atol=1e-12)
    assert np.allclose(h.a_star[4:], want[4:].astype(np.float32), atol=1e-7)
    # with the gate half open the two misreadings of the centring order are far away
    alt1 = 1.0 / (1.0 + np.exp(-4.0 * (x - 0.2)))
    alt2 = 1.0 / (1.0 + np.exp(-4.0 * ((np.maximum(0.0, x) - x.mean()) - 0.2)))
    for alt in (alt1, alt2):
        other = (1.0 - alt) * w[2] * x + alt * x
        assert np.max(np.abs(other[4:] - want[4:])) > 2e-2


def test_weights_softmax_properties():
    rng = np.random.default_rng(3)
    K = _rand_keys(rng, 180, 16)
    h = oracle.score_head(K)
    assert abs(h.w.sum() - 1.0) < 1e-15
    z = np.log([0.4, 0.4, 0.2]) + 3.0 * h.delta
    assert np.allclose(h.w, np.exp(z) / np.exp(z).sum(), atol=1e-15)
    p = oracle.default_params()
    p.beta = 0.0
    assert np.allclose(oracle.score_head(K, p).w, [0.4, 0.4, 0.2], atol=1e-15)
    # the more discriminative scale gains weight relative to the prior ratio
    order = np.argsort(h.delta)
    ratio = h.w / np.array([0.4, 0.4, 0.2])
    assert ratio[order[0]] <= ratio[order[1]] <= ratio[order[2]]


def test_gate_bounds_and_ablation_modes():
    """blend <= a* <= max for every token; 'only average' returns the blend and
    'only max' the winner (router ablation table)."""
    rng = np.random.default_rng(8)
    K = _rand_keys(rng, 260, 32)
    ref = bf.final_score(K)
    h = oracle.score_head(K)
    body = slice(4, None)
    assert np.all(h.a_star[body] >= ref["blend"][body].astype(np.float32) - 1e-6)
    assert np.all(h.a_star[body] <= ref["win"][body].astype(np.float32) + 1e-6)
    p = oracle.default_params()
    p.gate_mode = oracle.GATE_AVERAGE
    assert np.allclose(oracle.score_head(K, p).a_star[body], ref["blend"][body], atol=1e-6)
    p.gate_mode = oracle.GATE_MAX
    assert np.allclose(oracle.score_head(K, p).a_star[body], ref["win"][body], atol=1e-6)


def test_sample_vs_population_std_is_immaterial():
    rng = np.random.default_rng(21)
    K = _rand_keys(rng, 140, 16)
    a0, a1 = bf.final_score(K, ddof=0), bf.final_score(K, ddof=1)
    assert np.allclose(a0["sn"], a1["sn"], atol=1e-13)
    assert np.allclose(a0["star"][4:], a1["star"][4:], atol=1e-7)


def test_single_anchor_special_case_is_key_distinctiveness():
    """prior (1,0,0) with beta=0 and the gate off: the score is the min-max of
    -cos(k_hat, mean k_hat), the single-anchor variant of the ablation table."""
    rng = np.random.default_rng(13)
    K = _rand_keys(rng, 333, 24)
    p = oracle.default_params()
    p.prior[0], p.prior[1], p.prior[2] = 1.0, 1e-300, 1e-300
    p.beta = 0.0
    p.gate_mode = oracle.GATE_AVERAGE
    h = oracle.score_head(K, p)
    X = K.astype(np.float64) / np.linalg.norm(K.astype(np.float64), axis=1, keepdims=True)
    mu = X.mean(0)
    score = -(X @ mu) / np.linalg.norm(mu)
    score = (score - score.min()) / (score.max() - score.min())
    assert np.allclose(h.a_star[4:], score[4:].astype(np.float32), atol=1e-6)


# --------------------------------------------------------------------------- brute force
@pytest.mark.parametrize("N,d,seed", [(5, 4, 0), (33, 8, 1), (64, 8, 2), (129, 16, 3), (300, 16, 4)])
def test_scores_match_bruteforce(N, d, seed):
    rng = np.random.default_rng(seed)
    K = _rand_keys(rng, N, d, structured=(seed % 2 == 0))
    h = oracle.score_head(K, want_mu_c=True)
    ref = bf.final_score(K)
    assert np.allclose(h.mu_s, ref["mu_s"], atol=1e-13)
    assert np.allclose(h.mu_e, ref["mu_e"], atol=1e-13)
    assert np.allclose(h.mu_c, ref["mu_c"], atol=1e-12)
    assert np.allclose(h.a_raw, ref["a"], atol=1e-12)
    assert np.allclose(h.delta, ref["delta"], atol=1e-12)
    assert np.allclose(h.w, ref["w"], atol=1e-12)
    assert h.m == ref["m"]
    assert np.allclose(h.s_mean, ref["sn"].mean(), atol=1e-12)
    fin = np.isfinite(ref["star"])
    assert np.array_equal(np.isinf(h.a_star), ~fin)
    assert np.allclose(h.a_star[fin], ref["star"][fin], atol=2e-7)


def test_bf16_input_is_widened_exactly():
    torch = pytest.importorskip("torch")
    rng = np.random.default_rng(2)
    K32 = torch.from_numpy(_rand_keys(rng, 70, 8))
    Kb = K32.to(torch.bfloat16)
    h1 = oracle.score_head(Kb)
    h2 = oracle.score_head(Kb.to(torch.float32))
    assert np.array_equal(h1.a_raw, h2.a_raw) and np.array_equal(h1.a_star, h2.a_star)


@pytest.mark.parametrize("H,N,r,seed", [(1, 20, 0.5, 0), (3, 40, 0.75, 1), (4, 64, 0.25, 2),
                                        (8, 50, 0.9, 3), (2, 30, 0.0, 4)])
def test_budget_and_selection_match_bruteforce(H, N, r, seed):
    rng = np.random.default_rng(seed)
    star = rng.random((H, N)).astype(np.float32)
    star *= rng.uniform(0.2, 1.0, size=(H, 1)).astype(np.float32)     # heads differ in scale
    if seed % 2 == 1:
        star = np.round(star * 8) / 8                                  # many exact ties
    star[:, :4] = np.inf
    sel = oracle.budget_select(star, r, want_ranks=True)
    B, kept, ranks = bf.budgets_and_sets(star, r)
    k = int(math.floor((1 - r) * N))
    assert np.array_equal(sel.budgets, B)
    assert sel.budgets.sum() == H * k == sel.offsets[-1]
    assert np.all(sel.budgets >= int(math.floor(0.2 * k)))
    for h in range(H):
        got = sel.idx[sel.offsets[h]:sel.offsets[h + 1]].tolist()
        assert got == kept[h]
        assert got == sorted(got)
        if k >= 4 and sel.budgets[h] >= 4:
            assert got[:4] == [0, 1, 2, 3]
        assert sorted(sel.ranks[h].tolist()) == list(range(N))
    assert np.array_equal(sel.ranks, ranks)


def test_uniform_budget_when_safeguard_is_one():
    """safeguard = 1.0 leaves nothing to compete for: the uniform-budget ablation."""
    rng = np.random.default_rng(9)
    star = rng.random((4, 48)).astype(np.float32)
    p = oracle.default_params()
    p.safeguard = 1.0
    sel = oracle.budget_select(star, 0.5, p)
    assert sel.budgets.tolist() == [24] * 4
    for h in range(4):
        got = sel.idx[sel.offsets[h]:sel.offsets[h + 1]]
        top = np.sort(np.argsort(-star[h], kind="stable")[:24])
        assert np.array_equal(got, top)


def test_heads_with_larger_scores_win_budget():
    rng = np.random.default_rng(10)
    star = rng.random((2, 100)).astype(np.float32)
    star[1] *= 0.01
    sel = oracle.budget_select(star, 0.5)
    k, ns = 50, 10
    assert sel.budgets.tolist() == [2 * k - ns, ns]


def test_tiny_budget_follows_the_total_order():
    """k = 2 per head leaves no safeguard (floor(0.2*2) = 0): the 4 layer slots go to
    the first 4 pairs of the order (score desc, head asc, position asc), which are the
    pinned sinks of head 0.  With a safeguard of one slot each head keeps its first sink."""
    star = np.full((2, 40), 0.5, np.float32)
    star[:, :4] = np.inf
    sel = oracle.budget_select(star, 0.95)      # k = 2 per head
    assert sel.budgets.tolist() == [4, 0]
    assert sel.idx.tolist() == [0, 1, 2, 3]
    p = oracle.default_params()
    p.safeguard = 0.5
    sel = oracle.budget_select(star, 0.95, p)
    assert sel.budgets.tolist() == [3, 1]
    assert sel.idx.tolist() == [0, 1, 2, 0]


def test_compaction_is_a_row_gather():
    rng = np.random.default_rng(12)
    X = rng.standard_normal((3, 30, 8)).astype(np.float32)
    star = rng.random((3, 30)).astype(np.float32)
    sel = oracle.budget_select(star, 0.5)
    out = oracle.compact(X, sel.idx, sel.offsets)
    want = np.concatenate([X[h][sel.idx[sel.offsets[h]:sel.offsets[h + 1]]] for h in range(3)])
    assert out.tobytes() == want.tobytes()


def test_end_to_end_group_invariants():
    from paper_2605_26678_b200 import workloads as wl
    cfg = wl.tiny_config(kv_heads=4, head_dim=32, seq_len=520, dtype="bf16")
    K, V = wl.make_cache(cfg)
    res = oracle.compress_group(K[0], V[0], 0.75)
    k = oracle.keep_per_head(520, 0.75)
    assert res.sel.budgets.sum() == 4 * k
    assert res.k_out.shape == (4 * k, 32) and res.v_out.shape == (4 * k, 32)
    Kraw = K[0].view(__import__("torch").int16).numpy().view(np.uint16)
    for h in range(4):
        rows = res.sel.idx[res.sel.offsets[h]:res.sel.offsets[h + 1]]
        assert np.array_equal(res.k_out[res.sel.offsets[h]:res.sel.offsets[h + 1]], Kraw[h][rows])
