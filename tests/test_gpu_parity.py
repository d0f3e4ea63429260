"""GPU parity: every stage of the CUDA path against the CPU oracle, through the C ABI.

Stage tests feed each GPU stage the oracle's output of the previous one ("teacher forcing"),
so integer stages are compared bit for bit.  End-to-end tests run the fused call and account
for near-tie swaps.  All inputs come from the seeded generator; the oracle reads the bytes the
GPU read.
"""
import math

import numpy as np
import pytest
import torch

import oracle
from paper_2605_26678_b200 import nkv
from paper_2605_26678_b200 import workloads as wl
from tests import parity as pr

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def _cache(N, d, dtype, H=2, layers=1, seed=11, seg=(32, 96)):
    cfg = wl.tiny_config(kv_heads=H, head_dim=d, seq_len=N, dtype=dtype, layers=layers, base_seed=seed,
                         seg_lo=seg[0], seg_hi=seg[1])
    K, V = wl.make_cache(cfg)
    return K.to(DEV), V.to(DEV)


SHAPES = [(1, 64, "fp32"), (3, 64, "bf16"), (63, 128, "bf16"), (64, 64, "fp32"), (65, 128, "fp32"),
          (200, 64, "bf16"), (257, 128, "bf16"), (1000, 128, "fp32"), (4133, 64, "bf16"), (6000, 128, "bf16"),
          (300, 64, "fp16"), (4133, 128, "fp16")]


@pytest.mark.parametrize("N,d,dtype", SHAPES)
def test_anchors_match_oracle(N, d, dtype):
    K, _ = _cache(N, d, dtype)
    mu_s, mu_e, inv_norm, mu_c = nkv.nkv_anchors(K, want_mu_c=(N <= 1000))
    torch.cuda.synchronize()
    for g in range(K.shape[0]):
        for h in range(K.shape[1]):
            ref = oracle.score_head(K[g, h].cpu(), want_mu_c=(N <= 1000))
            pr.assert_close(inv_norm[g, h].cpu().numpy(), ref.inv_norm, "inv_norm", 1e-5)
            pr.assert_close(mu_s[g, h].cpu().numpy(), ref.mu_s, "mu_s", 1e-5)
            pr.assert_close(mu_e[g, h].cpu().numpy(), ref.mu_e, "mu_e", 1e-5)
            if mu_c is not None:
                pr.assert_close(mu_c[g, h].cpu().numpy(), ref.mu_c, "mu_c", 1e-5)


@pytest.mark.parametrize("N,d,dtype", SHAPES)
def test_scores_match_oracle(N, d, dtype):
    K, _ = _cache(N, d, dtype)
    mu_s, mu_e, inv_norm, _ = nkv.nkv_anchors(K)
    a_star, a_raw, stats = nkv.nkv_score(K, mu_s, mu_e, inv_norm, want_raw=True, want_stats=True)
    torch.cuda.synchronize()
    for h in range(K.shape[1]):
        ref = oracle.score_head(K[0, h].cpu())
        pr.assert_close(a_raw[0, h].cpu().numpy(), ref.a_raw, "a_raw")
        st = stats[0, h].cpu().numpy()
        if N >= 8:   # with a handful of tokens the min-max range can be rounding noise in both precisions
            pr.assert_close(st[0:3], ref.lo, "lo")
            pr.assert_close(st[3:6], ref.hi, "hi")
            pr.assert_close(st[6:9], ref.delta, "delta")
            pr.assert_close(st[9:12], ref.w, "w")
            pr.assert_close(st[12:15], [ref.s_min, ref.s_max, ref.s_mean], "surprise stats")
            pr.assert_close(a_star[0, h].cpu().numpy(), ref.a_star, "a_star")
        assert st[15] == ref.m
        assert torch.isinf(a_star[0, h, :min(4, N)]).all()


KEY_SCAN_CASES = [("fma", 1, 64, "fp32"), ("fma", 63, 128, "bf16"), ("fma", 257, 128, "bf16"), ("fma", 1000, 128, "fp32"),
                  ("fma", 4133, 64, "bf16"), ("fma", 6000, 128, "bf16"), ("tensor", 100, 128, "bf16"),
                  ("tensor", 257, 128, "bf16"), ("tensor", 2500, 128, "bf16"), ("tensor", 4352, 128, "bf16"),
                  ("tensor", 8200, 128, "bf16"), ("tensor", 4133, 64, "bf16"), ("auto", 3000, 128, "bf16"),
                  ("auto", 2500, 128, "fp16"), ("tensor", 777, 64, "fp16")]


@pytest.mark.parametrize("mode,N,d,dtype", KEY_SCAN_CASES)
def test_key_scan_intermediates_match_oracle(mode, N, d, dtype):
    """The kernels nkv_compress times, stage by stage: 1/||k||, the anchors, the three raw anomalies and their
    per-head extremes straight out of the key scan, for the FMA and the tensor-core form."""
    K, _ = _cache(N, d, dtype, H=3)
    p = nkv.nkv_default_params()
    ws = nkv.alloc_workspace(K, p)
    nkv.nkv_set_key_passes(mode)
    try:
        inv_norm, mu_s, mu_e, a_raw, minmax = nkv.nkv_key_scan(K, p, ws=ws)
    finally:
        nkv.nkv_set_key_passes("auto")
    assert nkv.nkv_last_device_status(ws) == nkv.NKV_OK
    for h in range(K.shape[1]):
        ref = oracle.score_head(K[0, h].cpu())
        pr.assert_close(inv_norm[0, h].cpu().numpy(), ref.inv_norm, "inv_norm", 1e-5)
        pr.assert_close(mu_s[0, h].cpu().numpy(), ref.mu_s, "mu_s", 1e-5)
        pr.assert_close(mu_e[0, h].cpu().numpy(), ref.mu_e, "mu_e", 1e-5)
        pr.assert_close(a_raw[0, h].cpu().numpy(), ref.a_raw, "a_raw", 1e-5)
        mm = minmax[0, h].cpu().numpy()
        pr.assert_close(mm[0::2], ref.lo, "lo", 1e-5)
        pr.assert_close(mm[1::2], ref.hi, "hi", 1e-5)


@pytest.mark.parametrize("prior,gate", [((1.0, 0.0, 0.0), nkv.NKV_GATE_AVERAGE), ((0.5, 0.5, 0.0), nkv.NKV_GATE_AVERAGE),
                                        ((0.5, 0.5, 0.0), nkv.NKV_GATE_SURPRISE), ((0.0, 0.0, 1.0), nkv.NKV_GATE_MAX)])
def test_ablation_priors_switch_scales_off(prior, gate):
    """Single-anchor scoring (the "w/o continuum" row of the ablation table) and scoring without the current
    memory (the components table): a prior of zero removes a scale from the blend."""
    K, V = _cache(1500, 128, "bf16", H=2)
    p = nkv.nkv_default_params()
    p.gate_mode = gate
    for k in range(3):
        p.prior[k] = prior[k]
    res = nkv.nkv_compress(K, V, 0.75, p, want_a_star=True)
    torch.cuda.synchronize()
    for h in range(K.shape[1]):
        ref = oracle.score_head(K[0, h].cpu(), pr.oracle_params(p))
        assert [w == 0.0 for w in ref.w] == [x == 0.0 for x in prior]
        pr.assert_close(res.a_star[0, h].cpu().numpy(), ref.a_star, "a_star")
    if prior == (1.0, 0.0, 0.0):   # key distinctiveness: min-max of -cos(k_hat, mean k_hat)
        a = res.a_star[0, 0, 4:].cpu().numpy()
        ref = oracle.score_head(K[0, 0].cpu())
        want = (ref.a_raw[0] - ref.lo[0]) / (ref.hi[0] - ref.lo[0])
        pr.assert_close(a, want[4:], "single-anchor score")


@pytest.mark.parametrize("gate,window,n_sink,prior", [
    (nkv.NKV_GATE_AVERAGE, 64, 4, (0.4, 0.4, 0.2)), (nkv.NKV_GATE_MAX, 64, 0, (0.4, 0.4, 0.2)),
    (nkv.NKV_GATE_SURPRISE, 2, 4, (0.2, 0.3, 0.5)), (nkv.NKV_GATE_SURPRISE, 17, 8, (0.4, 0.4, 0.2)),
    (nkv.NKV_GATE_SURPRISE, 40, 16, (0.6, 0.3, 0.1))])
def test_score_parameter_switches(gate, window, n_sink, prior):
    K, _ = _cache(777, 128, "bf16")
    p = nkv.nkv_default_params()
    p.gate_mode, p.window, p.n_sink = gate, window, n_sink
    p.block_div, p.block_min, p.block_max = 64, 64, 128
    p.beta, p.tau, p.kappa = 2.0, 0.3, 6.0
    for k in range(3):
        p.prior[k] = prior[k]
    mu_s, mu_e, inv_norm, _ = nkv.nkv_anchors(K, p)
    a_star, a_raw, _ = nkv.nkv_score(K, mu_s, mu_e, inv_norm, p, want_raw=True)
    torch.cuda.synchronize()
    for h in range(K.shape[1]):
        ref = oracle.score_head(K[0, h].cpu(), pr.oracle_params(p))
        pr.assert_close(a_raw[0, h].cpu().numpy(), ref.a_raw, "a_raw")
        pr.assert_close(a_star[0, h].cpu().numpy(), ref.a_star, "a_star")


def _random_scores(G, H, N, seed, ties):
    rng = np.random.default_rng(seed)
    s = rng.random((G, H, N)).astype(np.float32) ** 3
    s *= rng.uniform(0.05, 1.0, size=(G, H, 1)).astype(np.float32)
    if ties == "many":
        s = np.round(s * 16) / 16
    elif ties == "all":
        s[:] = 0.25
    elif ties == "dense":          # bulk packed into a sliver of [0,1], like real scores
        s = (0.05 + 0.001 * s).astype(np.float32)
    s[:, :, :4] = np.inf
    return s


@pytest.mark.parametrize("G,H,N,r,ties", [
    (1, 1, 10, 0.5, "none"), (2, 3, 100, 0.75, "none"), (1, 8, 1000, 0.75, "many"), (2, 4, 5000, 0.95, "dense"),
    (1, 8, 3000, 0.5, "all"), (1, 2, 4097, 0.0, "none"), (3, 8, 2048, 0.9, "dense"), (1, 5, 40, 0.95, "none"),
    # large enough for the parallel form of the group competition; "dense" and "all" overflow its candidate list
    (2, 8, 20000, 0.75, "none"), (2, 8, 12000, 0.5, "many"), (1, 8, 16384, 0.95, "dense"), (1, 8, 9000, 0.5, "all"),
    (3, 5, 14001, 0.9, "none")])
def test_budget_and_select_bit_exact_on_oracle_scores(G, H, N, r, ties):
    s = _random_scores(G, H, N, seed=N + H, ties=ties)
    a_star = torch.from_numpy(s).to(DEV)
    budgets = nkv.nkv_budget(a_star, r)
    k = nkv.nkv_keep_per_head(N, r)
    idx, offs, ranks = nkv.nkv_select(a_star, budgets, H * k, want_ranks=(N <= 5000))
    torch.cuda.synchronize()
    for g in range(G):
        ref = oracle.budget_select(s[g], r, want_ranks=True)
        assert np.array_equal(budgets[g].cpu().numpy(), ref.budgets)
        assert np.array_equal(offs[g].cpu().numpy(), ref.offsets)
        assert np.array_equal(idx[g].cpu().numpy(), ref.idx)
        if ranks is not None:
            assert np.array_equal(ranks[g].cpu().numpy(), ref.ranks)


def test_safeguard_one_gives_uniform_budgets():
    s = _random_scores(2, 4, 600, seed=3, ties="none")
    p = nkv.nkv_default_params()
    p.safeguard = 1.0
    budgets = nkv.nkv_budget(torch.from_numpy(s).to(DEV), 0.75, p)
    assert budgets.cpu().tolist() == [[150] * 4] * 2


@pytest.mark.parametrize("d,dv,dtype,mode", [(128, 128, "bf16", "out"), (64, 64, "fp32", "out"),
                                             (128, 128, "fp32", "in"), (64, 64, "bf16", "in"),
                                             (128, 64, "bf16", "out"), (64, 128, "fp32", "out"),
                                             (128, 64, "bf16", "in"), (128, 128, "fp16", "out")])
def test_compaction_copies_rows_verbatim(d, dv, dtype, mode):
    K, V = _cache(900, d, dtype, H=3, layers=2)
    if dv != d:   # values of another width (the paper's V in R^{N x d_v}): same rows, other row length
        V = _cache(900, dv, dtype, H=3, layers=2, seed=12)[1]
    s = _random_scores(2, 3, 900, seed=5, ties="none")
    sel = [oracle.budget_select(s[g], 0.6) for g in range(2)]
    idx = torch.from_numpy(np.stack([x.idx for x in sel])).to(DEV)
    offs = torch.from_numpy(np.stack([x.offsets for x in sel])).to(DEV)
    Kr, Vr = pr.raw_rows(K), pr.raw_rows(V)
    if mode == "out":
        K_out, V_out = nkv.nkv_compact(K, V, idx, offs)
        torch.cuda.synchronize()
        for g in range(2):
            assert np.array_equal(pr.raw_rows(K_out[g]), oracle.compact(K[g].cpu(), sel[g].idx, sel[g].offsets))
            assert np.array_equal(pr.raw_rows(V_out[g]), oracle.compact(V[g].cpu(), sel[g].idx, sel[g].offsets))
    else:
        Kc, Vc = K.clone(), V.clone()
        nkv.nkv_compact(Kc, Vc, idx, offs, mode=nkv.NKV_IN_PLACE)
        torch.cuda.synchronize()
        Kg, Vg = pr.raw_rows(Kc), pr.raw_rows(Vc)
        for g in range(2):
            for h in range(3):
                rows = sel[g].idx[sel[g].offsets[h]:sel[g].offsets[h + 1]]
                assert np.array_equal(Kg[g, h, :len(rows)], Kr[g, h][rows])
                assert np.array_equal(Vg[g, h, :len(rows)], Vr[g, h][rows])


@pytest.mark.parametrize("N,d,dtype,H,layers,r", [
    (5, 64, "fp32", 2, 1, 0.5), (300, 64, "bf16", 4, 2, 0.75), (1000, 128, "fp32", 8, 1, 0.5),
    (2500, 128, "bf16", 8, 2, 0.95), (4133, 64, "bf16", 3, 1, 0.0), (777, 128, "bf16", 1, 3, 0.9),
    (3000, 128, "fp16", 4, 2, 0.85), (900, 64, "fp16", 2, 1, 0.25)])
def test_fused_compress_end_to_end(N, d, dtype, H, layers, r):
    K, V = _cache(N, d, dtype, H=H, layers=layers)
    p = nkv.nkv_default_params()
    ws = nkv.alloc_workspace(K, p)
    res = nkv.nkv_compress(K, V, r, p, ws=ws, want_a_star=True)
    assert nkv.nkv_last_device_status(ws) == nkv.NKV_OK
    rep = pr.SwapReport()
    for g in range(K.shape[0]):
        pr.check_group_against_oracle(K, V, res, g, r, p, rep)
    assert rep.swapped_tokens <= max(2, rep.heads)   # near-tie swaps are rare at fp32 accuracy


@pytest.mark.parametrize("N,H,layers,r", [
    (100, 2, 1, 0.5), (777, 1, 3, 0.9), (2500, 8, 2, 0.95), (4096, 4, 1, 0.75), (8200, 3, 1, 0.75),
    (4352, 2, 1, 0.75), (6144, 2, 1, 0.5)])   # the last two: blocks of 136 and 192 keys straddle the 128-key tiles
@pytest.mark.parametrize("mode,d", [("tensor", 128), ("fma", 128), ("tensor", 64)])
def test_key_pass_kernels_end_to_end(N, H, layers, r, mode, d):
    """Both key passes on the tensor cores (tcgen05: band sums of the keys' Gram matrix, dots with the
    split anchors) and both as FMA kernels, each against the oracle.  With d = 64 only the second pass
    has a tensor-core form."""
    K, V = _cache(N, d, "bf16", H=H, layers=layers)
    p = nkv.nkv_default_params()
    ws = nkv.alloc_workspace(K, p)
    before = nkv.nkv_launch_count()
    nkv.nkv_set_key_passes(mode)
    try:
        res = nkv.nkv_compress(K, V, r, p, ws=ws, want_a_star=True)
    finally:
        nkv.nkv_set_key_passes("auto")
    assert nkv.nkv_last_device_status(ws) == nkv.NKV_OK
    assert nkv.nkv_launch_count() > before
    rep = pr.SwapReport()
    for g in range(K.shape[0]):
        pr.check_group_against_oracle(K, V, res, g, r, p, rep)
    assert rep.swapped_tokens <= max(2, rep.heads)


@pytest.mark.parametrize("N,d,dtype,H,layers,r", [(600, 128, "bf16", 2, 9, 0.75), (333, 64, "fp32", 3, 10, 0.5)])
def test_many_groups_and_repeated_calls(N, d, dtype, H, layers, r):
    """Nine and ten layer groups in one call: every group matches the oracle, and two calls in a row on
    the same buffers and workspace give identical outputs (nothing is left over from the first)."""
    K, V = _cache(N, d, dtype, H=H, layers=layers)
    p = nkv.nkv_default_params()
    ws = nkv.alloc_workspace(K, p)
    res = nkv.nkv_compress(K, V, r, p, ws=ws, want_a_star=True)
    torch.cuda.synchronize()
    assert nkv.nkv_last_device_status(ws) == nkv.NKV_OK
    first = (res.idx.clone(), res.k_out.clone(), res.v_out.clone(), res.budgets.clone())
    rep = pr.SwapReport()
    for g in range(K.shape[0]):
        pr.check_group_against_oracle(K, V, res, g, r, p, rep)
    assert rep.swapped_tokens <= max(2, rep.heads)
    res = nkv.nkv_compress(K, V, r, p, out=res, ws=ws)
    torch.cuda.synchronize()
    assert all(torch.equal(a, b) for a, b in zip(first, (res.idx, res.k_out, res.v_out, res.budgets)))


def test_identical_keys_take_the_tie_path():
    """All keys equal: every score is 0 and every selection is decided by position alone."""
    K = torch.ones((1, 2, 3000, 64), dtype=torch.bfloat16, device=DEV)
    V = torch.randn((1, 2, 3000, 64), device=DEV).to(torch.bfloat16)
    ws = nkv.alloc_workspace(K)
    res = nkv.nkv_compress(K, V, 0.75, ws=ws, want_a_star=True)
    assert nkv.nkv_last_device_status(ws) == nkv.NKV_OK
    a = res.a_star.cpu().numpy()
    assert np.isinf(a[0, :, :4]).all() and (a[0, :, 4:] == 0).all()
    ref = oracle.budget_select(a[0], 0.75)
    assert np.array_equal(res.budgets[0].cpu().numpy(), ref.budgets)
    assert np.array_equal(res.idx[0].cpu().numpy(), ref.idx)


def test_strided_heads_outermost_layout():
    """A [H, G, N, d] allocation viewed as [G, H, N, d]: strides, not copies."""
    K, V = _cache(600, 128, "bf16", H=3, layers=2)
    Kt = K.permute(1, 0, 2, 3).contiguous().permute(1, 0, 2, 3)
    Vt = V.permute(1, 0, 2, 3).contiguous().permute(1, 0, 2, 3)
    assert not Kt.is_contiguous()
    a = nkv.nkv_compress(K, V, 0.75, want_a_star=True)
    b = nkv.nkv_compress(Kt, Vt, 0.75, want_a_star=True)
    torch.cuda.synchronize()
    assert torch.equal(a.idx, b.idx) and torch.equal(a.k_out, b.k_out) and torch.equal(a.v_out, b.v_out)
    assert torch.equal(a.a_star, b.a_star)


def test_argument_errors_are_reported_not_thrown():
    K, V = _cache(100, 64, "fp32")
    with pytest.raises(nkv.NkvError) as e:
        nkv.nkv_compress(K, V, 1.0)
    assert e.value.status == nkv.NKV_ERR_INVALID_ARG
    with pytest.raises(nkv.NkvError) as e:
        nkv.nkv_compress(K, V, 0.999)      # k = 0
    assert e.value.status == nkv.NKV_ERR_INVALID_ARG
    with pytest.raises(nkv.NkvError) as e:
        nkv.nkv_compress(K[..., :48].contiguous(), V[..., :48].contiguous(), 0.5)
    assert e.value.status == nkv.NKV_ERR_UNSUPPORTED
    for bad_window in (65, 1, 0):
        p = nkv.nkv_default_params()
        p.window = bad_window
        with pytest.raises(nkv.NkvError) as e:
            nkv.nkv_compress(K, V, 0.5, p)
        assert e.value.status == nkv.NKV_ERR_UNSUPPORTED
    p = nkv.nkv_default_params()
    p.prior[0] = p.prior[1] = p.prior[2] = 0.0
    with pytest.raises(nkv.NkvError) as e:
        nkv.nkv_compress(K, V, 0.5, p)
    assert e.value.status == nkv.NKV_ERR_INVALID_ARG
    with pytest.raises(nkv.NkvError) as e:
        nkv.nkv_compress(K, V, 0.5, ws=torch.empty(1024, dtype=torch.uint8, device=DEV))
    assert e.value.status == nkv.NKV_ERR_WORKSPACE
    with pytest.raises(nkv.NkvError) as e:
        nkv.nkv_compress(K.double(), V.double(), 0.5)
    assert e.value.status == nkv.NKV_ERR_UNSUPPORTED


def test_host_buffer_entry_point_matches_device_entry_point():
    K, V = _cache(1500, 128, "bf16", H=4, layers=5)
    dev = nkv.nkv_compress(K, V, 0.75)
    torch.cuda.synchronize()
    Kh, Vh = K.cpu().pin_memory(), V.cpu().pin_memory()
    G, H, N, d = K.shape
    k = nkv.nkv_keep_per_head(N, 0.75)
    out = nkv.Compressed(torch.empty((G, H * k, d), dtype=K.dtype).pin_memory(),
                         torch.empty((G, H * k, d), dtype=K.dtype).pin_memory(),
                         torch.empty((G, H * k), dtype=torch.int32).pin_memory(),
                         torch.empty((G, H + 1), dtype=torch.int32).pin_memory(),
                         torch.empty((G, H), dtype=torch.int32).pin_memory(), None)
    nbytes = nkv.nkv_host_staging_bytes(H, N, d, nkv.NKV_BF16, 0.75, 2)
    staging = torch.empty(nbytes, dtype=torch.uint8, device=DEV)
    nkv.nkv_compress_host(Kh, Vh, 0.75, out, staging, 2)
    assert torch.equal(out.idx, dev.idx.cpu()) and torch.equal(out.budgets, dev.budgets.cpu())
    assert torch.equal(out.head_offsets, dev.head_offsets.cpu())
    assert torch.equal(out.k_out, dev.k_out.cpu()) and torch.equal(out.v_out, dev.v_out.cpu())


def test_too_many_heads_is_an_argument_error():
    """More than 65535 heads in one call is refused before anything is launched."""
    K = torch.zeros((8200, 8, 1, 64), dtype=torch.bfloat16, device=DEV)
    before = nkv.nkv_launch_count()
    with pytest.raises(nkv.NkvError) as e:
        nkv.nkv_compress(K, K, 0.0)
    assert e.value.status == nkv.NKV_ERR_UNSUPPORTED
    assert nkv.nkv_launch_count() == before


def test_host_entry_point_reports_a_device_status_of_any_chunk():
    """A device-side status raised while any chunk runs comes back from nkv_compress_host: the status words
    of every chunk are copied out before the chunk's slot is reused.  The status is planted by the library's
    test hook, nothing on the device misbehaves."""
    K, V = _cache(600, 64, "bf16", H=2, layers=6)
    Kh, Vh = K.cpu().pin_memory(), V.cpu().pin_memory()
    G, H, N, d = K.shape
    k = nkv.nkv_keep_per_head(N, 0.5)
    out = nkv.Compressed(torch.empty((G, H * k, d), dtype=K.dtype).pin_memory(),
                         torch.empty((G, H * k, d), dtype=K.dtype).pin_memory(),
                         torch.empty((G, H * k), dtype=torch.int32).pin_memory(),
                         torch.empty((G, H + 1), dtype=torch.int32).pin_memory(),
                         torch.empty((G, H), dtype=torch.int32).pin_memory(), None)
    staging = torch.empty(nkv.nkv_host_staging_bytes(H, N, d, nkv.NKV_BF16, 0.5, 2), dtype=torch.uint8, device=DEV)
    nkv.nkv_compress_host(Kh, Vh, 0.5, out, staging, 2)           # three chunks, all fine
    for chunk, code in ((0, nkv.NKV_ERR_TIMEOUT), (1, nkv.NKV_ERR_DEVICE_CHECK), (2, nkv.NKV_ERR_TIMEOUT)):
        nkv.nkv_debug_set("inject_host_status", chunk * 16 + code)
        try:
            with pytest.raises(nkv.NkvError) as e:
                nkv.nkv_compress_host(Kh, Vh, 0.5, out, staging, 2)
            assert e.value.status == code
        finally:
            nkv.nkv_debug_set("inject_host_status", 0)
    nkv.nkv_compress_host(Kh, Vh, 0.5, out, staging, 2)           # and fine again


@pytest.mark.gpu
def test_a_wait_that_runs_out_is_reported_and_leaves_the_device_usable():
    """The hand-overs of the tensor-core key passes are bounded mbarrier waits.  The probe runs that same wait on a
    barrier nothing arrives at: it must end by itself, the status words must say NKV_ERR_TIMEOUT with the probe's
    detail code, and the next ordinary call on the same workspace must be clean."""
    cfg = wl.CONFIGS["cfg1_single_layer_fp32_4k"]
    K, V = wl.make_cache(cfg, "cuda:0")
    p = nkv.nkv_default_params()
    ws = nkv.alloc_workspace(K, p)
    nkv.nkv_debug_wait_probe(2000, ws)
    assert nkv.nkv_last_device_status(ws) == nkv.NKV_ERR_TIMEOUT
    words = ws[:16].view(torch.int32).cpu().tolist()
    assert words[0] == nkv.NKV_ERR_TIMEOUT and 799 in words[:4]
    with pytest.raises(nkv.NkvError):
        nkv.nkv_debug_wait_probe(0, ws)
    out = nkv.nkv_compress(K, V, 0.75, p, ws=ws)
    assert nkv.nkv_last_device_status(ws) == nkv.NKV_OK
    assert int(out.budgets.sum()) == K.shape[1] * nkv.nkv_keep_per_head(K.shape[2], 0.75)


@pytest.mark.gpu
@pytest.mark.parametrize("r", [0.5, 0.75, 0.95])
def test_budget_thresholds_bracket_the_budgets(r):
    """nkv_budget's optional thresholds: per head, the tokens scoring above the threshold fit into the budget and the
    tokens scoring at least the threshold fill it (Section 2.6: the threshold is the score of the last slot taken)."""
    g = torch.Generator(device="cpu").manual_seed(11)
    G, H, N = 3, 8, 5000
    a = torch.rand((G, H, N), generator=g, dtype=torch.float32)
    a[:, :, ::7] = a[:, :, 1::7][:, :, : a[:, :, ::7].shape[2]]   # plant exact ties
    a[:, :, :4] = float("inf")
    a_dev = a.cuda()
    budgets, thr = nkv.nkv_budget(a_dev, r, want_thresholds=True)
    assert torch.equal(budgets.cpu(), nkv.nkv_budget(a_dev, r).cpu())
    above = (a_dev > thr[:, :, None]).sum(dim=2)
    at_least = (a_dev >= thr[:, :, None]).sum(dim=2)
    assert bool((above <= budgets).all()) and bool((budgets <= at_least).all())
    assert int(budgets.sum()) == G * H * nkv.nkv_keep_per_head(N, r)


@pytest.mark.gpu
@pytest.mark.parametrize("seed", [7, 23])
def test_random_shapes_end_to_end(seed):
    """Twenty seeded random calls per seed (N from 65 to 12000 with tile-aligned and ragged lengths, d, storage, heads,
    layers, ratio and key-pass form drawn at random), each compared with the oracle group by group."""
    import random
    rng = random.Random(seed)
    p = nkv.nkv_default_params()
    swaps = heads = 0
    for case in range(20):
        d = rng.choice([64, 128, 128])
        dtype = rng.choice(["bf16", "bf16", "fp16", "fp32"])
        N = rng.choice([rng.randint(65, 700), rng.randint(700, 5000), rng.randint(5000, 12000), 128 * rng.randint(1, 40),
                        256 * rng.randint(1, 20) + rng.choice([0, 1, 127])])
        H, layers = rng.randint(1, 8), rng.randint(1, 3)
        r = rng.choice([0.25, 0.5, 0.75, 0.85, 0.95])
        mode = rng.choice(["auto", "tensor", "tensor", "fma"])
        if nkv.nkv_keep_per_head(N, r) < 1:
            continue
        K, V = _cache(N, d, dtype, H=H, layers=layers, seed=100 * seed + case, seg=(32, rng.choice([96, 400, 2000])))
        ws = nkv.alloc_workspace(K, p)
        nkv.nkv_set_key_passes(mode)
        try:
            res = nkv.nkv_compress(K, V, r, p, ws=ws, want_a_star=True)
        finally:
            nkv.nkv_set_key_passes("auto")
        assert nkv.nkv_last_device_status(ws) == nkv.NKV_OK, (case, N, d, dtype, H, layers, r, mode)
        rep = pr.SwapReport()
        for g in range(K.shape[0]):
            pr.check_group_against_oracle(K, V, res, g, r, p, rep)
        swaps += rep.swapped_tokens
        heads += rep.heads
    assert swaps <= max(4, heads // 50)
