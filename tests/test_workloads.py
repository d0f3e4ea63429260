"""The synthetic cache generator: determinism, shapes and the stated structure."""
import numpy as np
import torch

from paper_2605_26678_b200 import workloads as wl


def test_five_configs_have_the_stated_shapes():
    c = wl.CONFIGS
    assert [v.keys for v in c.values()] == [32768, 2359296, 4194304, 37748736, 37748736]
    assert [v.kv_bytes() for v in c.values()] == [33554432, 1207959552, 1073741824, 19327352832, 19327352832]
    assert c["cfg4_qwen3_4b_32k_b4"].ratios == (0.50, 0.75, 0.95)
    assert c["cfg5_qwen3_8b_128k"].seg_lo == 512 and c["cfg5_qwen3_8b_128k"].seg_hi == 8192


def test_generation_is_deterministic_and_group_local():
    cfg = wl.tiny_config(layers=3, kv_heads=2, head_dim=16, seq_len=200, dtype="bf16")
    K1, V1 = wl.make_cache(cfg, groups_per_call=2)
    K2, V2 = wl.make_groups(cfg, [0, 1, 2])
    assert torch.equal(K1, K2) and torch.equal(V1, V2)
    K3, _ = wl.make_groups(cfg, [2])
    assert torch.equal(K1[2:3], K3)
    assert not torch.equal(K1[0], K1[1])
    assert K1.dtype == torch.bfloat16 and K1.shape == (3, 2, 200, 16)


def test_structure_statistics():
    cfg = wl.tiny_config(kv_heads=4, head_dim=64, seq_len=4000, dtype="fp32", seg_lo=256, seg_hi=2048)
    K, V = wl.make_cache(cfg)
    st = wl.draw_structure(cfg, [0])
    assert len(st.needles[0]) == 4 and st.needles[0].min() >= 4
    assert len(set(st.needles[0].tolist())) == 4
    seg_lens = np.bincount(st.seg_id[0])
    assert np.all(seg_lens[:-1] >= 256) and np.all(seg_lens <= 2048)
    norms = K[0, 0].norm(dim=-1)
    body = torch.ones(4000, dtype=torch.bool)
    body[:4] = False
    body[torch.from_numpy(st.needles[0])] = False
    # sinks are the same distribution scaled by 8
    assert norms[:4].mean() > 6 * norms[body].mean()
    # needle rows are N(0, 9 I): norm about 3*sqrt(d)
    assert abs(norms[torch.from_numpy(st.needles[0])].mean().item() - 3 * 8) < 4
    assert abs(V.std().item() - 1.0) < 0.01 and abs(V.mean().item()) < 0.01
    assert abs(st.mu.std() - 2.0) < 0.4 and abs(st.offsets.std() - 0.5) < 0.05
