"""The C-ABI library without a GPU: it loads, exports every declared symbol, and its host-side
size functions agree with the paper's constants (no kernel is launched here)."""
import os
import re

import pytest

from paper_2605_26678_b200 import build as nkv_build
from paper_2605_26678_b200 import nkv

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
GOLDEN = os.path.join(ROOT, "tests", "golden")


@pytest.fixture(scope="module")
def lib():
    nkv_build.build_library()
    return nkv.load_library()


def _declared_symbols():
    text = open(os.path.join(ROOT, "include", "nkv.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    names = set(re.findall(r"\b(nkv_[a-z_0-9]+)\s*\(", text))
    return sorted(names)


def test_every_declared_entry_point_is_exported(lib):
    names = _declared_symbols()
    assert {"nkv_anchors", "nkv_score", "nkv_budget", "nkv_select", "nkv_compact", "nkv_compress"} <= set(names)
    for n in names:
        assert hasattr(lib, n), "%s is declared in nkv.h but not exported" % n
    assert set(nkv.EXPORTS) == set(names)


def test_defaults_and_derived_sizes(lib):
    p = nkv.nkv_default_params()
    want = {}
    for line in open(os.path.join(GOLDEN, "hyperparameters.txt")):
        if line.strip() and not line.startswith("#"):
            k, v = line.split()
            want[k] = float(v)
    assert (p.prior[0], p.prior[1], p.prior[2]) == (want["prior_s"], want["prior_e"], want["prior_c"])
    assert (p.window, p.n_sink, p.block_div, p.block_min, p.block_max) == (64, 4, 32, 128, 256)
    assert (p.beta, p.tau, p.kappa, p.safeguard, p.top_frac) == (3.0, 0.60, 10.0, 0.20, 0.10)
    for line in open(os.path.join(GOLDEN, "block_size.txt")):
        if line.strip() and not line.startswith("#"):
            N, b, nb = map(int, line.split())
            assert nkv.nkv_block_size(N) == b and nkv.nkv_num_blocks(N) == nb
    for line in open(os.path.join(GOLDEN, "budget_counts.txt")):
        if line.strip() and not line.startswith("#"):
            N, r, k, ns = line.split()
            assert nkv.nkv_keep_per_head(int(N), float(r)) == int(k)
            assert nkv.nkv_safeguard_count(int(N), float(r)) == int(ns)
    assert nkv.nkv_top_count(4096) == 409 and nkv.nkv_top_count(3) == 1
    assert nkv.nkv_keep_per_head(100, 1.0) == -1 and nkv.nkv_block_size(0) == -1
    assert nkv.status_string(0) == "ok" and "workspace" in nkv.status_string(3)


def test_no_cpu_fallback():
    import torch
    if torch.cuda.is_available():
        pytest.skip("a GPU is present")
    with pytest.raises(nkv.NkvUnavailable):
        nkv.Handle(0)
