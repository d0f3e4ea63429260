"""ctypes front end of the CPU oracle (``nkv_oracle.c``) -- TEST INFRASTRUCTURE ONLY.

Only tests, the smoke check and the bench's CPU-baseline legs may import this
package; the product path never does.  It shares nothing with the CUDA library.
The C file is compiled with gcc on first use (or by ``build_oracle()``).
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from dataclasses import dataclass
from typing import List, Optional, Sequence

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "nkv_oracle.c")
_LIB = os.path.join(_HERE, "libnkv_oracle.so")

BF16, F32, F16 = 0, 1, 2
GATE_SURPRISE, GATE_AVERAGE, GATE_MAX = 0, 1, 2


class Params(ctypes.Structure):
    _fields_ = [
        ("window", ctypes.c_int32),
        ("n_sink", ctypes.c_int32),
        ("block_div", ctypes.c_int32),
        ("block_min", ctypes.c_int32),
        ("block_max", ctypes.c_int32),
        ("gate_mode", ctypes.c_int32),
        ("top_frac", ctypes.c_double),
        ("prior", ctypes.c_double * 3),
        ("beta", ctypes.c_double),
        ("tau", ctypes.c_double),
        ("kappa", ctypes.c_double),
        ("safeguard", ctypes.c_double),
    ]


def build_oracle(force: bool = False) -> str:
    """Compile the oracle with gcc (no-op when the library is newer than the source)."""
    if (not force and os.path.exists(_LIB)
            and os.path.getmtime(_LIB) >= os.path.getmtime(_SRC)):
        return _LIB
    tmp = _LIB + ".tmp.%d" % os.getpid()
    subprocess.check_call(["gcc", "-O2", "-std=c99", "-fPIC", "-shared", "-o", tmp, _SRC, "-lm"])
    os.replace(tmp, _LIB)
    return _LIB


_lib = None


def lib():
    global _lib
    if _lib is None:
        L = ctypes.CDLL(build_oracle())
        i64, dbl, vp = ctypes.c_int64, ctypes.c_double, ctypes.c_void_p
        pp = ctypes.POINTER(Params)
        L.nkvo_default_params.argtypes = [pp]
        L.nkvo_default_params.restype = None
        for name in ("nkvo_block_size", "nkvo_num_blocks", "nkvo_top_count"):
            getattr(L, name).argtypes = [i64, pp]
            getattr(L, name).restype = i64
        L.nkvo_keep_per_head.argtypes = [i64, dbl]
        L.nkvo_keep_per_head.restype = i64
        L.nkvo_safeguard_count.argtypes = [i64, dbl, pp]
        L.nkvo_safeguard_count.restype = i64
        L.nkvo_score_head.argtypes = [vp, ctypes.c_int, i64, i64, i64, pp, vp, vp, vp, vp, vp, vp, vp]
        L.nkvo_score_head.restype = ctypes.c_int
        L.nkvo_budget_select.argtypes = [vp, i64, i64, dbl, pp, vp, vp, vp, vp]
        L.nkvo_budget_select.restype = ctypes.c_int
        L.nkvo_compact.argtypes = [vp, i64, i64, i64, i64, i64, vp, vp, vp]
        L.nkvo_compact.restype = ctypes.c_int
        _lib = L
    return _lib


def default_params() -> Params:
    p = Params()
    lib().nkvo_default_params(ctypes.byref(p))
    return p


def block_size(N: int, p: Optional[Params] = None) -> int:
    p = p or default_params()
    return int(lib().nkvo_block_size(N, ctypes.byref(p)))


def num_blocks(N: int, p: Optional[Params] = None) -> int:
    p = p or default_params()
    return int(lib().nkvo_num_blocks(N, ctypes.byref(p)))


def keep_per_head(N: int, r: float) -> int:
    return int(lib().nkvo_keep_per_head(N, float(r)))


def safeguard_count(N: int, r: float, p: Optional[Params] = None) -> int:
    p = p or default_params()
    return int(lib().nkvo_safeguard_count(N, float(r), ctypes.byref(p)))


def top_count(N: int, p: Optional[Params] = None) -> int:
    p = p or default_params()
    return int(lib().nkvo_top_count(N, ctypes.byref(p)))


def _ptr(a: Optional[np.ndarray]):
    return None if a is None else a.ctypes.data_as(ctypes.c_void_p)


def _as_bytes_2d(x) -> (np.ndarray, int):
    """[N, d] array of bf16 / fp16 (torch), fp16 / fp32 (numpy) -> (contiguous numpy view, dtype code)."""
    try:
        import torch
    except Exception:  # pragma: no cover
        torch = None
    if torch is not None and isinstance(x, torch.Tensor):
        x = x.detach().cpu().contiguous()
        if x.dtype == torch.bfloat16:
            return x.view(torch.int16).numpy().view(np.uint16), BF16
        if x.dtype == torch.float32:
            return x.numpy(), F32
        if x.dtype == torch.float16:
            return x.view(torch.int16).numpy().view(np.uint16), F16
        raise TypeError("oracle accepts bf16, fp16 or fp32 keys, got %s" % x.dtype)
    x = np.ascontiguousarray(x)
    if x.dtype == np.float32:
        return x, F32
    if x.dtype == np.uint16:
        return x, BF16
    if x.dtype == np.float16:
        return x.view(np.uint16), F16
    raise TypeError("oracle accepts float32, float16 or raw-bf16 (uint16) arrays, got %s" % x.dtype)


@dataclass
class HeadScore:
    inv_norm: np.ndarray   # [N] f64
    mu_s: np.ndarray       # [d]
    mu_e: np.ndarray       # [nb, d]
    mu_c: Optional[np.ndarray]  # [N, d] or None
    a_raw: np.ndarray      # [3, N] f64
    lo: np.ndarray         # [3]
    hi: np.ndarray         # [3]
    delta: np.ndarray      # [3]
    w: np.ndarray          # [3]
    s_min: float
    s_max: float
    s_mean: float          # mean of the min-max-normalised surprise
    m: int
    a_star: np.ndarray     # [N] f32, sinks = +inf


def score_head(K, params: Optional[Params] = None, want_mu_c: bool = False) -> HeadScore:
    """Sections 2.1-2.4 for one head: K is [N, d] (bf16 or fp32)."""
    p = params or default_params()
    k2, code = _as_bytes_2d(K)
    N, d = k2.shape
    nb = num_blocks(N, p)
    inv = np.empty(N, np.float64)
    mu_s = np.empty(d, np.float64)
    mu_e = np.empty((nb, d), np.float64)
    mu_c = np.empty((N, d), np.float64) if want_mu_c else None
    a_raw = np.empty((3, N), np.float64)
    stats = np.empty(16, np.float64)
    a_star = np.empty(N, np.float32)
    rc = lib().nkvo_score_head(_ptr(k2), code, N, d, d, ctypes.byref(p), _ptr(inv), _ptr(mu_s),
                               _ptr(mu_e), _ptr(mu_c), _ptr(a_raw), _ptr(stats), _ptr(a_star))
    if rc != 0:
        raise RuntimeError("nkvo_score_head failed (%d)" % rc)
    return HeadScore(inv, mu_s, mu_e, mu_c, a_raw, stats[0:3].copy(), stats[3:6].copy(),
                     stats[6:9].copy(), stats[9:12].copy(), float(stats[12]), float(stats[13]),
                     float(stats[14]), int(stats[15]), a_star)


@dataclass
class GroupSelection:
    budgets: np.ndarray    # [H] i32
    idx: np.ndarray        # [H*k] i32
    offsets: np.ndarray    # [H+1] i32
    ranks: Optional[np.ndarray]  # [H, N] i32


def budget_select(a_star: np.ndarray, r: float, params: Optional[Params] = None,
                  want_ranks: bool = False) -> GroupSelection:
    """Sections 2.5-2.6 for one layer group: a_star is [H, N] fp32."""
    p = params or default_params()
    a = np.ascontiguousarray(a_star, dtype=np.float32)
    H, N = a.shape
    k = keep_per_head(N, r)
    if k < 1:
        raise ValueError("r leaves no token: k=%d" % k)
    budgets = np.empty(H, np.int32)
    idx = np.empty(H * k, np.int32)
    offsets = np.empty(H + 1, np.int32)
    ranks = np.empty((H, N), np.int32) if want_ranks else None
    rc = lib().nkvo_budget_select(_ptr(a), H, N, float(r), ctypes.byref(p), _ptr(budgets), _ptr(idx),
                                  _ptr(offsets), _ptr(ranks))
    if rc != 0:
        raise RuntimeError("nkvo_budget_select failed (%d)" % rc)
    return GroupSelection(budgets, idx, offsets, ranks)


def compact(X, idx: np.ndarray, offsets: np.ndarray) -> np.ndarray:
    """Gather rows of X [H, N, d] (bf16/fp32) -> [sum B_h, d] raw (uint16 or float32)."""
    H, N = X.shape[0], X.shape[1]
    rows: List[np.ndarray] = []
    code = None
    for h in range(H):
        r2, code = _as_bytes_2d(X[h])
        rows.append(r2)
    src = np.ascontiguousarray(np.stack(rows, 0))
    d = src.shape[2]
    row_bytes = d * src.itemsize
    dst = np.empty((int(offsets[H]), d), src.dtype)
    rc = lib().nkvo_compact(_ptr(src), H, N, row_bytes, N * row_bytes, row_bytes,
                            _ptr(np.ascontiguousarray(idx, np.int32)),
                            _ptr(np.ascontiguousarray(offsets, np.int32)), _ptr(dst))
    if rc != 0:
        raise RuntimeError("nkvo_compact failed (%d)" % rc)
    return dst


@dataclass
class GroupResult:
    heads: List[HeadScore]
    a_star: np.ndarray     # [H, N] f32
    sel: GroupSelection
    k_out: Optional[np.ndarray]
    v_out: Optional[np.ndarray]


def compress_group(K, V, r: float, params: Optional[Params] = None, want_ranks: bool = False,
                   want_mu_c: bool = False) -> GroupResult:
    """The whole path for one layer group: K, V are [H, N, d] (V may be None)."""
    p = params or default_params()
    H = K.shape[0]
    heads = [score_head(K[h], p, want_mu_c=want_mu_c) for h in range(H)]
    a_star = np.stack([hs.a_star for hs in heads], 0)
    sel = budget_select(a_star, r, p, want_ranks=want_ranks)
    k_out = compact(K, sel.idx, sel.offsets)
    v_out = compact(V, sel.idx, sel.offsets) if V is not None else None
    return GroupResult(heads, a_star, sel, k_out, v_out)
