"""Thin Python binding of the nkv C ABI (``include/nkv.h``).

Argument marshalling only: every step of the compression path runs in the CUDA
library.  PyTorch supplies device memory and the current stream.  The functions
carry the names of the C entry points; each takes torch CUDA tensors, allocates
the outputs the C call writes into, and returns them.

There is no CPU fallback.  If ``libnkv.so`` is missing or cannot be loaded the
first call raises ``NkvUnavailable``.
"""
from __future__ import annotations

import ctypes
import os
from dataclasses import dataclass
from typing import Dict, Optional, Tuple

import torch

_PKG = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_PKG, "libnkv.so")

NKV_OK = 0
NKV_ERR_INVALID_ARG, NKV_ERR_UNSUPPORTED, NKV_ERR_WORKSPACE = 1, 2, 3
NKV_ERR_CUDA, NKV_ERR_TIMEOUT, NKV_ERR_DEVICE_CHECK = 4, 5, 6
NKV_BF16, NKV_F32, NKV_F16 = 0, 1, 2
NKV_GATE_SURPRISE, NKV_GATE_AVERAGE, NKV_GATE_MAX = 0, 1, 2
NKV_OUT_OF_PLACE, NKV_IN_PLACE = 0, 1
NKV_HEAD_STATS = 16
NKV_NUM_STAGES = 6
NKV_STATIC_MAX_UNITS = 4096
STAGE_NAMES = ("anchors", "score", "head", "budget", "select", "compact")

EXPORTS = (
    "nkv_version", "nkv_status_string", "nkv_default_params", "nkv_block_size", "nkv_num_blocks",
    "nkv_keep_per_head", "nkv_safeguard_count", "nkv_top_count", "nkv_create", "nkv_destroy",
    "nkv_workspace_bytes", "nkv_anchors", "nkv_score", "nkv_budget", "nkv_select", "nkv_compact",
    "nkv_compress", "nkv_host_staging_bytes", "nkv_compress_host", "nkv_last_device_status",
    "nkv_set_timing", "nkv_get_stage_ms", "nkv_launch_count", "nkv_budget_static", "nkv_set_key_passes",
    "nkv_key_scan", "nkv_debug_set", "nkv_debug_wait_probe",
)


class NkvUnavailable(RuntimeError):
    pass


class NkvError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        super().__init__("%s failed: %s (%d)" % (where, status_string(status), status))


class Params(ctypes.Structure):
    _fields_ = [
        ("window", ctypes.c_int32), ("n_sink", ctypes.c_int32), ("block_div", ctypes.c_int32),
        ("block_min", ctypes.c_int32), ("block_max", ctypes.c_int32), ("gate_mode", ctypes.c_int32),
        ("top_frac", ctypes.c_double), ("prior", ctypes.c_double * 3), ("beta", ctypes.c_double),
        ("tau", ctypes.c_double), ("kappa", ctypes.c_double), ("safeguard", ctypes.c_double),
    ]


class Tensor(ctypes.Structure):
    _fields_ = [
        ("ptr", ctypes.c_void_p), ("dtype", ctypes.c_int32), ("reserved", ctypes.c_int32),
        ("G", ctypes.c_int64), ("H", ctypes.c_int64), ("N", ctypes.c_int64), ("d", ctypes.c_int64),
        ("stride_g", ctypes.c_int64), ("stride_h", ctypes.c_int64), ("stride_n", ctypes.c_int64),
    ]


_lib = None


def load_library():
    """dlopen the CUDA library and declare its signatures (no CUDA call is made)."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(LIB_PATH):
        raise NkvUnavailable("%s not found: build it with `python -m paper_2605_26678_b200.build` "
                             "(there is no CPU fallback)" % LIB_PATH)
    try:
        L = ctypes.CDLL(LIB_PATH)
    except OSError as e:  # pragma: no cover
        raise NkvUnavailable("cannot load %s: %s" % (LIB_PATH, e))
    vp, i32, i64, dbl, sz = ctypes.c_void_p, ctypes.c_int32, ctypes.c_int64, ctypes.c_double, ctypes.c_size_t
    pp, tp = ctypes.POINTER(Params), ctypes.POINTER(Tensor)
    L.nkv_version.restype = ctypes.c_char_p
    L.nkv_status_string.argtypes = [ctypes.c_int]
    L.nkv_status_string.restype = ctypes.c_char_p
    L.nkv_default_params.argtypes = [pp]
    for n in ("nkv_block_size", "nkv_num_blocks", "nkv_top_count"):
        getattr(L, n).argtypes = [i64, pp]
        getattr(L, n).restype = i64
    L.nkv_keep_per_head.argtypes = [i64, dbl]
    L.nkv_keep_per_head.restype = i64
    L.nkv_safeguard_count.argtypes = [i64, dbl, pp]
    L.nkv_safeguard_count.restype = i64
    L.nkv_create.argtypes = [ctypes.POINTER(vp), ctypes.c_int]
    L.nkv_destroy.argtypes = [vp]
    L.nkv_workspace_bytes.argtypes = [vp, i64, i64, i64, i64, i32, pp, ctypes.POINTER(sz)]
    L.nkv_anchors.argtypes = [vp, tp, pp, vp, vp, vp, vp, vp, sz, vp]
    L.nkv_score.argtypes = [vp, tp, vp, vp, vp, pp, vp, vp, vp, vp, sz, vp]
    L.nkv_budget.argtypes = [vp, vp, i64, i64, i64, dbl, pp, vp, vp, vp, sz, vp]
    L.nkv_select.argtypes = [vp, vp, vp, i64, i64, i64, i64, vp, vp, vp, vp, sz, vp]
    L.nkv_compact.argtypes = [vp, tp, tp, vp, vp, i64, vp, vp, i32, vp, sz, vp]
    L.nkv_compress.argtypes = [vp, tp, tp, dbl, pp, vp, vp, vp, vp, vp, vp, vp, sz, vp]
    L.nkv_host_staging_bytes.argtypes = [vp, i64, i64, i64, i32, dbl, pp, i64, ctypes.POINTER(sz)]
    L.nkv_compress_host.argtypes = [vp, tp, tp, dbl, pp, vp, vp, vp, vp, vp, i64, vp, sz]
    L.nkv_last_device_status.argtypes = [vp, vp, vp]
    L.nkv_set_timing.argtypes = [vp, ctypes.c_int]
    L.nkv_get_stage_ms.argtypes = [vp, ctypes.POINTER(ctypes.c_float)]
    L.nkv_launch_count.argtypes = [vp]
    L.nkv_launch_count.restype = i64
    L.nkv_key_scan.argtypes = [vp, tp, pp, vp, vp, vp, vp, vp, vp, sz, vp]
    L.nkv_debug_set.argtypes = [vp, ctypes.c_int, i64]
    L.nkv_debug_wait_probe.argtypes = [vp, i64, vp, sz, vp]
    L.nkv_set_key_passes.argtypes = [vp, ctypes.c_int]
    L.nkv_budget_static.argtypes = [vp, i64, i64, i64, dbl, pp, vp, vp]
    _lib = L
    return L


def status_string(status: int) -> str:
    return load_library().nkv_status_string(int(status)).decode()


def nkv_version() -> str:
    return load_library().nkv_version().decode()


def nkv_default_params() -> Params:
    p = Params()
    _check(load_library().nkv_default_params(ctypes.byref(p)), "nkv_default_params")
    return p


def nkv_block_size(N: int, params: Optional[Params] = None) -> int:
    return int(load_library().nkv_block_size(N, ctypes.byref(params or nkv_default_params())))


def nkv_num_blocks(N: int, params: Optional[Params] = None) -> int:
    return int(load_library().nkv_num_blocks(N, ctypes.byref(params or nkv_default_params())))


def nkv_keep_per_head(N: int, r: float) -> int:
    return int(load_library().nkv_keep_per_head(N, float(r)))


def nkv_safeguard_count(N: int, r: float, params: Optional[Params] = None) -> int:
    return int(load_library().nkv_safeguard_count(N, float(r), ctypes.byref(params or nkv_default_params())))


def nkv_top_count(N: int, params: Optional[Params] = None) -> int:
    return int(load_library().nkv_top_count(N, ctypes.byref(params or nkv_default_params())))


def _check(status: int, where: str) -> None:
    if status != NKV_OK:
        raise NkvError(status, where)


def _dtype_code(t: torch.Tensor) -> int:
    if t.dtype == torch.bfloat16:
        return NKV_BF16
    if t.dtype == torch.float32:
        return NKV_F32
    if t.dtype == torch.float16:
        return NKV_F16
    raise NkvError(NKV_ERR_UNSUPPORTED, "dtype %s" % t.dtype)


def _tensor(t: torch.Tensor) -> Tensor:
    if t.dim() != 4:
        raise NkvError(NKV_ERR_INVALID_ARG, "cache tensor must be [G, H, N, d]")
    if t.stride(3) != 1:
        raise NkvError(NKV_ERR_UNSUPPORTED, "d must be contiguous")
    G, H, N, d = t.shape
    return Tensor(t.data_ptr(), _dtype_code(t), 0, G, H, N, d, t.stride(0), t.stride(1), t.stride(2))


def _stream() -> int:
    return torch.cuda.current_stream().cuda_stream


def _p(t: Optional[torch.Tensor]):
    return None if t is None else ctypes.c_void_p(t.data_ptr())


class Handle:
    """An nkv_handle bound to one CUDA device."""

    def __init__(self, device: int = 0):
        if not torch.cuda.is_available():
            raise NkvUnavailable("no CUDA device: the nkv library has no CPU fallback")
        self.lib = load_library()
        self.device = int(device)
        h = ctypes.c_void_p()
        with torch.cuda.device(self.device):
            _check(self.lib.nkv_create(ctypes.byref(h), self.device), "nkv_create")
        self.h = h

    def close(self):
        if getattr(self, "h", None):
            self.lib.nkv_destroy(self.h)
            self.h = None

    def __del__(self):  # pragma: no cover
        try:
            self.close()
        except Exception:
            pass


_handles: Dict[int, Handle] = {}


def handle(device: Optional[int] = None) -> Handle:
    dev = torch.cuda.current_device() if device is None else int(device)
    if dev not in _handles:
        _handles[dev] = Handle(dev)
    return _handles[dev]


def nkv_workspace_bytes(G: int, H: int, N: int, d: int, dtype: int, params: Optional[Params] = None,
                        h: Optional[Handle] = None) -> int:
    h = h or handle()
    out = ctypes.c_size_t()
    _check(h.lib.nkv_workspace_bytes(h.h, G, H, N, d, dtype, ctypes.byref(params or nkv_default_params()),
                                     ctypes.byref(out)), "nkv_workspace_bytes")
    return int(out.value)


def alloc_workspace(K: torch.Tensor, params: Optional[Params] = None, h: Optional[Handle] = None) -> torch.Tensor:
    G, H, N, d = K.shape
    n = nkv_workspace_bytes(G, H, N, d, _dtype_code(K), params, h)
    return torch.empty(n, dtype=torch.uint8, device=K.device)


def nkv_anchors(K: torch.Tensor, params: Optional[Params] = None, want_mu_c: bool = False,
                ws: Optional[torch.Tensor] = None, h: Optional[Handle] = None):
    """-> (mu_s [G,H,d], mu_e [G,H,nb,d], inv_norm [G,H,N], mu_c [G,H,N,d] or None)"""
    h = h or handle()
    params = params or nkv_default_params()
    G, H, N, d = K.shape
    nb = nkv_num_blocks(N, params)
    f32 = dict(dtype=torch.float32, device=K.device)
    mu_s = torch.empty((G, H, d), **f32)
    mu_e = torch.empty((G, H, nb, d), **f32)
    inv_norm = torch.empty((G, H, N), **f32)
    mu_c = torch.empty((G, H, N, d), **f32) if want_mu_c else None
    ws = ws if ws is not None else alloc_workspace(K, params, h)
    kt = _tensor(K)
    _check(h.lib.nkv_anchors(h.h, ctypes.byref(kt), ctypes.byref(params), _p(mu_s), _p(mu_e), _p(inv_norm),
                             _p(mu_c), _p(ws), ws.numel(), _stream()), "nkv_anchors")
    return mu_s, mu_e, inv_norm, mu_c


def nkv_score(K: torch.Tensor, mu_s: torch.Tensor, mu_e: torch.Tensor, inv_norm: torch.Tensor,
              params: Optional[Params] = None, want_raw: bool = False, want_stats: bool = False,
              ws: Optional[torch.Tensor] = None, h: Optional[Handle] = None):
    """-> (a_star [G,H,N], a_raw [G,H,3,N] or None, head_stats [G,H,16] or None)"""
    h = h or handle()
    params = params or nkv_default_params()
    G, H, N, d = K.shape
    f32 = dict(dtype=torch.float32, device=K.device)
    a_star = torch.empty((G, H, N), **f32)
    a_raw = torch.empty((G, H, 3, N), **f32) if want_raw else None
    stats = torch.empty((G, H, NKV_HEAD_STATS), **f32) if want_stats else None
    ws = ws if ws is not None else alloc_workspace(K, params, h)
    kt = _tensor(K)
    _check(h.lib.nkv_score(h.h, ctypes.byref(kt), _p(mu_s), _p(mu_e), _p(inv_norm), ctypes.byref(params),
                           _p(a_raw), _p(a_star), _p(stats), _p(ws), ws.numel(), _stream()), "nkv_score")
    return a_star, a_raw, stats


def _small_ws(device) -> torch.Tensor:
    return torch.empty(1 << 20, dtype=torch.uint8, device=device)


def nkv_budget(a_star: torch.Tensor, r: float, params: Optional[Params] = None,
               ws: Optional[torch.Tensor] = None, h: Optional[Handle] = None, want_thresholds: bool = False):
    """a_star [G,H,N] f32 -> budgets [G,H] i32 (and, with want_thresholds, each head's selection threshold, f32 [G,H]:
    the head keeps the tokens scoring above it and as many of those scoring exactly it as the budget allows)"""
    h = h or handle()
    params = params or nkv_default_params()
    a_star = a_star.contiguous()
    G, H, N = a_star.shape
    budgets = torch.empty((G, H), dtype=torch.int32, device=a_star.device)
    # status words, thresholds and the scratch of the parallel form of the group competition
    ws = ws if ws is not None else torch.empty(8192 + 16 * G * H + G * H * 8192 + G * (256 + 5 * 8192), dtype=torch.uint8,
                                               device=a_star.device)
    thresholds = torch.empty((G, H), dtype=torch.float32, device=a_star.device) if want_thresholds else None
    _check(h.lib.nkv_budget(h.h, _p(a_star), G, H, N, float(r), ctypes.byref(params), _p(budgets), _p(thresholds), _p(ws),
                            ws.numel(), _stream()), "nkv_budget")
    return (budgets, thresholds) if want_thresholds else budgets


def nkv_budget_static(a_star: torch.Tensor, r: float, params: Optional[Params] = None,
                      out: Optional[torch.Tensor] = None) -> torch.Tensor:
    """a_star [G,H,N] f32 -> budgets [G,H] i32, for callers that cannot allocate device memory.

    The C call takes no handle and no workspace: its scratch is a fixed array inside the library
    (at most NKV_STATIC_MAX_UNITS heads per call).  Pass `out` (an int32 [G,H] CUDA tensor you
    already own) and this wrapper allocates nothing either; without `out` it creates the result
    tensor for convenience.  Calls on one device share that scratch, so keep them stream-ordered."""
    params = params or nkv_default_params()
    if not a_star.is_contiguous():
        raise NkvError(NKV_ERR_INVALID_ARG, "nkv_budget_static: a_star must be contiguous")
    G, H, N = a_star.shape
    budgets = out if out is not None else torch.empty((G, H), dtype=torch.int32, device=a_star.device)
    _check(load_library().nkv_budget_static(_p(a_star), G, H, N, float(r), ctypes.byref(params), _p(budgets),
                                            _stream()), "nkv_budget_static")
    return budgets


def nkv_select(a_star: torch.Tensor, budgets: torch.Tensor, idx_capacity: int, want_ranks: bool = False,
               ws: Optional[torch.Tensor] = None, h: Optional[Handle] = None):
    """-> (idx [G,cap] i32, head_offsets [G,H+1] i32, ranks [G,H,N] i32 or None)"""
    h = h or handle()
    a_star = a_star.contiguous()
    budgets = budgets.contiguous()
    G, H, N = a_star.shape
    i32 = dict(dtype=torch.int32, device=a_star.device)
    idx = torch.full((G, idx_capacity), -1, **i32)
    offs = torch.empty((G, H + 1), **i32)
    ranks = torch.empty((G, H, N), **i32) if want_ranks else None
    ws = ws if ws is not None else _small_ws(a_star.device)
    _check(h.lib.nkv_select(h.h, _p(a_star), _p(budgets), G, H, N, int(idx_capacity), _p(idx), _p(offs),
                            _p(ranks), _p(ws), ws.numel(), _stream()), "nkv_select")
    return idx, offs, ranks


def nkv_compact(K: torch.Tensor, V: torch.Tensor, idx: torch.Tensor, head_offsets: torch.Tensor,
                mode: int = NKV_OUT_OF_PLACE, ws: Optional[torch.Tensor] = None, h: Optional[Handle] = None):
    """Out of place: -> (K_out [G,cap,d], V_out [G,cap,d_v]).  In place: K, V are modified, returns (K, V)."""
    h = h or handle()
    G, H, N, d = K.shape
    cap = idx.shape[1]
    ws = ws if ws is not None else _small_ws(K.device)
    kt, vt = _tensor(K), _tensor(V)
    if mode == NKV_OUT_OF_PLACE:
        K_out = torch.empty((G, cap, d), dtype=K.dtype, device=K.device)
        V_out = torch.empty((G, cap, V.shape[3]), dtype=V.dtype, device=V.device)
    else:
        K_out = V_out = None
    _check(h.lib.nkv_compact(h.h, ctypes.byref(kt), ctypes.byref(vt), _p(idx), _p(head_offsets), cap, _p(K_out),
                             _p(V_out), mode, _p(ws), ws.numel(), _stream()), "nkv_compact")
    return (K_out, V_out) if mode == NKV_OUT_OF_PLACE else (K, V)


@dataclass
class Compressed:
    k_out: torch.Tensor         # [G, H*k, d]
    v_out: torch.Tensor         # [G, H*k, d]
    idx: torch.Tensor           # [G, H*k] i32
    head_offsets: torch.Tensor  # [G, H+1] i32
    budgets: torch.Tensor       # [G, H] i32
    a_star: Optional[torch.Tensor]  # [G, H, N] f32


def alloc_outputs(K: torch.Tensor, V: torch.Tensor, r: float, want_a_star: bool = False) -> Compressed:
    G, H, N, d = K.shape
    k = nkv_keep_per_head(N, r)
    if k < 1:
        raise NkvError(NKV_ERR_INVALID_ARG, "r leaves no token")
    i32 = dict(dtype=torch.int32, device=K.device)
    return Compressed(torch.empty((G, H * k, d), dtype=K.dtype, device=K.device),
                      torch.empty((G, H * k, V.shape[3]), dtype=V.dtype, device=V.device),
                      torch.empty((G, H * k), **i32), torch.empty((G, H + 1), **i32), torch.empty((G, H), **i32),
                      torch.empty((G, H, N), dtype=torch.float32, device=K.device) if want_a_star else None)


def nkv_compress(K: torch.Tensor, V: torch.Tensor, r: float, params: Optional[Params] = None,
                 out: Optional[Compressed] = None, ws: Optional[torch.Tensor] = None,
                 want_a_star: bool = False, h: Optional[Handle] = None) -> Compressed:
    """The fused path: anchors -> score -> budget -> select -> compact."""
    h = h or handle()
    params = params or nkv_default_params()
    out = out or alloc_outputs(K, V, r, want_a_star)
    ws = ws if ws is not None else alloc_workspace(K, params, h)
    kt, vt = _tensor(K), _tensor(V)
    _check(h.lib.nkv_compress(h.h, ctypes.byref(kt), ctypes.byref(vt), float(r), ctypes.byref(params),
                              _p(out.k_out), _p(out.v_out), _p(out.idx), _p(out.head_offsets), _p(out.budgets),
                              _p(out.a_star), _p(ws), ws.numel(), _stream()), "nkv_compress")
    return out


def nkv_host_staging_bytes(H: int, N: int, d: int, dtype: int, r: float, groups_per_chunk: int,
                           params: Optional[Params] = None, h: Optional[Handle] = None) -> int:
    h = h or handle()
    out = ctypes.c_size_t()
    _check(h.lib.nkv_host_staging_bytes(h.h, H, N, d, dtype, float(r), ctypes.byref(params or nkv_default_params()),
                                        int(groups_per_chunk), ctypes.byref(out)), "nkv_host_staging_bytes")
    return int(out.value)


def nkv_compress_host(K: torch.Tensor, V: torch.Tensor, r: float, out: Compressed, staging: torch.Tensor,
                      groups_per_chunk: int, params: Optional[Params] = None, h: Optional[Handle] = None) -> Compressed:
    """K, V and every tensor of `out` live in (pinned) host memory; `staging` is device scratch."""
    h = h or handle()
    params = params or nkv_default_params()
    kt, vt = _tensor(K), _tensor(V)
    _check(h.lib.nkv_compress_host(h.h, ctypes.byref(kt), ctypes.byref(vt), float(r), ctypes.byref(params),
                                   _p(out.k_out), _p(out.v_out), _p(out.idx), _p(out.head_offsets), _p(out.budgets),
                                   int(groups_per_chunk), _p(staging), staging.numel()), "nkv_compress_host")
    return out


def nkv_last_device_status(ws: torch.Tensor, h: Optional[Handle] = None) -> int:
    h = h or handle()
    return int(h.lib.nkv_last_device_status(h.h, _p(ws), _stream()))


def nkv_set_timing(enable: bool, h: Optional[Handle] = None) -> None:
    h = h or handle()
    _check(h.lib.nkv_set_timing(h.h, 1 if enable else 0), "nkv_set_timing")


def nkv_get_stage_ms(h: Optional[Handle] = None) -> Tuple[float, ...]:
    h = h or handle()
    arr = (ctypes.c_float * NKV_NUM_STAGES)()
    _check(h.lib.nkv_get_stage_ms(h.h, arr), "nkv_get_stage_ms")
    return tuple(float(x) for x in arr)


def nkv_launch_count(h: Optional[Handle] = None) -> int:
    h = h or handle()
    return int(h.lib.nkv_launch_count(h.h))


KEY_PASS = {"auto": 0, "fma": 1, "tensor": 2}


def nkv_set_key_passes(mode: str = "auto", h: Optional[Handle] = None) -> None:
    """Kernels of the two key passes: "auto", "fma" or "tensor" (bf16, d = 128 only); see nkv.h."""
    h = h or handle()
    _check(h.lib.nkv_set_key_passes(h.h, KEY_PASS[mode]), "nkv_set_key_passes")


DEBUG = {"inject_host_status": 5}


def nkv_debug_set(what: str, value: int, h: Optional[Handle] = None) -> None:
    """Test hook of the library (see nkv.h)."""
    h = h or handle()
    _check(h.lib.nkv_debug_set(h.h, DEBUG[what], int(value)), "nkv_debug_set")


def nkv_debug_wait_probe(polls: int, ws: torch.Tensor, h: Optional[Handle] = None) -> None:
    """Test hook: a bounded device-side wait that runs out (see nkv.h); read the outcome with nkv_last_device_status."""
    h = h or handle()
    _check(h.lib.nkv_debug_wait_probe(h.h, int(polls), _p(ws), ws.numel() * ws.element_size(), _stream()),
           "nkv_debug_wait_probe")


def nkv_key_scan(K: torch.Tensor, params: Optional[Params] = None, ws: Optional[torch.Tensor] = None,
                 h: Optional[Handle] = None):
    """The key scan of nkv_compress with its intermediates copied out:
    -> (inv_norm [G,H,N], mu_s [G,H,d], mu_e [G,H,nb,d], a_raw [G,H,3,N], minmax [G,H,6])"""
    h = h or handle()
    params = params or nkv_default_params()
    G, H, N, d = K.shape
    nb = nkv_num_blocks(N, params)
    f32 = dict(dtype=torch.float32, device=K.device)
    inv_norm = torch.empty((G, H, N), **f32)
    mu_s = torch.empty((G, H, d), **f32)
    mu_e = torch.empty((G, H, nb, d), **f32)
    a_raw = torch.empty((G, H, 3, N), **f32)
    minmax = torch.empty((G, H, 6), **f32)
    ws = ws if ws is not None else alloc_workspace(K, params, h)
    kt = _tensor(K)
    _check(h.lib.nkv_key_scan(h.h, ctypes.byref(kt), ctypes.byref(params), _p(inv_norm), _p(mu_s), _p(mu_e),
                              _p(a_raw), _p(minmax), _p(ws), ws.numel(), _stream()), "nkv_key_scan")
    return inv_norm, mu_s, mu_e, a_raw, minmax
