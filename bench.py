#!/usr/bin/env python
"""Benchmark of the NestedKV compression hot path on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl reference]
                    [--workload NAME] [--ratio R]

One "step" is one fused pass (anchors -> scores -> budgets -> selection -> compaction) over
the whole synthetic KV cache of the workload, through the C ABI (nkv_compress).  The default
workload is the headline shape: Qwen3-4B-shaped cache, batch 4, 32k tokens, r = 0.75.
Rank 0 prints ONE JSON line.  With N > 1 (torchrun) every rank compresses its own cache of
the same shape (independent sequences: weak scaling, no data-path collective).

`--impl reference` times the CPU oracle (as it stands, on the host cores) on a bounded sample
of the same workload and prints the same line with "impl": "reference".
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import time
from concurrent.futures import ThreadPoolExecutor

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import torch

from paper_2605_26678_b200 import workloads as wl

METRIC = "keys_compressed_per_sec"
UNIT = "keys/s"
DEFAULT_WORKLOAD = "cfg4_qwen3_4b_32k_b4"
DEFAULT_RATIO = 0.75
# DRAM bytes per key of each kernel (dram__bytes_read.sum + dram__bytes_write.sum of one launch / keys of the
# launch) come from the ncu capture summarised in profiles/; the file lists kernel, storage, head_dim, bytes
# per key and the digest of the kernel's source file at capture time.  A kernel whose source has changed since
# reports no traffic.
TRAFFIC_FILE = os.path.join(ROOT, "profiles", "dram_bytes_per_key.txt")
STAGE_KERNEL = {"anchors": ("gram_pass_kernel", "nkv_gram.cu"), "score": ("anchor_dots_kernel", "nkv_dots.cu"),
                "compact": ("gather_kernel", "nkv_compact.cu"), "head": ("scale_stats_kernel", "nkv_select.cu"),
                "budget": ("budget_kernel", "nkv_select.cu"), "select": ("select_kernel", "nkv_select.cu")}
NOMINAL_HBM_GBS = 8000.0
FALLBACK_HBM_GBS = 6650.0


def source_digest(name):
    """Digest of a kernel's source file together with the two headers every kernel includes."""
    import hashlib
    h = hashlib.sha256()
    try:
        for f in (name, "nkv_sm100.cuh", "nkv_common.cuh"):
            with open(os.path.join(ROOT, "paper_2605_26678_b200", "csrc", f), "rb") as fh:
                h.update(fh.read())
    except OSError:
        return None
    return h.hexdigest()[:16]


def measured_traffic_per_key(kernel, source, storage, head_dim):
    """Bytes per key from the tracked ncu summary, or None if absent or taken on another version of the kernel."""
    try:
        with open(TRAFFIC_FILE) as f:
            for line in f:
                parts = line.split()
                if len(parts) >= 5 and not line.startswith("#") and parts[0] == kernel and parts[1] == storage \
                        and int(parts[2]) == head_dim:
                    return float(parts[3]) if parts[4] == source_digest(source) else None
    except OSError:
        pass
    return None


def parse_args():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=100)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="nkv", choices=["nkv", "reference"])
    ap.add_argument("--workload", default=DEFAULT_WORKLOAD, choices=sorted(wl.ALL_CONFIGS))
    ap.add_argument("--ratio", type=float, default=None)
    ap.add_argument("--e2e-steps", type=int, default=2)
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-config-table", action="store_true", help="skip the per-configuration table")
    ap.add_argument("--key-passes", default="auto", choices=["auto", "fma", "tensor"],
                    help="kernels of the two key passes (library default: auto)")
    return ap.parse_args()


def measured_peak():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(path) as f:
            return float(json.load(f)["hbm_gbs"]), "measured (MEASURED_PEAKS.json, copy bandwidth)"
    except Exception:
        return FALLBACK_HBM_GBS, "fallback (no MEASURED_PEAKS.json)"


class ClockSampler:
    """Samples nvidia-smi clocks and throttle reasons while the timed region runs."""

    FIELDS = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
              "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
              "clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.index = index
        self.proc = None

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", "-i", str(self.index), "--query-gpu=" + self.FIELDS,
                 "--format=csv,noheader,nounits", "-lms", "100"],
                stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
        except Exception:
            self.proc = None

    def stop(self):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        time.sleep(0.15)
        self.proc.terminate()
        try:
            out, _ = self.proc.communicate(timeout=5)
        except Exception:
            self.proc.kill()
            out = ""
        sm, mx, power, reasons = [], [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for line in out.strip().splitlines():
            parts = [p.strip() for p in line.split(",")]
            if len(parts) < 7:
                continue
            try:
                sm.append(float(parts[0]))
                mx.append(float(parts[1]))
                power.append(float(parts[2]))
            except ValueError:
                continue
            for name, val in zip(names, parts[3:7]):
                if val.lower().startswith("active"):
                    reasons.add(name)
        return {"sm_mhz": statistics.median(sm) if sm else None,
                "sm_max_mhz": max(mx) if mx else None,
                "power_w_max": max(power) if power else None,
                "samples": len(sm), "reasons": sorted(reasons)}


def physical_gpu_index(local: int) -> int:
    vis = os.environ.get("CUDA_VISIBLE_DEVICES")
    if vis:
        try:
            return int(vis.split(",")[local])
        except Exception:
            return local
    return local


def replica_config(cfg, rank):
    """The cache a rank owns: same shape on every rank, different sequences (independent replicas)."""
    if rank == 0:
        return cfg
    return wl.CacheConfig(**{**cfg.__dict__, "base_seed": cfg.base_seed + 977 * rank})


def whole_job_throughput(ms_local, steps, keys_per_rank, world, dist=None, device="cpu"):
    """(keys/s over all ranks, ms per step): the slowest rank's time bounds the job."""
    t = torch.tensor([ms_local], dtype=torch.float64, device=device)
    if dist is not None and world > 1:
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
    ms_per_step = float(t.item()) / steps
    return keys_per_rank * world / (ms_per_step * 1e-3), ms_per_step


def bench_config(cfg, r, key_passes):
    """The `config` object of the JSON line (the same for both arms)."""
    return {"workload": "%s r=%.2f" % (cfg.name, r), "groups": cfg.groups, "kv_heads": cfg.kv_heads,
            "seq_len": cfg.seq_len, "head_dim": cfg.head_dim, "storage": cfg.dtype,
            "keys_per_step_per_gpu": cfg.keys, "kv_bytes_per_gpu": cfg.kv_bytes(),
            "l2": "inputs (%.1f GB) are far larger than the 126 MB L2; no flush needed" % (
                cfg.kv_bytes() / 1e9) if cfg.kv_bytes() > 1e9 else "inputs fit L2: warm-cache number",
            "key_passes": key_passes,
            "parallelism": "independent sequences per GPU (replicas), no collective"}


def algorithmic_bytes(cfg, r):
    """Bytes the method must move through HBM for one step (per GPU)."""
    from paper_2605_26678_b200 import nkv
    k = nkv.nkv_keep_per_head(cfg.seq_len, r)
    row = cfg.head_dim * cfg.elem_bytes
    per_unit = {
        "anchors": cfg.seq_len * row + 4 * cfg.seq_len,          # first touch of K, 1/norm out
        "score": cfg.seq_len * row + 16 * cfg.seq_len,           # second touch of K, 1/norm in, 3 anomalies out
        "head": 16 * cfg.seq_len,                                # anomalies in, final score out
        "budget": 4 * cfg.seq_len,
        "select": 4 * cfg.seq_len + 4 * k,
        "compact": 4 * k * row + 4 * k,                          # K and V rows in and out, positions in
    }
    per_unit_min = cfg.seq_len * row + 4 * k * row               # K once + retained rows in and out
    return {s: v * cfg.units for s, v in per_unit.items()}, per_unit_min * cfg.units


# ----------------------------------------------------------------------------------------------
# CPU oracle legs
# ----------------------------------------------------------------------------------------------
def oracle_throughput(cfg, r, groups_kv, threads, keep=None):
    """Times the oracle over the given [(K[H,N,d], V[H,N,d])] host groups with `threads` workers."""
    import oracle
    oracle.lib()
    t0 = time.perf_counter()
    with ThreadPoolExecutor(max_workers=threads) as ex:
        results = list(ex.map(lambda kv: oracle.compress_group(kv[0], kv[1], r), groups_kv))
    dt = time.perf_counter() - t0
    keys = len(groups_kv) * cfg.kv_heads * cfg.seq_len
    if keep is not None:
        keep.extend(results)
    return keys / dt, dt


def run_reference(args, cfg, r):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    cores = os.cpu_count() or 1
    threads = min(cores, 32)
    per_step_groups = max(1, min(cfg.groups, threads))
    # bound the whole run to a few minutes: a 32k group costs ~3 s of one core
    cost_per_group = 3.0 * (cfg.seq_len / 32768.0) * (cfg.head_dim / 128.0)
    budget_s = 150.0
    total_steps = args.steps + args.warmup
    while per_step_groups > 1 and total_steps * cost_per_group * per_step_groups / threads > budget_s:
        per_step_groups -= 1
    groups = list(range(per_step_groups))
    K, V = wl.make_groups(cfg, groups, "cpu")
    data = [(K[i], V[i]) for i in range(len(groups))]
    for _ in range(args.warmup):
        oracle_throughput(cfg, r, data, threads)
    t0 = time.perf_counter()
    for _ in range(args.steps):
        oracle_throughput(cfg, r, data, threads)
    dt = time.perf_counter() - t0
    keys = args.steps * len(groups) * cfg.kv_heads * cfg.seq_len
    value = keys / dt
    sample = "%d of %d layer groups of %s per step (%d keys), %d threads" % (
        len(groups), cfg.groups, cfg.name, len(groups) * cfg.kv_heads * cfg.seq_len, min(threads, len(groups)))
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": 1e3 * dt / max(1, args.steps),
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": bench_config(cfg, r, args.key_passes),
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": min(threads, len(groups)), "kind": "oracle",
                         "sample": sample},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line))


# ----------------------------------------------------------------------------------------------
# CUDA arm
# ----------------------------------------------------------------------------------------------
def run_nkv(args, cfg, r):
    from paper_2605_26678_b200 import nkv

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device (no CPU fallback); use --impl reference for the oracle arm")
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    dist = None
    if world > 1:
        import torch.distributed as dist_mod
        dist = dist_mod
        dist.init_process_group("nccl", device_id=dev)

    def barrier():
        if dist is not None:
            dist.barrier()
        torch.cuda.synchronize()

    # every rank owns an independent cache of the same shape (different sequences)
    my_cfg = replica_config(cfg, rank)
    K, V = wl.make_cache(my_cfg, dev, groups_per_call=4)
    params = nkv.nkv_default_params()
    ws = nkv.alloc_workspace(K, params)
    out = nkv.alloc_outputs(K, V, r)
    h = nkv.handle(local)
    nkv.nkv_set_key_passes(args.key_passes, h)

    def step():
        nkv.nkv_compress(K, V, r, params, out=out, ws=ws, h=h)

    # ---- device-resident throughput --------------------------------------------------------
    for _ in range(max(3, args.warmup)):
        step()
    barrier()
    sampler = ClockSampler(physical_gpu_index(local))
    sampler.start()
    launches0 = nkv.nkv_launch_count(h)
    ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    barrier()
    ev0.record()
    for _ in range(args.steps):
        step()
    ev1.record()
    barrier()
    ms_total = ev0.elapsed_time(ev1)
    launches = nkv.nkv_launch_count(h) - launches0
    clocks = sampler.stop()
    status = nkv.nkv_last_device_status(ws, h)
    if status != nkv.NKV_OK:
        raise SystemExit("device status %d after the timed region" % status)
    value, ms_per_step = whole_job_throughput(ms_total, args.steps, cfg.keys, world, dist, dev)
    if clocks.get("sm_mhz"):
        # million SM cycles per step at the clock sampled under load: comparable between runs that the power cap
        # held at different clocks
        clocks["sm_mcycles_per_step"] = ms_per_step * clocks["sm_mhz"] / 1000.0

    # ---- per-stage device time (events recorded on the launching stream inside the library) --
    nkv.nkv_set_timing(True, h)
    stage_ms = [[] for _ in range(nkv.NKV_NUM_STAGES)]
    for _ in range(min(args.steps, 20)):
        step()
        for i, v in enumerate(nkv.nkv_get_stage_ms(h)):
            stage_ms[i].append(v)
    nkv.nkv_set_timing(False, h)
    stage_avg = {name: sum(v) / len(v) for name, v in zip(nkv.STAGE_NAMES, stage_ms)}
    stage_bytes, bytes_min = algorithmic_bytes(cfg, r)
    peak, peak_src = measured_peak()
    dominant = max(stage_avg, key=stage_avg.get)
    dom_gbs = stage_bytes[dominant] / (stage_avg[dominant] * 1e-3) / 1e9
    kernel_name, kernel_src = STAGE_KERNEL[dominant]
    per_key = measured_traffic_per_key(kernel_name, kernel_src, cfg.dtype, cfg.head_dim)
    roofline = {
        "bound": "hbm", "kernel": kernel_name, "stage": dominant, "achieved": dom_gbs, "peak": peak, "unit": "GB/s",
        "frac": dom_gbs / peak,
        "traffic": per_key * cfg.keys if per_key is not None else None,
        "peak_source": peak_src,
        "algorithmic_bytes_per_launch": stage_bytes[dominant], "ms_per_launch": stage_avg[dominant],
        "stages_ms": stage_avg,
        "stages_gbs": {s: stage_bytes[s] / (stage_avg[s] * 1e-3) / 1e9 for s in stage_avg if stage_avg[s] > 1e-3},
    }
    pipe_gbs = bytes_min / (ms_per_step * 1e-3) / 1e9
    pipeline = {
        "algorithmic_bytes_per_step": bytes_min, "achieved_gbs": pipe_gbs,
        "frac_of_measured": pipe_gbs / peak, "frac_of_nominal_8TBs": pipe_gbs / NOMINAL_HBM_GBS,
        "nominal_kv_gbs": cfg.kv_bytes() / (ms_per_step * 1e-3) / 1e9,
        "ms_per_36_layer_sequence": ms_per_step / cfg.batch,
    }

    # ---- end to end through the host-buffer entry point -------------------------------------
    e2e = None
    if not args.no_e2e:
        e2e = run_e2e(args, cfg, r, K, V, h, params, dist, dev, world)

    # ---- CPU oracle beside it (rank 0, single GPU runs only): waves of layer groups for about 12 s
    cpu = None
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        cores = os.cpu_count() or 1
        threads = min(cores, 32)
        done_groups, spent, g0 = 0, 0.0, 0
        oracle_groups = []   # the oracle's results for groups 0, 1, ...: reused for the near-tie count
        while g0 < cfg.groups and spent < 12.0:
            wave = list(range(g0, min(cfg.groups, g0 + threads)))
            data = [(K[g].cpu(), V[g].cpu()) for g in wave]
            _, dt = oracle_throughput(cfg, r, data, threads, keep=oracle_groups if g0 == 0 else None)
            spent += dt
            done_groups += len(wave)
            g0 += len(wave)
        cpu = {"value": done_groups * cfg.kv_heads * cfg.seq_len / spent, "unit": UNIT,
               "cores": min(threads, done_groups), "kind": "oracle",
               "sample": "%d of %d layer groups (%d keys) in %.1f s, %d worker threads" % (
                   done_groups, cfg.groups, done_groups * cfg.kv_heads * cfg.seq_len, spent, threads)}

    # ---- near-tie swaps: the timed call's retained sets against the oracle's on the groups it just did ----
    swaps = None
    if cpu is not None and oracle_groups:
        swaps = near_tie_swaps(K, V, r, params, ws, h, oracle_groups)

    # ---- the other configurations (one GPU, rank 0 only; the headline line above is unaffected) ----
    table = None
    if rank == 0 and world == 1 and not args.no_config_table:
        del K, V, out, ws
        torch.cuda.empty_cache()
        table = config_table(args, cfg, r, ms_per_step, h, peak)

    if rank == 0:
        line = {
            "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
            "warmup": max(3, args.warmup), "ms_per_step": ms_per_step, "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "f32", "data": "synthetic",
            "config": bench_config(cfg, r, args.key_passes),
            "clocks": clocks, "e2e": e2e, "gpu_launches": launches, "roofline": roofline, "pipeline": pipeline,
            "cpu_baseline": cpu, "near_tie_swaps": swaps, "configs": table,
        }
        print(json.dumps(line))
    if dist is not None:
        dist.destroy_process_group()


def near_tie_swaps(K, V, r, params, ws, h, oracle_groups):
    """Retained sets of the CUDA path against the oracle's on the first groups of the workload: heads whose
    sets differ, tokens that changed sides, and how far (in score) the farthest of them is from the threshold
    it crossed.  The oracle results are the ones the CPU baseline leg just produced."""
    import numpy as np
    from paper_2605_26678_b200 import nkv
    res = nkv.nkv_compress(K, V, r, params, ws=ws, want_a_star=True, h=h)
    torch.cuda.synchronize()
    heads = with_swaps = tokens = 0
    worst_score = worst_gap = 0.0
    for g, ref in enumerate(oracle_groups):
        a_gpu = res.a_star[g].cpu().numpy()
        idx = res.idx[g].cpu().numpy()
        offs = res.head_offsets[g].cpu().numpy()
        fin = np.isfinite(ref.a_star)
        worst_score = max(worst_score, float(np.abs(a_gpu[fin] - ref.a_star[fin]).max()))
        for hd in range(K.shape[1]):
            heads += 1
            want = set(ref.sel.idx[ref.sel.offsets[hd]:ref.sel.offsets[hd + 1]].tolist())
            got = set(idx[offs[hd]:offs[hd + 1]].tolist())
            diff = want ^ got
            if not diff:
                continue
            with_swaps += 1
            tokens += len(diff)
            thr = float(ref.a_star[hd, sorted(want)].min()) if want else 0.0
            worst_gap = max(worst_gap, max(abs(float(ref.a_star[hd, i]) - thr) for i in diff))
    return {"groups_checked": len(oracle_groups), "heads_checked": heads, "heads_with_swaps": with_swaps,
            "swapped_tokens": tokens, "max_score_difference": worst_score,
            "max_distance_of_a_swapped_token_from_its_heads_threshold": worst_gap}


def time_steps(step, steps, flush=None):
    """Milliseconds per step: back to back (flush None), or each step timed alone after `flush()`."""
    for _ in range(3):
        step()
    torch.cuda.synchronize()
    if flush is None:
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for _ in range(steps):
            step()
        e1.record()
        torch.cuda.synchronize()
        return e0.elapsed_time(e1) / steps
    total = 0.0
    for _ in range(steps):
        flush()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        step()
        e1.record()
        torch.cuda.synchronize()
        total += e0.elapsed_time(e1)
    return total / steps


def config_table(args, head_cfg, head_r, head_ms, h, peak):
    """ms, keys/s and pipeline fraction of every benchmark configuration (and of the other ratios of the
    headline one).  Caches that fit L2 are timed twice: warm (back to back) and cold (a buffer larger than L2
    is overwritten before every step)."""
    from paper_2605_26678_b200 import nkv
    dev = torch.device("cuda", torch.cuda.current_device())
    params = nkv.nkv_default_params()
    flush_buf = torch.empty(512 << 20, dtype=torch.uint8, device=dev)
    rows = {}
    for name, cfg in wl.CONFIGS.items():
        K, V = wl.make_cache(cfg, dev, groups_per_call=4)
        ws = nkv.alloc_workspace(K, params)
        for r in cfg.ratios:
            if name == head_cfg.name and r == head_r:
                ms = head_ms
                cold = None
            else:
                out = nkv.alloc_outputs(K, V, r)
                step = lambda: nkv.nkv_compress(K, V, r, params, out=out, ws=ws, h=h)
                small = cfg.kv_bytes() < (4 << 30)
                ms = time_steps(step, 50 if small else 10)
                cold = time_steps(step, 20, flush=lambda: flush_buf.fill_(1)) if small else None
                del out
            _, bytes_min = algorithmic_bytes(cfg, r)
            row = {"ms_per_step": ms, "keys_per_s": cfg.keys / (ms * 1e-3),
                   "pipeline_frac_of_measured": bytes_min / (ms * 1e-3) / 1e9 / peak,
                   "ms_per_sequence": ms / cfg.batch}
            if cold is not None:
                row["l2"] = "warm (back to back); cold = every step after a 512 MB overwrite"
                row["ms_per_step_cold"] = cold
                row["pipeline_frac_of_measured_cold"] = bytes_min / (cold * 1e-3) / 1e9 / peak
            rows["%s r=%.2f" % (name, r)] = row
        del K, V, ws
        torch.cuda.empty_cache()
    return rows


def run_e2e(args, cfg, r, K, V, h, params, dist, dev, world):
    """Same metric with HOST input and output buffers: nkv_compress_host, copies inside the timed region."""
    from paper_2605_26678_b200 import nkv
    G, H, N, d = K.shape
    k = nkv.nkv_keep_per_head(N, r)
    # keep the pinned footprint well inside the host's memory
    avail = 0
    try:
        for line in open("/proc/meminfo"):
            if line.startswith("MemAvailable"):
                avail = int(line.split()[1]) * 1024
    except Exception:
        pass
    need_full = cfg.kv_bytes() * (1.0 + (1.0 - r)) * 1.1
    groups = G if avail > 3 * need_full * max(1, world) else min(G, cfg.layers)
    try:
        Kh = torch.empty((groups, H, N, d), dtype=K.dtype, pin_memory=True)
        Vh = torch.empty((groups, H, N, d), dtype=V.dtype, pin_memory=True)
        Kh.copy_(K[:groups])
        Vh.copy_(V[:groups])
        out = nkv.Compressed(torch.empty((groups, H * k, d), dtype=K.dtype, pin_memory=True),
                             torch.empty((groups, H * k, d), dtype=V.dtype, pin_memory=True),
                             torch.empty((groups, H * k), dtype=torch.int32, pin_memory=True),
                             torch.empty((groups, H + 1), dtype=torch.int32, pin_memory=True),
                             torch.empty((groups, H), dtype=torch.int32, pin_memory=True), None)
    except RuntimeError as e:
        return {"value": None, "unit": UNIT, "error": "pinned allocation failed: %s" % str(e)[:80]}
    chunk = 4
    staging = torch.empty(nkv.nkv_host_staging_bytes(H, N, d, nkv._dtype_code(K), r, chunk, params, h),
                          dtype=torch.uint8, device=dev)
    torch.cuda.synchronize()

    def step():
        nkv.nkv_compress_host(Kh, Vh, r, out, staging, chunk, params, h)

    step()  # warm-up
    if dist is not None:
        dist.barrier()
    steps = max(1, args.e2e_steps)
    t0 = time.perf_counter()
    for _ in range(steps):
        step()          # returns after the results are on the host
    dt = time.perf_counter() - t0
    t = torch.tensor([dt], dtype=torch.float64, device=dev)
    if dist is not None:
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
    dt = float(t.item())
    keys = groups * H * N * world
    h2d = Kh.numel() * Kh.element_size() + Vh.numel() * Vh.element_size()
    d2h = sum(x.numel() * x.element_size() for x in (out.k_out, out.v_out, out.idx, out.head_offsets, out.budgets))
    return {"value": keys * steps / dt, "unit": UNIT, "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h,
            "steps": steps, "ms_per_step": 1e3 * dt / steps,
            "workload": "%d of %d layer groups per GPU, pinned host buffers, %d groups per staged chunk" % (
                groups, G, chunk),
            "pcie_gbs": (h2d + d2h) / (dt / steps) / 1e9}


def main():
    args = parse_args()
    cfg = wl.ALL_CONFIGS[args.workload]
    r = args.ratio if args.ratio is not None else (DEFAULT_RATIO if DEFAULT_RATIO in cfg.ratios else cfg.ratios[0])
    if args.impl == "reference":
        run_reference(args, cfg, r)
    else:
        run_nkv(args, cfg, r)


if __name__ == "__main__":
    main()
