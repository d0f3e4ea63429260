"""The N > 1 path of the bench on CPU: two gloo ranks.

The compression path has no exchange step, so N GPUs run N independent replicas.  What the
ranks share is host logic only: each rank derives its own cache (same shape, different
sequences) and the job's throughput is all ranks' keys over the slowest rank's time.
"""
import os
import socket

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

import bench
from paper_2605_26678_b200 import workloads as wl


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _rank_main(rank, world, port, out_dir):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    cfg = wl.tiny_config("replica", kv_heads=2, head_dim=64, seq_len=96, layers=1)
    mine = bench.replica_config(cfg, rank)
    K, _ = wl.make_cache(mine)
    # rank r pretends to need (r + 1) * 10 ms for 5 steps
    value, ms = bench.whole_job_throughput(10.0 * (rank + 1), 5, cfg.keys, world, dist)
    sums = [torch.zeros(1, dtype=torch.float64) for _ in range(world)]
    dist.all_gather(sums, K.double().sum().reshape(1))
    if rank == 0:
        torch.save({"value": value, "ms": ms, "sums": [float(x) for x in sums], "keys": cfg.keys},
                   os.path.join(out_dir, "r0.pt"))
    dist.barrier()
    dist.destroy_process_group()


def test_two_replicas_own_different_caches_and_time_is_max_over_ranks(tmp_path):
    world = 2
    mp.spawn(_rank_main, args=(world, _free_port(), str(tmp_path)), nprocs=world, join=True)
    got = torch.load(os.path.join(str(tmp_path), "r0.pt"))
    assert got["ms"] == 20.0 / 5                        # the slower rank's 20 ms over 5 steps
    assert got["value"] == got["keys"] * world / (got["ms"] * 1e-3)
    assert got["sums"][0] != got["sums"][1]             # different sequences on the two ranks


def test_replica_config_keeps_the_shape():
    cfg = wl.CONFIGS["cfg4_qwen3_4b_32k_b4"]
    other = bench.replica_config(cfg, 3)
    assert (other.groups, other.kv_heads, other.seq_len, other.head_dim, other.dtype) == (
        cfg.groups, cfg.kv_heads, cfg.seq_len, cfg.head_dim, cfg.dtype)
    assert other.base_seed != cfg.base_seed and bench.replica_config(cfg, 0) is cfg
