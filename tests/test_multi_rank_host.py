"""The N>1 path of the benchmark on CPU: two gloo ranks shard the prompts without any data-path
collective, and the only communication is the max of the per-rank times."""
import os
import sys

import numpy as np
import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)


def _worker(rank, world, port, out_dir):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    import bench
    from paper_2502_01941_b200 import workloads as wl
    cfg = bench.rank_config(wl.CONFIGS[0], rank)
    off = wl.all_shot_offsets(cfg)
    _, K, _ = wl.prefill_unit(cfg, 0, 0, off[0])
    local_ms = 10.0 + 5.0 * rank                       # rank 1 is the slow one
    ms = bench.max_over_ranks(local_ms, world, torch.device("cpu"))
    tokens = cfg.B * cfg.N * world
    np.save(os.path.join(out_dir, f"r{rank}.npy"), np.array([ms, tokens, float(K.float().sum()), float(off.sum())]))
    dist.barrier()
    dist.destroy_process_group()


def test_two_gloo_ranks_shard_prompts_and_take_the_slowest_time(tmp_path):
    world, port = 2, 29531 + os.getpid() % 200
    mp.spawn(_worker, args=(world, port, str(tmp_path)), nprocs=world, join=True)
    r0, r1 = np.load(tmp_path / "r0.npy"), np.load(tmp_path / "r1.npy")
    assert r0[0] == r1[0] == 15.0                      # every rank reports the slowest rank's time
    assert r0[1] == r1[1] == 2 * 512                   # whole-job units = sum over ranks
    assert r0[2] != r1[2]                              # each rank draws its own prompts (distinct seeds)
