"""The N > 1 path on CPU: two gloo ranks exercise the sharding bookkeeping bench.py uses.

The decoding step has no exchange between units, so a multi-GPU run is one process per GPU, each
with its own image batch; what can go wrong is on the host: ranks generating the same images,
the step time not being the slowest rank's, the whole-job throughput not counting every rank.
"""
import os
import socket

import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from workloads import get_config, sharding


def _free_port() -> int:
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank: int, world: int, port: int, out_dir: str):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        cfg = get_config(0)
        gen = sharding.rank_generator(cfg, rank)
        q, k, v = gen.qkv(0, 3)
        # every rank decodes different images: gather a checksum of Q and compare
        mine = torch.tensor([float(q.double().sum()), float(k.double().abs().sum())], dtype=torch.float64)
        allsums = [torch.zeros_like(mine) for _ in range(world)]
        dist.all_gather(allsums, mine)
        assert all(not torch.equal(allsums[0], allsums[r]) for r in range(1, world))
        # ... but the head mask (the offline classification) is the same everywhere
        mask = gen.head_is_contextual.to(torch.int32)
        masks = [torch.zeros_like(mask) for _ in range(world)]
        dist.all_gather(masks, mask)
        assert all(torch.equal(masks[0], m) for m in masks)
        # the step time of the job is the slowest rank's
        sharding.barrier(dist)
        local_ms = 10.0 + 5.0 * rank
        ms = sharding.max_over_ranks(local_ms, dist)
        assert ms == 10.0 + 5.0 * (world - 1)
        tokens = cfg.batch * cfg.total_tokens
        value = sharding.job_throughput(world, tokens, ms)
        assert abs(value - world * tokens / (ms * 1e-3)) < 1e-6
        with open(os.path.join(out_dir, f"rank{rank}.ok"), "w") as f:
            f.write(f"{ms} {value}\n")
    finally:
        dist.destroy_process_group()


def test_two_gloo_ranks_shard_without_exchange(tmp_path):
    world = 2
    mp.spawn(_worker, args=(world, _free_port(), str(tmp_path)), nprocs=world, join=True)
    lines = [open(tmp_path / f"rank{r}.ok").read() for r in range(world)]
    assert lines[0] == lines[1]            # both ranks agree on the job's time and throughput


def test_single_process_helpers_need_no_group():
    assert sharding.max_over_ranks(3.5) == 3.5
    assert sharding.job_throughput(1, 1000, 2.0) == pytest.approx(500000.0)
    sharding.barrier(None)
