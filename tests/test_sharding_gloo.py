"""The N>1 host logic (per-rank inputs, max-over-ranks timing, head sharding) on two gloo ranks, CPU only."""
import os
import socket

import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from paper_2409_12490_b200 import CONFIGS
from paper_2409_12490_b200.inputs import make_qkv
from paper_2409_12490_b200.sharding import (aggregate_time_metric, head_shard, layer_seed_for_rank,
                                            max_over_ranks)


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, out):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        cfg = CONFIGS["C1"].with_(seq_len=256)
        Q, K, V = make_qkv(cfg, layer=layer_seed_for_rank(0, rank), threads=1)
        checksum = float(Q.double().sum())
        # ranks must draw different inputs
        sums = [torch.zeros(1, dtype=torch.float64) for _ in range(world)]
        dist.all_gather(sums, torch.tensor([checksum], dtype=torch.float64))
        assert len({round(float(s), 6) for s in sums}) == world
        # the job's time is the slowest rank's
        local_ms = 10.0 + 5.0 * rank
        agg = aggregate_time_metric(local_ms, world, dist)
        assert agg["ms_per_step"] == 10.0 + 5.0 * (world - 1)
        assert agg["layer_passes_per_s"] == pytest.approx(world * 1e3 / agg["ms_per_step"])
        assert max_over_ranks([float(rank), 1.0], dist) == [float(world - 1), 1.0]
        dist.barrier()
        out.put((rank, "ok"))
    finally:
        dist.destroy_process_group()


def test_two_gloo_ranks():
    world, port = 2, _free_port()
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    procs = [ctx.Process(target=_worker, args=(r, world, port, out)) for r in range(world)]
    for p in procs:
        p.start()
    for p in procs:
        p.join(120)
        assert p.exitcode == 0
    assert sorted(out.get(timeout=5) for _ in range(world)) == [(0, "ok"), (1, "ok")]


def test_head_shard_partitions_kv_heads():
    for hkv, world in [(8, 1), (8, 2), (8, 4), (8, 8), (4, 2)]:
        seen = [h for r in range(world) for h in head_shard(hkv, r, world)]
        assert seen == list(range(hkv))
    with pytest.raises(ValueError):
        head_shard(4, 0, 3)


def test_single_process_identity():
    assert max_over_ranks([1.5, 2.5]) == [1.5, 2.5]
    assert aggregate_time_metric(4.0, 1)["layer_passes_per_s"] == 250.0
