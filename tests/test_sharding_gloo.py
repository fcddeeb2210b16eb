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
                                            max_over_ranks, shard_heads)


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


def _shard_worker(rank, world, port, out):
    """One rank of a head-sharded layer on CPU: the oracle stands in for the kernels (same inputs, same
    views, same parameters as the CUDA path would get); the parameters and views are what is under test."""
    import numpy as np
    import oracle
    from paper_2409_12490_b200 import binding as cp
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        cfg = CONFIGS["C1"].with_(seq_len=512, n_q_heads=8, n_kv_heads=4)
        Q, K, V = make_qkv(cfg, threads=1)                       # every rank draws the same full problem
        sh = shard_heads(cfg, rank, world)
        q, k, v = sh.slice_q(Q), sh.slice_kv(K), sh.slice_kv(V)
        # the parameters the C ABI would receive for this shard: head counts of the shard, strides of the FULL tensors
        p = cp.Problem.from_config(sh.cfg).params(Q=q, K=k, V=v, O=sh.slice_q(torch.empty_like(Q)))
        assert (p.n_q_heads, p.n_kv_heads) == (cfg.n_q_heads // world, cfg.n_kv_heads // world)
        assert list(p.q_stride) == list(Q.stride()[:3]) and list(p.k_stride) == list(K.stride()[:3])
        g = cfg.n_q_heads // cfg.n_kv_heads
        assert q.storage_offset() == sh.q_heads.start * Q.stride(1) and k.storage_offset() == sh.kv_heads.start * K.stride(1)
        assert sh.q_heads.start == sh.kv_heads.start * g and len(sh.q_heads) == g * len(sh.kv_heads)
        # the shard's result with the oracle
        S = oracle.estimate(q, k, cfg.segment_size, cfg.block_size, est_scale=cfg.est_scale, alpha=cfg.alpha)
        idx, cnt = oracle.select(S, cfg.segment_size, cfg.block_size, cfg.budget_blocks)
        O, _ = oracle.sparse_attention(q, k, v, idx, cnt, cfg.segment_size, cfg.block_size, 1.0 / np.sqrt(cfg.head_dim))
        # gather the shards along the head axis and compare with the unsharded result (rank 0)
        parts = [torch.zeros(O.shape, dtype=torch.float64) for _ in range(world)]
        dist.all_gather(parts, torch.from_numpy(O))
        heads = [torch.zeros(2, dtype=torch.int64) for _ in range(world)]
        dist.all_gather(heads, torch.tensor([sh.q_heads.start, sh.q_heads.stop]))
        if rank == 0:
            cover = [h for a, b in (t.tolist() for t in heads) for h in range(a, b)]
            assert cover == list(range(cfg.n_q_heads))           # every query head exactly once, in order
            S_full = oracle.estimate(Q, K, cfg.segment_size, cfg.block_size, est_scale=cfg.est_scale, alpha=cfg.alpha)
            idx_f, cnt_f = oracle.select(S_full, cfg.segment_size, cfg.block_size, cfg.budget_blocks)
            O_full, _ = oracle.sparse_attention(Q, K, V, idx_f, cnt_f, cfg.segment_size, cfg.block_size, 1.0 / np.sqrt(cfg.head_dim))
            assert np.array_equal(torch.cat(parts, dim=1).numpy(), O_full)
        agg = aggregate_time_metric(5.0 + rank, world, dist, replicas=False)
        assert agg["ms_per_step"] == 5.0 + world - 1 and agg["layer_passes_per_s"] == pytest.approx(1e3 / agg["ms_per_step"])
        dist.barrier()
        out.put((rank, "ok"))
    finally:
        dist.destroy_process_group()


def test_head_sharded_layer_on_two_gloo_ranks_equals_the_unsharded_layer():
    world, port = 2, _free_port()
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    procs = [ctx.Process(target=_shard_worker, args=(r, world, port, out)) for r in range(world)]
    for p in procs:
        p.start()
    for p in procs:
        p.join(180)
        assert p.exitcode == 0
    assert sorted(out.get(timeout=5) for _ in range(world)) == [(0, "ok"), (1, "ok")]


def test_shard_heads_views():
    cfg = CONFIGS["C4"]
    for world in (1, 2, 4, 8):
        seen_q, seen_kv = [], []
        for r in range(world):
            sh = shard_heads(cfg, r, world)
            assert sh.cfg.n_q_heads * world == cfg.n_q_heads and sh.cfg.n_kv_heads * world == cfg.n_kv_heads
            assert sh.cfg.seq_len == cfg.seq_len and sh.cfg.budget_blocks == cfg.budget_blocks
            seen_q += list(sh.q_heads); seen_kv += list(sh.kv_heads)
        assert seen_q == list(range(cfg.n_q_heads)) and seen_kv == list(range(cfg.n_kv_heads))
