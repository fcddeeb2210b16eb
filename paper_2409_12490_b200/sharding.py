"""Host-side logic of multi-GPU runs.

The path has no exchange step: every (batch item, head) is independent in Algorithm 1 and
Algorithm 2 and the carried score S' is per head.  N ranks therefore run N independent batch
items (weak scaling); the only communication is the barrier around the timed region and the
max-over-ranks of the timings, which works on any torch.distributed backend (NCCL on GPUs,
gloo in the CPU tests).
"""
from __future__ import annotations

import os
from dataclasses import dataclass

import torch


@dataclass(frozen=True)
class RankInfo:
    rank: int
    world: int
    local_rank: int

    @classmethod
    def from_env(cls) -> "RankInfo":
        return cls(int(os.environ.get("RANK", "0")), int(os.environ.get("WORLD_SIZE", "1")),
                   int(os.environ.get("LOCAL_RANK", "0")))


def layer_seed_for_rank(layer: int, rank: int, n_layers: int = 1) -> int:
    """Each rank works on its own batch item: same shapes, its own seeded draw.  The value is
    the `layer` argument of inputs.make_qkv; ranks never share a draw."""
    return rank * n_layers + layer


def head_shard(n_kv_heads: int, rank: int, world: int) -> range:
    """KV heads owned by `rank` when one problem is split across ranks by KV group (each rank
    also owns the g query heads of its KV heads; no collective is needed on the path)."""
    if n_kv_heads % world:
        raise ValueError(f"{n_kv_heads} KV heads do not split evenly over {world} ranks")
    per = n_kv_heads // world
    return range(rank * per, (rank + 1) * per)


def max_over_ranks(values, dist=None, device="cpu"):
    """Element-wise maximum of a list of floats over all ranks (identity without a process group)."""
    if dist is None or not dist.is_initialized() or dist.get_world_size() == 1:
        return [float(v) for v in values]
    t = torch.tensor(list(values), dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return t.tolist()


def aggregate_time_metric(ms_per_step_local: float, world: int, dist=None, device="cpu"):
    """Whole-job numbers from a per-rank step time: the job's step time is the slowest rank's;
    units per second add up over the ranks (one layer pass per rank per step)."""
    (ms,) = max_over_ranks([ms_per_step_local], dist, device)
    return {"ms_per_step": ms, "layer_passes_per_s": world * 1e3 / ms}
