"""Host-side logic of multi-GPU runs.

The path has no exchange step: every (batch item, head) is independent in Algorithm 1 and
Algorithm 2 and the carried score S' is per head.  Two ways to use N ranks follow from that:

* head sharding (one problem, strong scaling): rank p owns the KV heads ``head_shard(Hkv, p, N)``
  and the g query heads of each of them.  Its sub-problem is the same layer with fewer heads, on
  strided views of the full tensors; no collective is needed on the path (a consumer that is not
  itself head-parallel can all-gather O along the head axis afterwards);
* replicas (weak scaling): every rank runs its own batch item of the same shape.

The only communication either way is the barrier around the timed region and the max-over-ranks
of the timings, which works on any torch.distributed backend (NCCL on GPUs, gloo in the CPU tests).
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
    """Replica mode: each rank works on its own batch item: same shapes, its own seeded draw.  The value
    is the `layer` argument of inputs.make_qkv; ranks never share a draw."""
    return rank * n_layers + layer


def head_shard(n_kv_heads: int, rank: int, world: int) -> range:
    """KV heads owned by `rank` when one problem is split across ranks by KV group (each rank
    also owns the g query heads of its KV heads; no collective is needed on the path)."""
    if n_kv_heads % world:
        raise ValueError(f"{n_kv_heads} KV heads do not split evenly over {world} ranks")
    per = n_kv_heads // world
    return range(rank * per, (rank + 1) * per)


@dataclass(frozen=True)
class HeadShard:
    """What one rank of a head-sharded layer works on."""
    kv_heads: range          # KV heads of the full problem owned by this rank
    q_heads: range           # query heads of the full problem owned by this rank
    cfg: object              # the rank's sub-problem: the full config with its own head counts

    def slice_q(self, t: torch.Tensor) -> torch.Tensor:
        """View of a [B, Hq, ...] tensor of the full problem (Q, O, S, idx, cnt, lse) on this rank's query heads."""
        return t[:, self.q_heads.start:self.q_heads.stop]

    def slice_kv(self, t: torch.Tensor) -> torch.Tensor:
        """View of a [B, Hkv, ...] tensor of the full problem (K, V) on this rank's KV heads."""
        return t[:, self.kv_heads.start:self.kv_heads.stop]


def shard_heads(cfg, rank: int, world: int) -> HeadShard:
    """Head-sharded sub-problem of `rank`: KV heads head_shard(Hkv, rank, world) and their g query heads.
    Query head h of the full problem uses KV head h // g, so the rank's query heads are the contiguous
    range [kv.start * g, kv.stop * g) and inside the shard local head h' still maps to local KV head h' // g."""
    kv = head_shard(cfg.n_kv_heads, rank, world)
    g = cfg.n_q_heads // cfg.n_kv_heads
    q = range(kv.start * g, kv.stop * g)
    sub = cfg.with_(name=f"{cfg.name}[kv {kv.start}:{kv.stop} of {cfg.n_kv_heads}]", n_q_heads=len(q), n_kv_heads=len(kv))
    return HeadShard(kv, q, sub)


def max_over_ranks(values, dist=None, device="cpu"):
    """Element-wise maximum of a list of floats over all ranks (identity without a process group)."""
    if dist is None or not dist.is_initialized() or dist.get_world_size() == 1:
        return [float(v) for v in values]
    t = torch.tensor(list(values), dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return t.tolist()


def aggregate_time_metric(ms_per_step_local: float, world: int, dist=None, device="cpu", replicas: bool = True):
    """Whole-job numbers from a per-rank step time: the job's step time is the slowest rank's.  With replicas
    every rank completes one layer pass per step (they add up); with head sharding all ranks together
    complete one."""
    (ms,) = max_over_ranks([ms_per_step_local], dist, device)
    return {"ms_per_step": ms, "layer_passes_per_s": (world if replicas else 1) * 1e3 / ms}
