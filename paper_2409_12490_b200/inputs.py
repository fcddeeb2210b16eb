"""Seeded synthetic Q/K/V with the structure the method relies on.

This module only draws random inputs.  It contains none of the method's arithmetic
(no summaries, scores, selection or attention) and is the one module that both the
CUDA path's tests/bench and the CPU oracle's tests may use.

Recipe (stands in for long-context QA activations, which are not available):
  * per KV head h: ``ncl`` cluster centres C_h[c] ~ N(0, I_d); the key at position u
    belongs to a cluster that is piecewise constant over runs of U{blk..4*blk} tokens;
    K_h[u] = C_h[z(u)] + 0.3 * eps;  V_h[u] ~ N(0, I_d)
  * per query head q (KV head h = q // g): a target cluster that is piecewise constant
    over dwells of U{2*seg..6*seg} tokens; an AR(1) walk
    Q_q[t] = rho * Q_q[t-1] + (1-rho) * C_h[c(t)] + 0.5 * sqrt(1-rho^2) * eps_t,
    Q_q[0] = C_h[c(0)]
so that attention mass is sparse (queries point at one cluster's keys) and neighbouring
queries share their critical keys (the locality the paper's Section 2.2 observes).
Values are rounded once to the storage dtype; every consumer sees the same bits.
"""
from __future__ import annotations

from concurrent.futures import ThreadPoolExecutor

import numpy as np
import torch

from .configs import Config

BASE_SEED = 20240912


def _piecewise_ids(rng: np.random.Generator, n: int, lo: int, hi: int, n_ids: int) -> np.ndarray:
    """ids[t] constant on consecutive runs whose lengths are uniform in [lo, hi]."""
    n_runs = n // lo + 2
    lengths = rng.integers(lo, hi + 1, size=n_runs)
    ids = rng.integers(0, n_ids, size=n_runs)
    return np.repeat(ids, lengths)[:n]


def _ar1(x: np.ndarray, rho: float) -> np.ndarray:
    """y[0] = x[0], y[t] = rho*y[t-1] + x[t] along axis 0."""
    from scipy.signal import lfilter

    return lfilter([1.0], [1.0, -rho], x, axis=0)


def _to_storage(x: np.ndarray, dtype: str) -> torch.Tensor:
    t = torch.from_numpy(np.ascontiguousarray(x, dtype=np.float32))
    return t.to({"bf16": torch.bfloat16, "f16": torch.float16, "f32": torch.float32}[dtype])


def make_qkv(cfg: Config, layer: int = 0, threads: int = 8):
    """Return (Q[B,Hq,n,d], K[B,Hkv,n,d], V[B,Hkv,n,d]) as CPU tensors in cfg.dtype."""
    B, Hq, Hkv, n, d = cfg.batch, cfg.n_q_heads, cfg.n_kv_heads, cfg.seq_len, cfg.head_dim
    g = Hq // Hkv
    seed = BASE_SEED + 1000 * cfg.index + layer
    tdt = {"bf16": torch.bfloat16, "f16": torch.float16, "f32": torch.float32}[cfg.dtype]
    Q = torch.empty((B, Hq, n, d), dtype=tdt)
    K = torch.empty((B, Hkv, n, d), dtype=tdt)
    V = torch.empty((B, Hkv, n, d), dtype=tdt)

    # structure (cluster runs, query dwells) depends on the config only, so the layers of
    # a stack share it; centres and noise are drawn per layer
    struct_ss = np.random.SeedSequence([BASE_SEED, cfg.index, 7])
    value_ss = np.random.SeedSequence([seed, 11])

    def kv_head(b: int, h: int, sseq, vseq):
        srng = np.random.Generator(np.random.PCG64(sseq))
        vrng = np.random.Generator(np.random.PCG64(vseq))
        centres = vrng.standard_normal((cfg.n_clusters, d), dtype=np.float32)
        z = _piecewise_ids(srng, n, cfg.block_size, 4 * cfg.block_size, cfg.n_clusters)
        k = centres[z] + np.float32(0.3) * vrng.standard_normal((n, d), dtype=np.float32)
        v = vrng.standard_normal((n, d), dtype=np.float32)
        K[b, h] = _to_storage(k, cfg.dtype)
        V[b, h] = _to_storage(v, cfg.dtype)
        return centres

    def q_head(b: int, q: int, centres, sseq, vseq):
        srng = np.random.Generator(np.random.PCG64(sseq))
        vrng = np.random.Generator(np.random.PCG64(vseq))
        c = _piecewise_ids(srng, n, 2 * cfg.segment_size, 6 * cfg.segment_size, cfg.n_clusters)
        x = np.float32(1.0 - cfg.rho) * centres[c]
        x += np.float32(0.5 * np.sqrt(1.0 - cfg.rho ** 2)) * vrng.standard_normal((n, d), dtype=np.float32)
        x[0] = centres[c[0]]
        Q[b, q] = _to_storage(_ar1(x.astype(np.float64), cfg.rho), cfg.dtype)

    s_kv = struct_ss.spawn(B * Hkv + B * Hq)
    v_kv = value_ss.spawn(B * Hkv + B * Hq)
    with ThreadPoolExecutor(max_workers=max(1, threads)) as ex:
        cents = list(ex.map(lambda bh: kv_head(bh // Hkv, bh % Hkv, s_kv[bh], v_kv[bh]), range(B * Hkv)))
        off = B * Hkv
        list(ex.map(lambda bq: q_head(bq // Hq, bq % Hq, cents[(bq // Hq) * Hkv + (bq % Hq) // g],
                                      s_kv[off + bq], v_kv[off + bq]), range(B * Hq)))
    return Q, K, V


def make_uniform_qkv(B, Hq, Hkv, n, d, dtype="bf16", seed=0, scale=1.0):
    """Plain i.i.d. N(0, scale^2) Q/K/V for edge-case tests (no cluster structure)."""
    rng = np.random.Generator(np.random.PCG64(seed))
    mk = lambda h: _to_storage(scale * rng.standard_normal((B, h, n, d), dtype=np.float32), dtype)
    return mk(Hq), mk(Hkv), mk(Hkv)
