#!/usr/bin/env python
"""Benchmark of the CritiPrefill prefill hot path on B200.

One "step" is one pass of the whole path over one layer's Q/K/V:
    critiprefill_estimate -> critiprefill_select -> critiprefill_attention
on the 128K-token Llama3-8B-shaped workload (config C4), with inputs resident in HBM.
Prints ONE JSON line (rank 0).  `--impl reference` times the fp64 CPU oracle instead.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--config C4] [--impl ours|reference] [--shard replicas|heads]

With --gpus N > 1 and no torchrun environment the script starts the N ranks itself
(python -m torch.distributed.run on 127.0.0.1); under torchrun it is one of the ranks.
"""
from __future__ import annotations

import argparse
import json
import math
import os
import sys
import threading
import time

import numpy as np
import torch

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

from paper_2409_12490_b200 import CONFIGS  # noqa: E402
from paper_2409_12490_b200.inputs import make_qkv  # noqa: E402
from paper_2409_12490_b200.sharding import (RankInfo, aggregate_time_metric, layer_seed_for_rank, max_over_ranks,  # noqa: E402
                                            shard_heads)

METRIC = "128K prefill-attention ms (estimate+select+sparse attention, one layer)"


def load_ncu_counters():
    """Counters of the sparse attention kernel taken under ncu and kept beside the profile summaries
    (profiles/attention_counters.json: per workload the DRAM bytes read + written by one launch, the tensor-pipe
    and XU-pipe active percentages, and the commit and command they were captured with).  They describe the
    capture, not this run; the run's own figure is the event-timed `achieved`."""
    path = os.path.join(ROOT, "profiles", "attention_counters.json")
    if not os.path.exists(path):
        return {}
    with open(path) as f:
        return json.load(f)


def load_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            d = json.load(f)
        return {"bf16_tflops": d["bf16_tflops"], "bf16_tflops_sustained": d.get("bf16_tflops_sustained"),
                "hbm_gbs": d["hbm_gbs"], "source": "measured"}
    return {"bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0, "hbm_gbs": 6650.0, "source": "fallback"}


def flop_counts(cfg):
    """FLOPs per layer pass: what the sparse kernel executes (128x128 tiles, fully masked
    diagonal tiles skipped), the causal-useful part, and dense causal attention."""
    d, Hq, n, seg, blk, k, r, n1 = (cfg.head_dim, cfg.n_q_heads, cfg.seq_len, cfg.segment_size, cfg.block_size,
                                    cfg.budget_blocks, cfg.r, cfg.n1)
    tile = 4 * 128 * 128 * d                       # QK^T + PV for one 128x128 tile
    q_tiles = seg // 128
    executed = 0
    listed = 0
    for j in range(n1):
        cnt = min(k, (j + 1) * r)
        listed += cnt
        past_tiles = -(-(cnt - r) * blk // 128)
        for i in range(q_tiles):
            executed += (past_tiles + i + 1) * tile
    executed *= Hq * cfg.batch
    full_tiles = 4 * seg * blk * d * Hq * listed * cfg.batch          # every listed block against the whole segment
    useful = full_tiles - 4 * d * Hq * n1 * (seg * seg - seg * (seg + 1) // 2) * cfg.batch
    dense = 4 * d * Hq * n * (n + 1) // 2 * cfg.batch
    return {"executed": executed, "listed_full_tiles": full_tiles, "useful": useful, "dense": dense}


class ClockSampler:
    """Samples SM clock and throttle reasons through NVML while the timed region runs."""

    def __init__(self, index: int, period_s: float = 0.02):
        self.samples, self.reasons, self.max_mhz = [], set(), None
        self._stop = threading.Event()
        self._thread = None
        try:
            import pynvml
            pynvml.nvmlInit()
            self._nv = pynvml
            self._h = pynvml.nvmlDeviceGetHandleByIndex(index)
            self.max_mhz = pynvml.nvmlDeviceGetMaxClockInfo(self._h, pynvml.NVML_CLOCK_SM)
        except Exception:
            self._nv = None
        self.period = period_s

    def _run(self):
        nv = self._nv
        names = {
            nv.nvmlClocksThrottleReasonHwSlowdown: "hw_slowdown",
            nv.nvmlClocksThrottleReasonHwThermalSlowdown: "hw_thermal_slowdown",
            nv.nvmlClocksThrottleReasonSwThermalSlowdown: "sw_thermal_slowdown",
            nv.nvmlClocksThrottleReasonSwPowerCap: "sw_power_cap",
            nv.nvmlClocksThrottleReasonHwPowerBrakeSlowdown: "hw_power_brake",
        }
        while not self._stop.is_set():
            try:
                self.samples.append(nv.nvmlDeviceGetClockInfo(self._h, nv.NVML_CLOCK_SM))
                mask = nv.nvmlDeviceGetCurrentClocksThrottleReasons(self._h)
                for bit, name in names.items():
                    if mask & bit:
                        self.reasons.add(name)
            except Exception:
                pass
            time.sleep(self.period)

    def __enter__(self):
        if self._nv is not None:
            self._thread = threading.Thread(target=self._run, daemon=True)
            self._thread.start()
        return self

    def __exit__(self, *exc):
        self._stop.set()
        if self._thread is not None:
            self._thread.join()

    def summary(self):
        return {"sm_mhz": float(np.median(self.samples)) if self.samples else None, "sm_max_mhz": self.max_mhz,
                "reasons": sorted(self.reasons), "samples": len(self.samples)}


def physical_gpu_index(local: int) -> int:
    vis = os.environ.get("CUDA_VISIBLE_DEVICES")
    if vis:
        try:
            return int(vis.split(",")[local])
        except Exception:
            return local
    return local


# ----------------------------------------------------------------------------- reference arm
def oracle_step(cfg, Q, K, V, head, n_rows, seed, keep=None):
    """A bounded sample of one layer pass on the CPU oracle: Algorithm 1 + selection for one
    query head, Algorithm 2 for `n_rows` random rows of it.  Returns (seconds_est_sel, seconds_attn);
    with a dict in `keep` the oracle's results are left there for a comparison with the CUDA path."""
    import oracle
    g = cfg.n_q_heads // cfg.n_kv_heads
    q, k, v = Q[:, head:head + 1], K[:, head // g:head // g + 1], V[:, head // g:head // g + 1]
    t0 = time.perf_counter()
    S = oracle.estimate(q, k, cfg.segment_size, cfg.block_size, est_scale=cfg.est_scale, alpha=cfg.alpha)
    idx, cnt = oracle.select(S, cfg.segment_size, cfg.block_size, cfg.budget_blocks)
    t1 = time.perf_counter()
    rng = np.random.default_rng(seed)
    rows = np.stack([np.zeros(n_rows, np.int64), np.zeros(n_rows, np.int64),
                     rng.integers(0, cfg.seq_len, n_rows)], axis=1)
    O_rows, _ = oracle.sparse_attention_rows(q, k, v, idx, cnt, cfg.segment_size, cfg.block_size,
                                             1.0 / math.sqrt(cfg.head_dim), rows)
    t2 = time.perf_counter()
    if keep is not None:
        keep.update(S=S, idx=idx, cnt=cnt, rows=rows, O_rows=O_rows)
    return t1 - t0, t2 - t1


def parity_summary(head, ref, S, idx, cnt, O):
    """The timed outputs of the CUDA path against what the oracle sample computed for the same head."""
    S_gpu = S[:, head:head + 1].cpu().numpy()
    fin = np.isfinite(ref["S"])
    same_mask = bool(np.array_equal(np.isfinite(S_gpu), fin))
    idx_gpu, cnt_gpu = idx[:, head:head + 1].cpu().numpy(), cnt[:, head:head + 1].cpu().numpy()
    units = int(np.prod(cnt_gpu.shape))
    equal = np.all(idx_gpu == ref["idx"], axis=-1) & (cnt_gpu == ref["cnt"])
    rows = ref["rows"]
    O_gpu = O[rows[:, 0], head, rows[:, 2]].float().cpu().numpy().astype(np.float64)
    err = np.abs(O_gpu - ref["O_rows"])
    return {"head": head, "ln_S_max_abs_diff": float(np.abs(S_gpu[fin] - ref["S"][fin]).max()) if same_mask else None,
            "mask_equal": same_mask, "selection_units": units, "selection_units_differing": int(units - equal.sum()),
            "attention_rows": int(len(rows)), "attention_max_abs_err": float(err.max()), "attention_mean_abs_err": float(err.mean()),
            "note": "oracle = fp64 CPU restatement of Algorithms 1-2; attention rows use the oracle's lists"}


def oracle_ms_per_layer(cfg, t_est, t_attn, n_rows):
    """Extrapolate the sample to a whole layer pass by unit counts."""
    total_rows = cfg.batch * cfg.n_q_heads * cfg.seq_len
    return 1e3 * (t_est * cfg.n_q_heads * cfg.batch + t_attn * total_rows / n_rows)


def run_reference(args, cfg):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    import oracle.build
    oracle.build.build()
    Q, K, V = make_qkv(cfg)
    n_rows = min(cfg.seq_len, 8192)
    cores = os.cpu_count()
    for i in range(args.warmup):
        oracle_step(cfg, Q, K, V, i % cfg.n_q_heads, n_rows, i)
    ms = []
    for i in range(args.steps):
        te, ta = oracle_step(cfg, Q, K, V, (7 * i + 3) % cfg.n_q_heads, n_rows, 100 + i)
        ms.append(oracle_ms_per_layer(cfg, te, ta, n_rows))
    value = float(np.mean(ms))
    sample = (f"per step: Algorithm 1 + selection for 1 of {cfg.n_q_heads} query heads (all segments) and "
              f"Algorithm 2 for {n_rows} random rows of it; extrapolated to the layer by head and row counts")
    print(json.dumps({
        "impl": "reference", "metric": METRIC, "value": value, "unit": "ms", "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": value, "higher_is_better": False,
        "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": workload_config(cfg),
        "cpu_baseline": {"value": value, "unit": "ms", "cores": cores, "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": "ms", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }))


def workload_config(cfg):
    return {"workload": f"{cfg.name}: 1 layer, batch {cfg.batch}, seq {cfg.seq_len}, {cfg.n_q_heads}Q/{cfg.n_kv_heads}KV "
                        f"heads, head_dim {cfg.head_dim}, {cfg.dtype}, segment {cfg.segment_size}, block {cfg.block_size}, "
                        f"budget {cfg.budget_tokens} tokens, est_scale {cfg.est_scale}, "
                        + (f"{cfg.layers}-layer stack with layer fusion alpha {cfg.alpha}" if cfg.layers > 1 else "no layer fusion (first layer)"),
            "inputs": "seeded clustered-key / AR(1)-query generator", "l2": "inputs larger than L2 (Q alone "
            f"{cfg.batch * cfg.n_q_heads * cfg.seq_len * cfg.head_dim * 2 / 1e6:.0f} MB vs 126 MB); no explicit flush"}


# ----------------------------------------------------------------------------- our arm
def spawn_ranks(n: int) -> int:
    """Start `n` ranks of this script on this node (one per GPU) and wait for them; rank 0 prints the JSON line."""
    import socket
    import subprocess
    with socket.socket() as sk:
        sk.bind(("127.0.0.1", 0))
        port = sk.getsockname()[1]
    env = dict(os.environ)
    env.setdefault("NCCL_DEBUG", "INFO")                     # the communicator log (transports, NVLS) is kept, in a file:
    env.setdefault("NCCL_DEBUG_FILE", os.path.join("/tmp", "critiprefill_nccl_%h_%p.log"))   # stdout carries one JSON line only
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", f"--nproc-per-node={n}", "--master-addr", "127.0.0.1",
           "--master-port", str(port), os.path.abspath(__file__)] + sys.argv[1:]
    return subprocess.call(cmd, env=env)


def run_ours(args, cfg):
    info = RankInfo.from_env()
    rank, world, local = info.rank, info.world, info.local_rank
    if world != args.gpus:
        raise SystemExit(f"--gpus {args.gpus} but the launcher started {world} rank(s): start bench.py either plainly "
                         f"(it spawns its own ranks) or under torchrun with --nproc-per-node {args.gpus}")
    dist = None
    if world > 1:
        import torch.distributed as dist
        os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the hot path has no CPU fallback")
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)

    from paper_2409_12490_b200 import binding as cp
    from paper_2409_12490_b200.build import build
    if rank == 0:
        build()
    if dist is not None:
        dist.barrier()
    cp.load_library()

    # --shard replicas: every rank works on its own batch item (same shape, its own seed): weak scaling.
    # --shard heads: ONE problem; rank p owns the KV heads head_shard(Hkv, p, N) and their g query heads and runs
    # the library on strided views of the full tensors (every (batch, head) is independent in Algorithms 1 and 2):
    # strong scaling.  Neither mode has a collective on the data path.
    # A stack of L layers cycles through D distinct seeded layer inputs; the criticality scores are
    # carried from layer to layer (Algorithm 1, line 14) through two ping-pong buffers.
    by_heads = args.shard == "heads" and world > 1
    full_cfg = cfg
    shard = shard_heads(cfg, rank, world) if by_heads else None
    if by_heads:
        cfg = shard.cfg
    L = args.layers if args.layers else cfg.layers
    D = min(L, args.distinct_layers)
    layers_in = []
    for li in range(D):
        if by_heads:
            qf, kf, vf = (t.to(dev) for t in make_qkv(full_cfg, layer=li))               # the same full problem on every rank
            q, k, v = shard.slice_q(qf), shard.slice_kv(kf), shard.slice_kv(vf)         # views: strides of the full tensors
            layers_in.append((q, k, v))
            if li == 0:
                Q, K, V = q.cpu().contiguous(), k.cpu().contiguous(), v.cpu().contiguous()
            continue
        q, k, v = make_qkv(cfg, layer=layer_seed_for_rank(li, rank, D))
        if li == 0:
            Q, K, V = q, k, v
        layers_in.append(tuple(t.to(dev) for t in (q, k, v)))
    hQ, hK, hV = Q.pin_memory(), K.pin_memory(), V.pin_memory()
    dQ, dK, dV = layers_in[0]
    prob = cp.Problem.from_config(cfg)
    ws = cp.alloc_workspace(prob, dev)
    S = torch.empty((cfg.batch, cfg.n_q_heads, cfg.n1, cfg.n2), dtype=torch.float64, device=dev)
    S2 = torch.empty_like(S) if L > 1 else None
    idx = torch.empty((cfg.batch, cfg.n_q_heads, cfg.n1, cfg.budget_blocks), dtype=torch.int32, device=dev)
    cnt = torch.empty((cfg.batch, cfg.n_q_heads, cfg.n1), dtype=torch.int32, device=dev)
    O = torch.empty(dQ.shape, dtype=dQ.dtype, device=dev)
    hO = torch.empty_like(hQ).pin_memory()
    torch.cuda.synchronize()

    def step(ev=None):
        """One pass of the whole path over the stack (L = 1: one layer)."""
        if L == 1:
            if ev is not None:
                ev[0].record()
            cp.estimate(prob, dQ, dK, ws, S_out=S)
            if ev is not None:
                ev[1].record()
            cp.select(prob, S, ws, idx=idx, cnt=cnt)
            if ev is not None:
                ev[2].record()
            cp.attention(prob, dQ, dK, dV, idx, cnt, ws, O=O)
            if ev is not None:
                ev[3].record()
            return
        if ev is not None:
            ev[0].record()
        prev, cur = None, S
        for li in range(L):
            q, k, v = layers_in[li % D]
            cp.estimate(prob, q, k, ws, S_prev=prev, S_out=cur)
            cp.select(prob, cur, ws, idx=idx, cnt=cnt)
            cp.attention(prob, q, k, v, idx, cnt, ws, O=O)
            prev, cur = cur, (S2 if cur is S else S)
        if ev is not None:
            ev[1].record(); ev[2].record(); ev[3].record()

    def barrier():
        torch.cuda.synchronize()
        if dist is not None:
            dist.barrier()
            torch.cuda.synchronize()

    for _ in range(max(args.warmup, 3)):
        step()
    barrier()
    evs = [[torch.cuda.Event(enable_timing=True) for _ in range(4)] for _ in range(args.steps)]
    start, end = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    with ClockSampler(physical_gpu_index(local)) as clocks:
        barrier()
        start.record()
        for i in range(args.steps):
            step(evs[i])
        end.record()
        barrier()
    total_ms = start.elapsed_time(end)
    status = cp.device_status(ws)
    if status != 0:
        raise SystemExit(f"device status {status}: {cp.status_string(status)}")
    est_ms = float(np.mean([e[0].elapsed_time(e[1]) for e in evs]))
    sel_ms = float(np.mean([e[1].elapsed_time(e[2]) for e in evs]))
    att_ms = float(np.mean([e[2].elapsed_time(e[3]) for e in evs]))
    total_ms, est_ms, sel_ms, att_ms = max_over_ranks([total_ms, est_ms, sel_ms, att_ms], dist, dev)
    agg = aggregate_time_metric(total_ms / args.steps / L, world, replicas=not by_heads)      # per layer pass
    ms_per_step = agg["ms_per_step"]

    # dense baseline of the same library (the denominator of the speed-up)
    dense_ms = None
    if not args.no_dense:
        Od = torch.empty(dQ.shape, dtype=dQ.dtype, device=dev)
        cp.dense_attention(prob, dQ, dK, dV, ws, O=Od)
        torch.cuda.synchronize()
        d0, d1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        reps = 2
        d0.record()
        for _ in range(reps):
            cp.dense_attention(prob, dQ, dK, dV, ws, O=Od)
        d1.record()
        torch.cuda.synchronize()
        dense_ms = d0.elapsed_time(d1) / reps
        del Od

    # end to end through the public API with host buffers: H2D of Q,K,V, the path, D2H of O
    e2e_steps = max(2, min(5, args.steps))
    h2d = (hQ.numel() + hK.numel() + hV.numel()) * hQ.element_size()
    d2h = hO.numel() * hO.element_size()

    from paper_2409_12490_b200.pipeline import HostPipelinedLayer
    host_layer = HostPipelinedLayer(prob, dev) if cfg.batch == 1 else None

    def e2e_step():
        """Host buffers in, host buffer out, one layer through the public API (per-KV-group pipeline
        over copy-in / compute / copy-out streams; a plain copy-compute-copy sequence for batch > 1)."""
        if host_layer is not None:
            host_layer(hQ, hK, hV, hO)
            return
        dQ.copy_(hQ, non_blocking=True); dK.copy_(hK, non_blocking=True); dV.copy_(hV, non_blocking=True)
        cp.estimate(prob, dQ, dK, ws, S_out=S)
        cp.select(prob, S, ws, idx=idx, cnt=cnt)
        cp.attention(prob, dQ, dK, dV, idx, cnt, ws, O=O)
        hO.copy_(O, non_blocking=True)

    e2e_step()
    barrier()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(e2e_steps):
        e2e_step()
    e1.record()
    barrier()
    e2e_ms = e0.elapsed_time(e1) / e2e_steps
    (e2e_ms,) = max_over_ranks([e2e_ms], dist, dev)
    if host_layer is not None and host_layer.status() != 0:
        raise SystemExit("device status set in the end-to-end run")
    e2e_same = bool(torch.equal(hO.to(dev), O)) if L == 1 else None      # the pipelined result equals the resident one

    if rank != 0:
        if dist is not None:
            dist.destroy_process_group()
        return

    peaks = load_peaks()
    fl = flop_counts(cfg)
    if L > 1:   # the stack run has no per-kernel events: time the attention kernel alone
        a0, a1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a0.record()
        for _ in range(5):
            cp.attention(prob, dQ, dK, dV, idx, cnt, ws, O=O)
        a1.record()
        torch.cuda.synchronize()
        att_ms, est_ms, sel_ms = a0.elapsed_time(a1) / 5, None, None
    achieved = fl["executed"] / (att_ms * 1e-3) / 1e12
    ncu = load_ncu_counters().get(cfg.name, {})
    roofline = {"bound": "tensor", "kernel": "attention_sm100_kernel (critiprefill_attention)",
                "achieved": achieved, "peak": peaks["bf16_tflops"], "unit": "TFLOP/s",
                "frac": achieved / peaks["bf16_tflops"], "peak_source": f"{peaks['source']} (burst)",
                "frac_of_sustained": achieved / peaks["bf16_tflops_sustained"] if peaks["bf16_tflops_sustained"] else None,
                "flops_per_launch": fl["executed"], "traffic": ncu.get("dram_bytes_per_launch"),
                "tensor_pipe_active_pct_ncu": ncu.get("tensor_pipe_active_pct"),
                "ncu_capture": {k: ncu.get(k) for k in ("commit", "captured", "command")} if ncu else None,
                "traffic_unit": "bytes per launch (dram__bytes_read.sum + dram__bytes_write.sum, from the ncu capture named in "
                                "ncu_capture; not measured in this run)"}
    summary_bytes = (dQ.numel() + dK.numel()) * dQ.element_size()
    out = {
        "metric": METRIC, "value": ms_per_step, "unit": "ms", "n_gpus": world, "steps": args.steps,
        "warmup": max(args.warmup, 3), "ms_per_step": ms_per_step, "higher_is_better": False,
        "scaling": "strong" if by_heads else "weak",
        "sharding": ("heads: one layer, each rank owns Hkv/N KV heads and their query heads (no collective on the path)" if by_heads
                     else "replicas: one layer per rank (no collective on the path)") if world > 1 else "single GPU",
        "vs_baseline": None, "dtype": cfg.dtype, "data": "synthetic",
        "config": workload_config(full_cfg),
        "breakdown_ms": {"estimate": est_ms, "select": sel_ms, "attention": att_ms},
        "dense_ms": dense_ms,
        "speedup_vs_dense": (dense_ms / ms_per_step) if dense_ms else None,
        "dense_equiv_tflops": flop_counts(full_cfg)["dense"] * (1 if by_heads else world) / (ms_per_step * 1e-3) / 1e12,
        "dense_kernel_tflops": (fl["dense"] / (dense_ms * 1e-3) / 1e12) if dense_ms else None,
        "estimate_gbs": (summary_bytes / (est_ms * 1e-3) / 1e9) if est_ms else None,
        "layer_passes_per_s": agg["layer_passes_per_s"],
        "layers": L, "distinct_layer_inputs": D, "stack_ms": ms_per_step * L,
        "paper_context": "paper: 2.7x (Llama3-8B) / 3.0x (Yi-9B) end-to-end prefill speed-up at 128K on one A100, fp16",
        "roofline": roofline,
        "e2e": {"value": e2e_ms, "unit": "ms", "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h,
                "how": "pinned host Q,K,V -> device, estimate+select+attention, O -> pinned host; pipelined per KV group "
                       "over three streams" if host_layer is not None else "copy in, compute, copy out",
                "matches_resident_output": e2e_same},
        # kernels of this library launched inside the timed region: per layer pass summarize, the score step (one general
        # kernel, or the log-sum-exp + visible-score pair for 16-bit inputs with head_dim 128), select, attention
        "gpu_launches": (5 if (cfg.dtype in ("bf16", "f16") and cfg.head_dim == 128) else 4) * args.steps * L,
        "clocks": clocks.summary(),
    }
    if world == 1 and not args.no_cpu_baseline:
        import oracle.build
        oracle.build.build()
        n_rows = min(4 * cfg.seq_len, 262144)      # about 10 s of oracle work on 16 cores at C4
        ref = {} if L == 1 else None
        te, ta = oracle_step(cfg, Q, K, V, 5 % cfg.n_q_heads, n_rows, 0, keep=ref)
        if ref is not None:
            out["parity"] = parity_summary(5 % cfg.n_q_heads, ref, S, idx, cnt, O)
        out["cpu_baseline"] = {
            "value": oracle_ms_per_layer(cfg, te, ta, n_rows), "unit": "ms", "cores": os.cpu_count(), "kind": "oracle",
            "sample": f"Algorithm 1 + selection for 1 of {cfg.n_q_heads} query heads ({te:.1f} s, numpy) and Algorithm 2 "
                      f"for {n_rows} random rows ({ta:.1f} s, C/OpenMP); extrapolated to the layer by head and row counts"}
    print(json.dumps(out))
    if dist is not None:
        dist.destroy_process_group()


def run_sweep(args, cfg):
    """Accuracy-vs-speed trace: budget x block size, each against the dense kernel.  Mass recall is
    exp(lse_sparse - lse_dense), the share of a row's dense softmax mass that its listed keys hold."""
    from paper_2409_12490_b200 import binding as cp
    from paper_2409_12490_b200.build import build
    build()
    dev = torch.device("cuda", 0)
    torch.cuda.set_device(dev)
    Q, K, V = (t.to(dev) for t in make_qkv(cfg))
    rows = []
    dense = None
    for blk in (32, 64, 128):
        for budget in (1024, 2048, 4096, 8192):
            c = cfg.with_(block_size=blk, budget_tokens=budget)
            prob = cp.Problem.from_config(c)
            ws = cp.alloc_workspace(prob, dev)
            if dense is None:
                Od, lsed = cp.dense_attention(prob, Q, K, V, ws, want_lse=True)
                torch.cuda.synchronize()
                d0, d1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                d0.record()
                cp.dense_attention(prob, Q, K, V, ws, O=Od, lse=lsed)
                d1.record()
                torch.cuda.synchronize()
                dense = d0.elapsed_time(d1)
            for _ in range(3):
                O, S, idx, cnt = cp.prefill_layer(prob, Q, K, V, ws)
            e = [torch.cuda.Event(enable_timing=True) for _ in range(2)]
            reps = 5
            e[0].record()
            for _ in range(reps):
                S = cp.estimate(prob, Q, K, ws, S_out=S)
                cp.select(prob, S, ws, idx=idx, cnt=cnt)
                cp.attention(prob, Q, K, V, idx, cnt, ws, O=O)
            e[1].record()
            torch.cuda.synchronize()
            ms = e[0].elapsed_time(e[1]) / reps
            _, lse = cp.attention(prob, Q, K, V, idx, cnt, ws, O=O, want_lse=True)
            assert cp.device_status(ws) == 0
            recall = torch.exp(lse.double() - lsed.double())
            diff = (O.float() - Od.float()).abs()
            rows.append({"block": blk, "budget_tokens": budget, "ms": ms, "speedup_vs_dense": dense / ms,
                         "mass_recall_mean": recall.mean().item(), "mass_recall_median": recall.median().item(),
                         "mass_recall_p05": recall.flatten().kthvalue(max(1, recall.numel() // 20)).values.item(),
                         "out_vs_dense_max": diff.max().item(), "out_vs_dense_mean": diff.mean().item()})
    print(json.dumps({"sweep": rows, "dense_ms": dense, "config": workload_config(cfg), "data": "synthetic"}))


def run_fusion_ablation(args, cfg):
    """Layer fusion on / off (Algorithm 1, line 14; the "w/o fusion" row of the paper's ablation is alpha = 1)
    on a stack of seeded layers that share their cluster structure: per layer and per setting, the share of
    each row's dense softmax mass that the selected blocks hold, and the distance to the dense output."""
    from paper_2409_12490_b200 import binding as cp
    from paper_2409_12490_b200.build import build
    build()
    dev = torch.device("cuda", 0)
    torch.cuda.set_device(dev)
    L = args.layers if args.layers else 4
    variants = [("fusion", cfg), ("no_fusion", cfg.with_(alpha=1.0))]
    probs = {name: cp.Problem.from_config(c) for name, c in variants}
    ws = cp.alloc_workspace(probs["fusion"], dev)
    prev = {name: None for name, _ in variants}
    rows = []
    for li in range(L):
        Q, K, V = (t.to(dev) for t in make_qkv(cfg, layer=li))
        Od, lsed = cp.dense_attention(probs["fusion"], Q, K, V, ws, want_lse=True)
        for name, _ in variants:
            S = cp.estimate(probs[name], Q, K, ws, S_prev=prev[name])
            idx, cnt = cp.select(probs[name], S, ws)
            O, lse = cp.attention(probs[name], Q, K, V, idx, cnt, ws, want_lse=True)
            assert cp.device_status(ws) == 0
            recall = torch.exp(lse.double() - lsed.double())
            diff = (O.float() - Od.float()).abs()
            rows.append({"layer": li, "setting": name, "alpha": probs[name].alpha, "mass_recall_mean": recall.mean().item(),
                         "mass_recall_median": recall.median().item(),
                         "mass_recall_p05": recall.flatten().kthvalue(max(1, recall.numel() // 20)).values.item(),
                         "out_vs_dense_max": diff.max().item(), "out_vs_dense_mean": diff.mean().item()})
            prev[name] = S
            del O, lse, idx, cnt, recall, diff
        del Q, K, V, Od, lsed
    print(json.dumps({"fusion_ablation": rows, "layers": L, "config": workload_config(cfg), "data": "synthetic"}))


def run_overlap(args, cfg):
    """Token-wise critical sets (Eq. 3) and how much neighbouring queries share of them (the locality the
    paper's Section 2 builds on), over the whole sequence.  index_i = argtop_k(softmax(q_i K^T), k = 512): the
    softmax is monotone per row, so the set is the top-k of the logits q_i . k_u over the keys u <= i.  The logits
    are formed tile by tile over key ranges (a query chunk against every key chunk, torch matmul) and reduced with
    a running top-k, so no n x n matrix exists; |I_i & I_(i+delta)| / k is then counted from sorted index lists.
    A workload diagnostic outside the hot path (no library kernel is involved); two query heads."""
    dev = torch.device("cuda", 0)
    torch.cuda.set_device(dev)
    n, k = cfg.seq_len, 512
    Q, K, _ = make_qkv(cfg)
    g = cfg.n_q_heads // cfg.n_kv_heads
    rows = []
    qc, kc = 4096, 16384
    for h in (0, g):                                           # two query heads of different KV groups
        Qh = Q[0, h].to(dev).float()
        Kh = K[0, h // g].to(dev).float()
        top = torch.empty((n, k), dtype=torch.int32, device=dev)
        for q0 in range(0, n, qc):
            q1 = min(n, q0 + qc)
            best_v = torch.full((q1 - q0, k), float("-inf"), device=dev)
            best_i = torch.zeros((q1 - q0, k), dtype=torch.int64, device=dev)
            for k0 in range(0, q1, kc):                        # keys after the chunk's last query are never visible
                k1 = min(q1, k0 + kc)
                lg = Qh[q0:q1] @ Kh[k0:k1].T
                ui = torch.arange(k0, k1, device=dev)[None, :]
                lg.masked_fill_(ui > torch.arange(q0, q1, device=dev)[:, None], float("-inf"))
                v = torch.cat([best_v, lg], dim=1)
                i = torch.cat([best_i, ui.expand(q1 - q0, -1)], dim=1)
                best_v, pos = v.topk(k, dim=1)
                best_i = i.gather(1, pos)
            top[q0:q1] = best_i.sort(dim=1).values.int()
        for delta in (1, 8, 64, 512, 2048, 16384):
            a_, b_ = top[k:n - delta].long(), top[k + delta:n].long()          # rows whose lists are full
            share = torch.empty(a_.shape[0], dtype=torch.float64, device=dev)
            for c0 in range(0, a_.shape[0], 8192):                             # |A & B| through a sorted merge per row
                A, Bm = a_[c0:c0 + 8192], b_[c0:c0 + 8192]
                posn = torch.searchsorted(Bm, A)
                hit = Bm.gather(1, posn.clamp(max=k - 1)) == A
                share[c0:c0 + 8192] = hit.sum(1).double() / k
            rows.append({"head": h, "delta": delta, "overlap_mean": share.mean().item(), "overlap_median": share.median().item(),
                         "overlap_p05": share.kthvalue(max(1, share.numel() // 20)).values.item()})
        del top
    print(json.dumps({"token_critical_set_overlap": rows, "k": k, "tokens": n, "config": workload_config(cfg), "data": "synthetic"}))


def run_projection(args, cfg):
    """Upstream fusion (Eq. 1): the query / key projection kernel whose epilogue leaves the representatives of
    Algorithm 1 in the workspace, timed beside the estimate with and without its own pass over Q and K.
    Seeded random X and weights of the Llama3-8B width (d_model 4096); a kernel measurement, not the bench line."""
    from paper_2409_12490_b200 import binding as cp
    from paper_2409_12490_b200.build import build
    build()
    dev = torch.device("cuda", 0)
    torch.cuda.set_device(dev)
    d_model = args.d_model
    g = torch.Generator(device=dev).manual_seed(20240912)
    tdt = {"bf16": torch.bfloat16, "f16": torch.float16}[cfg.dtype]
    X = torch.randn((cfg.batch, cfg.seq_len, d_model), generator=g, device=dev, dtype=torch.float32).to(tdt)
    Wq = (torch.randn((cfg.n_q_heads * cfg.head_dim, d_model), generator=g, device=dev) / math.sqrt(d_model)).to(tdt)
    Wk = (torch.randn((cfg.n_kv_heads * cfg.head_dim, d_model), generator=g, device=dev) / math.sqrt(d_model)).to(tdt)
    inv = 500000.0 ** (-torch.arange(0, cfg.head_dim, 2, device=dev, dtype=torch.float64) / cfg.head_dim)
    ang = torch.arange(cfg.seq_len, device=dev, dtype=torch.float64)[:, None] * inv[None, :]
    cos, sin = torch.cos(ang).float().contiguous(), torch.sin(ang).float().contiguous()
    prob = cp.Problem.from_config(cfg)
    ready = cp.Problem.from_config(cfg, flags=cp.FLAG_SUMMARIES_READY)
    ws = cp.alloc_workspace(prob, dev)
    Q, K = cp.project_qk(prob, X, Wq, Wk, ws, rope_cos=cos, rope_sin=sin)
    S = cp.estimate(ready, Q, K, ws)
    S2 = cp.estimate(prob, Q, K, ws)
    same = bool(torch.equal(S, S2))
    torch.cuda.synchronize()
    ev = [torch.cuda.Event(enable_timing=True) for _ in range(4)]
    reps = max(3, min(args.steps, 10))
    ev[0].record()
    for _ in range(reps):
        cp.project_qk(prob, X, Wq, Wk, ws, rope_cos=cos, rope_sin=sin, Q_out=Q, K_out=K)
    ev[1].record()
    for _ in range(reps):
        cp.estimate(ready, Q, K, ws, S_out=S)
    ev[2].record()
    for _ in range(reps):
        cp.estimate(prob, Q, K, ws, S_out=S)
    ev[3].record()
    torch.cuda.synchronize()
    assert cp.device_status(ws) == 0
    proj_ms, est_ready_ms, est_plain_ms = (ev[i].elapsed_time(ev[i + 1]) / reps for i in range(3))
    # the same launch with the value projection of Eq. 1 added
    Wv = (torch.randn((cfg.n_kv_heads * cfg.head_dim, d_model), generator=g, device=dev) / math.sqrt(d_model)).to(tdt)
    _, _, V = cp.project_qkv(prob, X, Wq, Wk, Wv, ws, rope_cos=cos, rope_sin=sin, Q_out=Q, K_out=K)
    torch.cuda.synchronize()
    ev[0].record()
    for _ in range(reps):
        cp.project_qkv(prob, X, Wq, Wk, Wv, ws, rope_cos=cos, rope_sin=sin, Q_out=Q, K_out=K, V_out=V)
    ev[1].record()
    torch.cuda.synchronize()
    qkv_ms = ev[0].elapsed_time(ev[1]) / reps
    flops_qkv = 2.0 * cfg.batch * cfg.seq_len * d_model * (cfg.n_q_heads + 2 * cfg.n_kv_heads) * cfg.head_dim
    flops = 2.0 * cfg.batch * cfg.seq_len * d_model * (cfg.n_q_heads + cfg.n_kv_heads) * cfg.head_dim
    peaks = load_peaks()
    print(json.dumps({"projection_ms": proj_ms, "gemm_tflops": flops / (proj_ms * 1e-3) / 1e12,
                      "frac_of_bf16_peak": flops / (proj_ms * 1e-3) / 1e12 / peaks["bf16_tflops"], "peak_source": peaks["source"],
                      "projection_qkv_ms": qkv_ms, "qkv_gemm_tflops": flops_qkv / (qkv_ms * 1e-3) / 1e12,
                      "qkv_frac_of_bf16_peak": flops_qkv / (qkv_ms * 1e-3) / 1e12 / peaks["bf16_tflops"],
                      "estimate_ms_summaries_ready": est_ready_ms, "estimate_ms_with_own_pass": est_plain_ms,
                      "scores_identical": same, "d_model": d_model, "config": workload_config(cfg), "data": "synthetic"}))


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--config", default="C4", choices=sorted(CONFIGS))
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--layers", type=int, default=0, help="layers in the stack (default: the config's)")
    ap.add_argument("--distinct-layers", type=int, default=2, help="distinct seeded layer inputs cycled through a stack")
    ap.add_argument("--sweep", action="store_true", help="budget x block-size sweep (accuracy vs speed) instead of the bench line")
    ap.add_argument("--fusion-ablation", action="store_true",
                    help="layer fusion on/off over a stack of --layers seeded layers (quality diagnostic) instead of the bench line")
    ap.add_argument("--overlap", action="store_true",
                    help="token-wise critical-set overlap between neighbouring queries (Eq. 3; quality diagnostic) instead of the bench line")
    ap.add_argument("--shard", default="replicas", choices=["replicas", "heads"],
                    help="with --gpus N > 1: N independent layers (weak scaling) or one layer split by KV head group (strong scaling)")
    ap.add_argument("--projection", action="store_true",
                    help="time the fused query/key projection (Eq. 1) and the estimate that uses its summaries, instead of the bench line")
    ap.add_argument("--d-model", type=int, default=4096)
    ap.add_argument("--no-dense", action="store_true")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    args = ap.parse_args()
    cfg = CONFIGS[args.config]
    if args.impl == "ours" and args.gpus > 1 and "RANK" not in os.environ:
        raise SystemExit(spawn_ranks(args.gpus))
    if args.impl == "reference":
        run_reference(args, cfg)
    elif args.sweep:
        run_sweep(args, cfg)
    elif args.fusion_ablation:
        run_fusion_ablation(args, cfg)
    elif args.overlap:
        run_overlap(args, cfg)
    elif args.projection:
        run_projection(args, cfg)
    else:
        run_ours(args, cfg)


if __name__ == "__main__":
    main()
