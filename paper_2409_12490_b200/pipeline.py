"""Host-buffer front end: one layer of the path with Q/K/V in pinned host memory and O returned
to pinned host memory, pipelined per KV group over three CUDA streams.

Every (batch, KV group) is independent in Algorithm 1 and Algorithm 2, so the layer is cut into
Hkv sub-problems (g query heads + 1 KV head each).  Group i's host->device copy, the kernels of
group i-1 and the device->host copies of earlier outputs run concurrently; PCIe is full duplex,
so the layer costs about max(bytes in, bytes out) / link rate instead of their sum plus compute.
Within a group the attention runs head by head and each head's output is copied back as soon as
it is complete, which shortens the tail after the last input has arrived.
All arithmetic still runs in the CUDA library (critiprefill_estimate / _select / _attention on
strided views); this module only moves data and orders streams.
"""
from __future__ import annotations

import torch

from . import binding as cp


class HostPipelinedLayer:
    def __init__(self, prob: cp.Problem, device="cuda"):
        if prob.batch != 1:
            raise ValueError("the host pipeline cuts the layer by KV group and expects batch 1")
        self.prob = prob
        self.dev = torch.device(device)
        g = prob.n_q_heads // prob.n_kv_heads
        self.g = g
        self.sub = cp.Problem(1, g, 1, prob.seq_len, prob.head_dim, prob.segment_size, prob.block_size,
                              prob.budget_blocks, prob.dtype, prob.est_scale, prob.sm_scale, prob.alpha, prob.flags, prob.n_sink, prob.n_local)
        n, d = prob.seq_len, prob.head_dim
        self.dQ = torch.empty((1, prob.n_q_heads, n, d), dtype=prob.dtype, device=self.dev)
        self.dK = torch.empty((1, prob.n_kv_heads, n, d), dtype=prob.dtype, device=self.dev)
        self.dV = torch.empty_like(self.dK)
        self.dO = torch.empty_like(self.dQ)
        self.ws = cp.alloc_workspace(self.sub, self.dev)
        self.S = torch.empty((1, g, self.sub.n1, self.sub.n2), dtype=torch.float64, device=self.dev)
        self.idx = torch.empty((1, g, self.sub.n1, prob.budget_blocks), dtype=torch.int32, device=self.dev)
        self.cnt = torch.empty((1, g, self.sub.n1), dtype=torch.int32, device=self.dev)
        self.head = cp.Problem(1, 1, 1, prob.seq_len, prob.head_dim, prob.segment_size, prob.block_size,
                               prob.budget_blocks, prob.dtype, prob.est_scale, prob.sm_scale, prob.alpha, prob.flags, prob.n_sink, prob.n_local)
        self.s_in, self.s_run, self.s_out = (torch.cuda.Stream(self.dev) for _ in range(3))
        self.ev_in = [torch.cuda.Event() for _ in range(prob.n_kv_heads)]
        self.ev_run = [torch.cuda.Event() for _ in range(prob.n_q_heads)]

    def __call__(self, hQ, hK, hV, hO):
        """hQ/hO [1,Hq,n,d], hK/hV [1,Hkv,n,d] pinned host tensors.  Enqueues the whole layer and makes
        the caller's current stream wait for the last output copy; returns hO."""
        cur = torch.cuda.current_stream(self.dev)
        for s in (self.s_in, self.s_run, self.s_out):
            s.wait_stream(cur)
        g = self.g
        for i in range(self.prob.n_kv_heads):
            q = slice(i * g, (i + 1) * g)
            with torch.cuda.stream(self.s_in):
                self.dQ[:, q].copy_(hQ[:, q], non_blocking=True)
                self.dK[:, i:i + 1].copy_(hK[:, i:i + 1], non_blocking=True)
                self.dV[:, i:i + 1].copy_(hV[:, i:i + 1], non_blocking=True)
                self.ev_in[i].record(self.s_in)
            with torch.cuda.stream(self.s_run):
                self.s_run.wait_event(self.ev_in[i])
                Q, K, V, O = self.dQ[:, q], self.dK[:, i:i + 1], self.dV[:, i:i + 1], self.dO[:, q]
                cp.estimate(self.sub, Q, K, self.ws, S_out=self.S)
                cp.select(self.sub, self.S, self.ws, idx=self.idx, cnt=self.cnt)
                for h in range(g):
                    one = slice(h, h + 1)
                    cp.attention(self.head, Q[:, one], K, V, self.idx[:, one], self.cnt[:, one], self.ws, O=O[:, one])
                    self.ev_run[i * g + h].record(self.s_run)
            with torch.cuda.stream(self.s_out):
                for h in range(g):
                    self.s_out.wait_event(self.ev_run[i * g + h])
                    hO[:, i * g + h:i * g + h + 1].copy_(self.dO[:, i * g + h:i * g + h + 1], non_blocking=True)
        cur.wait_stream(self.s_out)
        cur.wait_stream(self.s_run)
        return hO

    def status(self) -> int:
        return cp.device_status(self.ws)
