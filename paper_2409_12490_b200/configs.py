"""Named workload shapes (attention shapes only; no weights, no datasets).

C1..C5 follow the five benchmark configurations: a tiny fp32 case, Llama3-8B-shaped
single layers at 8K / 32K / 128K tokens and a Yi-9B-shaped 48-layer stack at 128K.
The paper's own operating point (Section 3.1.3: segment 512, block 32, budget 1024,
alpha 0.25) is available as ``paper_128k``.
"""
from __future__ import annotations

from dataclasses import dataclass, replace


@dataclass(frozen=True)
class Config:
    name: str
    index: int            # enters the RNG seed
    batch: int
    n_q_heads: int
    n_kv_heads: int
    seq_len: int
    head_dim: int
    dtype: str            # "bf16" | "f16" | "f32"
    segment_size: int
    block_size: int
    budget_tokens: int
    n_clusters: int
    rho: float
    layers: int = 1
    alpha: float = 0.25   # Section 3.1.3
    est_scale: float = 1.0

    @property
    def n1(self) -> int:
        return -(-self.seq_len // self.segment_size)

    @property
    def n2(self) -> int:
        return -(-self.seq_len // self.block_size)

    @property
    def r(self) -> int:
        """Blocks overlapping one segment (the diagonal blocks)."""
        return self.segment_size // self.block_size

    @property
    def budget_blocks(self) -> int:
        return self.budget_tokens // self.block_size

    def with_(self, **kw) -> "Config":
        return replace(self, **kw)


CONFIGS = {
    "C1": Config("C1", 1, 1, 4, 2, 1024, 64, "f32", 128, 32, 8 * 32, 8, 0.95),
    "C2": Config("C2", 2, 1, 32, 8, 8192, 128, "bf16", 512, 64, 1024, 64, 0.95),
    "C3": Config("C3", 3, 1, 32, 8, 32768, 128, "bf16", 512, 64, 2048, 64, 0.95),
    "C4": Config("C4", 4, 1, 32, 8, 131072, 128, "bf16", 1024, 128, 4096, 256, 0.98),
    "C5": Config("C5", 5, 1, 32, 4, 131072, 128, "bf16", 1024, 128, 4096, 256, 0.98, layers=48),
    "paper_128k": Config("paper_128k", 6, 1, 32, 8, 131072, 128, "bf16", 512, 32, 1024, 256, 0.98),
}
