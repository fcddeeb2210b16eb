"""fp64 CPU oracle for the CritiPrefill prefill hot path.

TEST INFRASTRUCTURE ONLY: imported by tests/, by __graft_entry__.smoke() and by
bench.py's CPU-baseline legs.  The CUDA product path never imports it, and it
imports nothing from the CUDA package.
"""
from .estimation import summaries, logits, estimate, causal_block_mask, decode_estimate  # noqa: F401
from .selection import select, pool_group_scores, decode_select  # noqa: F401
from .attention import sparse_attention, dense_attention, sparse_attention_rows, dense_attention_rows  # noqa: F401
from .projection import project_qk, project_v, rope, rope_tables  # noqa: F401
from .varlen import prefill_varlen, sequence_bounds  # noqa: F401
