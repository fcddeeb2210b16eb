"""B200-native CritiPrefill prefill hot path (segment-wise criticality estimation,
top-k block selection, block-sparse causal GQA attention, dense causal baseline).

The compute lives in the CUDA C-ABI library under ``csrc/``; ``binding`` marshals
arguments to it and ``inputs`` holds the seeded synthetic workload generator.
Nothing here imports the CPU oracle.
"""

from .configs import CONFIGS, Config  # noqa: F401
