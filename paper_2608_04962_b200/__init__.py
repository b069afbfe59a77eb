"""SpecRoll per-step speculative hot path for NVIDIA B200 (sm_100a).

``binding`` exposes the C-ABI entry points of ``libspecroll.so`` (proposal, tree attention,
exact verification); ``inputs`` holds the seeded synthetic workloads; ``build`` compiles the
library in-tree.  There is no fallback path: without the built library every call raises.
"""
from . import inputs  # noqa: F401  (numpy only)

__all__ = ["inputs", "binding", "build"]
