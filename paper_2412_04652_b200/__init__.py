"""B200 (sm_100a) library for the scoring-and-compaction pass of Cross-Self Pruning.

`paper_2412_04652_b200.binding` mirrors the C interface in include/csp.h;
`paper_2412_04652_b200.build` compiles libcsp.so in-tree.
"""
from . import binding  # noqa: F401

__all__ = ["binding"]
