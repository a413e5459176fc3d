"""B200-native sparse-attention hot path (indexer, top-p selection, sparse / local / dense attention).

Importing the package is cheap; the CUDA library is loaded on first use by
``paper_2605_16928_b200.binding`` and every entry point fails loudly when it is
missing.  ``synth`` holds the seeded workload generators (numpy only).
"""
__all__ = ["binding", "synth"]
