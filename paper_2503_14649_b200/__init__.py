"""B200-native IVF-PQ / flat retrieval hot path (RAG retrieval stage).

The package holds the CUDA kernels and C-ABI library (`csrc/`), the thin
ctypes binding (`binding.py`) and the seeded synthetic-input generators
(`synth.py`).  Importing the package loads nothing; the shared library is
opened on first use of the binding and a missing library is an error, never a
fallback.
"""

__all__ = ["binding", "sharded", "synth"]
