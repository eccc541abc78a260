"""METok hot path on B200: event segmentation, per-event key-token top-k with
similarity merging, prefill text->visual attention pruning with hidden-state
compaction, and KV-cache selection with in-place gather.

Everything that computes lives in the CUDA library under ``csrc/`` behind a
C ABI (``include/metok.h``).  ``binding`` marshals torch tensors into that ABI;
``workloads`` builds the seeded synthetic inputs.  Importing this package does
not load the library; the first call that needs it does, and raises if it is
missing.
"""

__all__ = ["binding", "workloads", "build"]
