"""Flexible Context Parallelism hot path on B200: varlen causal attention forward/backward over a
packed batch, decomposed per sequence by a context-parallel block plan, plus the exact LSE merge.

The compute lives in ``libfcp.so`` (C ABI, hand-written sm_100a kernels).  ``fcp`` is the thin
ctypes binding.  Importing this package does not load the library; ``fcp.lib()`` does, and raises
if it is missing."""
