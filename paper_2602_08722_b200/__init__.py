"""QuoKA per-chunk sparse prefill attention for NVIDIA B200 (sm_100a).

The compute path lives in the C-ABI shared library built from ``csrc/``; ``api``
is a thin ctypes binding with the same entry-point names.  ``synth`` draws the
seeded synthetic inputs.  Importing the package is cheap; the shared library is
loaded on first use of ``api`` and a missing library is an error, never a
fallback.
"""
__all__ = ["api", "synth"]
