"""B200-native blocked adaptive randomized range finder (Householder QR based).

`paper_2608_28941_b200.rrf` is the thin ctypes binding over the C-ABI library
(`librrf.so`, built from `csrc/`); `paper_2608_28941_b200.workloads` generates
seeded synthetic inputs.  Nothing is loaded at import time: the shared library
is opened on first use and a missing library is an error, never a fallback.
"""
__all__ = ["rrf", "workloads"]
