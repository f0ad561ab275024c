"""B200-native trace-window analyzer: the reconstruction stage of the paper's
Analyzer (Sec. 6.1) as hand-written sm_100a CUDA kernels behind a C ABI.

`paper_2609_40247_b200.ta` is the binding of the C ABI (include/ta.h);
`paper_2609_40247_b200.synth` generates seeded synthetic windows.  Importing
this package loads nothing native; the CUDA library is loaded on first use and
there is no CPU fallback.
"""
__all__ = ["synth", "ta"]
