"""B200-native Cartridge decode attention (arXiv 2506.06266, serving hot path).

``synth``    seeded synthetic inputs (no attention arithmetic).
``binding``  thin ctypes binding over the C-ABI library ``libcart.so`` (imported on first use;
             raises if the CUDA library has not been built -- there is no CPU fallback).
"""
__all__ = ["synth", "binding", "buildlib"]
