"""B200-native cloud-side NAV verify pass of speculative decoding (paper Sec. 2.2 / App. B).

`binding` is the thin ctypes layer over the CUDA library (csrc/, include/pipesd.h); `synth` makes
seeded synthetic inputs.  The CUDA library is loaded on first use and there is no CPU fallback.
"""
__all__ = ["binding", "synth", "build"]
