"""mHC-lite residual-mixing hot path for B200 (sm_100a): CUDA kernels behind a C ABI.

``binding`` is the thin ctypes layer over the shared library; ``synth`` draws the
seeded synthetic inputs.  Nothing here computes on the CPU: every call into
``binding`` needs the compiled library and a CUDA device and fails loudly without.
"""
__all__ = ["synth", "binding", "build"]
