"""B200 activation codec (Channel-wise Mix Compression, FedHybrid, arXiv 2510.11400, Section 4.4.1).

`api` binds the C ABI of the CUDA library (include/fh.h); `synth` draws the seeded synthetic
activations; `build` compiles the library.  Importing this package loads nothing; the library is
loaded on first use and its absence is an error, never a fallback.
"""
__all__ = ["api", "synth", "build"]
