"""capmoe: capacity-aware MoE layer forward (route, Token Drop, Expanded Drop, permute,
grouped SwiGLU FFN, combine) as sm_100a CUDA kernels behind a C ABI.

`synth` holds the seeded input generators; `capmoe` is the ctypes binding of the CUDA
library (imported lazily so that CPU-only tooling can use `synth` without it)."""
__all__ = ["synth"]
