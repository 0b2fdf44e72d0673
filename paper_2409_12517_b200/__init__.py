"""FP8 Smooth-SwiGLU MLP block (forward + backward) for NVIDIA B200.

`binding` holds the Python mirror of the C ABI in include/fp8mlp.h (libfp8mlp.so, built by
`build`); `workloads` draws the seeded synthetic inputs.  Nothing is loaded at import time.
"""
__all__ = ["binding", "build", "workloads"]
