"""B200-native block-diffusion denoise step (Fast-dVLM decoding hot path) as a C-ABI CUDA library.

`inputs` holds the seeded synthetic workloads; `binding` is the thin ctypes layer over
`libfdvlm.so` (argument marshalling only -- every step of the path runs in the CUDA kernels).
"""
from . import inputs  # noqa: F401

__all__ = ["inputs", "binding", "build"]
