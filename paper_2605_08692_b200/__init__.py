"""B200 (sm_100a) AAAC per-layer quantisation path: a C-ABI CUDA library and a thin binding.

``binding`` marshals torch tensors (device pointers, the current stream) into the C ABI
declared in ``include/aaac.h``; every step of the path runs in the library's kernels.
``synth`` holds the seeded synthetic input generators, ``sharding`` the host logic of the
layer-parallel multi-rank path.  Nothing here falls back to a CPU
implementation: using ``binding`` without the built library raises.
"""
from . import synth  # noqa: F401

__all__ = ["synth", "binding", "build", "sharding"]
