"""B200-native draft-tree verification hot path of HeteroSpec (arXiv 2505.13254).

The package holds the CUDA kernels and their C-ABI (``csrc/``), the thin ctypes
binding (``binding``), the build step (``build``) and the seeded synthetic input
generators (``synth``).  Importing the package loads nothing native; the shared
library is loaded on first use of ``binding.lib()`` and a missing library is an
error, never a fallback.
"""

__all__ = ["binding", "build", "synth"]
