"""LoRAct activation-compression hot path for NVIDIA B200: a C-ABI CUDA library and its thin binding.

``binding`` loads the library lazily; ``synth`` draws the seeded synthetic workloads; ``build`` compiles
the CUDA sources in-tree.  Nothing here falls back to the CPU.
"""
from . import synth  # noqa: F401

__all__ = ["synth", "binding", "build"]
