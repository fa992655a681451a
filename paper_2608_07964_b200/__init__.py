"""Cross-layer MoE step (EasyBalance) for NVIDIA B200: C-ABI CUDA library plus a thin binding.

`synth` (seeded inputs) imports without CUDA; `binding` loads libeb.so and fails loudly if the
library cannot be found or built.
"""
from importlib import import_module

__all__ = ["synth", "binding", "build"]


def __getattr__(name):
    if name in __all__:
        return import_module(f"{__name__}.{name}")
    raise AttributeError(name)
