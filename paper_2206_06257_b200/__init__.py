"""B200-native hot path of DAT's outer-minimisation step (quantize -> aggregate -> LALR).

Sub-modules are imported on first use:
  api    -- thin ctypes binding of the C-ABI library (CUDA, sm_100a); fails loudly
            if the library has not been built
  build  -- nvcc build of the library
  synth  -- seeded synthetic inputs (no method arithmetic)
"""
import importlib

__all__ = ["api", "build", "synth"]


def __getattr__(name):
    if name in __all__:
        return importlib.import_module("." + name, __name__)
    raise AttributeError(name)
