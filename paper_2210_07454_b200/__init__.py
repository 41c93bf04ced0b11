"""B200-native SketchedAMSGrad (gradient averaging) step: CUDA library + thin ctypes binding.

Nothing is loaded at import time; `binding.lib()` loads the built shared library and raises if it is missing.
"""
__all__ = ["binding", "build", "synthetic"]
