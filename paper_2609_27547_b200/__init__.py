"""B200-native batched action generation (the rollout stage's generation hot path) behind a
C ABI: ``include/ebrl_actgen.h`` declares the calls, ``csrc/`` holds the CUDA kernels, and
``binding`` is the thin ctypes layer with the same names.  ``synth`` draws the seeded synthetic
inputs and holds none of the method's arithmetic."""
from . import synth  # noqa: F401

__all__ = ["synth", "binding", "build"]
