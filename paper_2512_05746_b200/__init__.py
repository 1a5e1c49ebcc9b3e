"""B200-native Hadamard-quantized layer forward (HQ-DM hot path).

Sub-modules:
  inputs   seeded synthetic input generators (no method arithmetic; shared by tests, bench and oracle checks)
  binding  ctypes binding of the C-ABI library ``libhq.so`` (loads the CUDA library; raises if it is missing)
  build    compiles ``csrc/*.cu`` for sm_100a into ``libhq.so`` next to this file

Importing the package itself loads nothing native; ``binding`` does, and fails loudly
when the CUDA library has not been built.
"""

__all__ = ["inputs", "binding", "build"]
