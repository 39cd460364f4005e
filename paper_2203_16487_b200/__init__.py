"""B200-native SpecDec draft -> verify -> commit path (CUDA library + ctypes binding).

`workloads` (seeded synthetic inputs) imports without a GPU; `binding` loads the
CUDA library and fails loudly when it is missing.
"""
__all__ = ["workloads", "binding", "build"]
