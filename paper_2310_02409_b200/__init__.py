"""B200-native implementation of the inference hot path of Dodo (arXiv 2310.02409):
score -> TopK select -> K/V gather into a nugget cache -> attention over nuggets plus local tokens.

Sub-modules are imported on demand so that ``inputs`` (the seeded input generators) can be
used without loading the CUDA library:

  ``inputs``   seeded synthetic tensors and workload shapes
  ``build``    compiles ``csrc/`` into ``libdodo.so`` with nvcc for sm_100a
  ``api``      thin ctypes binding over the C ABI declared in ``include/dodo.h``
"""
__all__ = ["inputs", "build", "api"]
