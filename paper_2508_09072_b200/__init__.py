"""B200-native batched tree verification for lossless speculative decoding.

The product is the C-ABI library ``libreader_verify.so`` (hand-written sm_100a
CUDA, sources under ``csrc/``, declarations in ``include/reader_verify.h``).
``binding`` is its thin ctypes wrapper; ``workloads`` draws seeded synthetic
inputs and contains none of the method's arithmetic.  Importing the package
does not load the library; calling into ``binding`` does, and raises if the
library has not been built.
"""
__all__ = ["workloads", "binding", "build"]
