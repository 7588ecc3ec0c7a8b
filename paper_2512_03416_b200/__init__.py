"""B200-native mixed paged-attention step of a Convertible Decoder (TokenScale, arXiv 2512.03416).

Sub-modules:
  binding    ctypes binding of libtokenscale.so (same names as include/tokenscale.h)
  decoder    convenience wrapper that owns the device buffers through PyTorch
  workloads  seeded synthetic workloads (no attention arithmetic, no CUDA)
  build      in-tree nvcc build of the library

Nothing is imported eagerly, so `workloads` can be used on a machine without the built library.
"""
__all__ = ["binding", "decoder", "workloads", "build"]
