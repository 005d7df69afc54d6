"""B200-native per-view training step of point-based (3D Gaussian) neural rendering behind a C ABI.

  workloads  seeded synthetic scenes and cameras (NumPy only, no method arithmetic)
  build      compiles csrc/*.cu into libodin.so for sm_100a
  binding    ctypes entry points with the names of include/odin.h
  engine     device buffers through PyTorch and the call sequence of one training view

Importing the package does not load the CUDA library; the first binding call does, and raises if it is missing.
"""
__all__ = ["workloads", "build", "binding", "engine"]
