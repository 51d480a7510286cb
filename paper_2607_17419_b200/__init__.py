"""KATA forward pass for B200 (sm_100a): hand-written CUDA kernels behind a C ABI.

``inputs`` draws the seeded synthetic workloads; ``binding`` is the thin ctypes layer
over ``libkata.so`` (built in-tree by ``build.py``).  Importing this package does not
load the library; ``binding.lib()`` does, and raises if it is missing.
"""
__all__ = ["inputs", "binding", "build"]
