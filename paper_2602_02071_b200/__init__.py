"""BAPS on B200: fused HiF8 attention forward (block-aware precision rescaling for softmax).

The product is the C-ABI CUDA library built from ``csrc/`` (declared in ``include/baps.h``);
``binding`` is a thin ctypes layer over it with the same entry-point names.  Importing this
package does not load the CUDA library; the first call through ``binding`` does, and fails
loudly if the library has not been built.
"""
__all__ = ["binding", "workloads"]
