"""B200-native Mixture-of-Channels (MoC) FFN operator.

The product is the C-ABI library built from ``csrc/`` (hand-written sm_100a CUDA kernels);
``binding`` is a thin ctypes layer with the same entry-point names, and ``synthetic`` holds the
seeded input recipe.  Importing the package is cheap: the shared library is loaded on the first
call into ``binding``, which raises if the library is missing -- there is no CPU fallback.
"""

__all__ = ["binding", "synthetic", "build"]
