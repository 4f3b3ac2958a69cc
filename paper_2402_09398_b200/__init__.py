"""B200-native LESS decode / prefill hot path (arxiv 2402.09398).

The product is the C-ABI library built from ``csrc/`` (see ``include/less.h``);
``binding`` is the thin ctypes layer over it and ``workloads`` holds the seeded
synthetic input generators.  Importing the package does not load the library:
``binding.lib()`` does, and raises if it has not been built.
"""
__all__ = ["binding", "workloads", "build"]
