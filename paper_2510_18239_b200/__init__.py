"""B200-native LIME ranking inference hot path: C-ABI CUDA library + thin Python binding.

`synth` draws the seeded synthetic workloads; `binding` marshals arguments to the C-ABI
library (built in-tree by `build`).  Importing the package does not load the CUDA library;
the first call through `binding` does, and raises if it is missing.
"""
__all__ = ["synth", "binding", "build", "shard"]
