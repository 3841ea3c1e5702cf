"""B200-native scheduled-Lasso round (STRADS, Algorithm 1): CUDA library + thin binding.

`workloads` (synthetic problem generators) imports without the CUDA library;
`binding` loads `libstrads_b200.so` and fails loudly when it is missing.
"""
__all__ = ["workloads", "binding"]
