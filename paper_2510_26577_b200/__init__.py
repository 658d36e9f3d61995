"""B200-native hot path of CAST (cost-aware dynamic draft trees for speculative
decoding): CUDA kernels for sm_100a behind a C-ABI library, plus a thin ctypes
binding.  Importing the package does not load the CUDA library; `binding`
does, and fails loudly if the library has not been built."""

__all__ = ["workloads", "binding", "replicas", "ablation", "cost_profile"]
