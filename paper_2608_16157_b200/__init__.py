"""B200-native expert-cached MoE layer: CUDA library (csrc/), its ctypes binding and the seeded
synthetic workloads.  ``binding`` loads the shared library and fails loudly if it is missing."""
__all__ = ["binding", "build", "workload"]
