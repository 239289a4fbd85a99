"""B200-native ESSA population-projection path: CUDA library (csrc/), ctypes binding, synthetic workloads.

Importing the package loads nothing heavy; `paper_2507_04453_b200.binding` loads the C-ABI
library on first use and raises if it has not been built.
"""
__all__ = ["workloads", "binding", "build"]
