"""B200-native W4 linear layers (int4 asymmetric group-quantised weights, fused dequantisation).

The package holds the CUDA kernels and the C-ABI library (``csrc/``), the build step
(``build.py``), the ctypes binding (``binding.py``) and the seeded synthetic input generators
(``inputs.py``).  Importing the package does not load the CUDA library; ``binding`` does, and
fails loudly when the library has not been built.
"""

__all__ = ["binding", "build", "inputs", "workloads"]
