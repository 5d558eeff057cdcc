"""B200-native hot path of AB-Training (factorised-layer training step and group synchronisation).

The package holds the CUDA kernels plus their C-ABI (``csrc/``), a thin ctypes
binding (``binding``) and the seeded synthetic-input generators (``synth``).
Importing the package does not load the CUDA library; ``binding`` loads it on
first use and raises if it is missing.
"""

__all__ = ["binding", "synth", "build"]
