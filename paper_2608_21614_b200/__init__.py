"""B200-native MoE expert step of SAEM (stage-aware expert management).

The package holds the CUDA kernels and their C-ABI library (``csrc/``), the
thin ctypes binding with the same names (``binding``), the seeded synthetic
input generators (``inputs``) and the host-side cache policy used by the
32-layer stack workload (``stack``).

Importing the package does not load the CUDA library; ``binding`` does, and
raises if the library is missing -- there is no CPU fallback.
"""

__all__ = ["inputs"]
