"""ConQuR online rotation-calibration hot path for B200 (sm_100a).

The package holds the CUDA kernels + C-ABI library (``csrc/``), a thin ctypes
binding (``binding.py``) and the seeded synthetic input generators
(``inputs.py``).  Importing the package does not load the CUDA library; the
binding loads it on first use and raises if it is missing (there is no CPU
fallback).
"""

__all__ = ["binding", "inputs"]
