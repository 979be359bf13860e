"""B200-native frozen-counts sweep of the LightLDA O(1) Metropolis-Hastings sampler.

The package holds the CUDA kernels and their C-ABI (``csrc/``), a ctypes
binding with the same names (``binding``), the nvcc build step (``build``) and
the seeded synthetic-corpus generator (``synth``).  Nothing is loaded on
import: the shared library is opened on first use of the binding and a missing
library raises instead of falling back to anything else.
"""

__all__ = ["binding", "build", "synth"]
