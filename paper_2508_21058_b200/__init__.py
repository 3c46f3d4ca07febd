"""B200-native Mixture-of-Contexts routing + sparse attention (C-ABI CUDA library + thin binding).

The binding only marshals arguments; every step of the path runs in the library's CUDA
kernels.  Loading fails loudly if ``libmoc.so`` is missing: there is no CPU fallback.
"""
from .binding import (MocError, MocPlan, FLAG_CAUSAL, WHOLE_SHOT, lib_path, load_library,
                      launch_count)

__all__ = ["MocError", "MocPlan", "FLAG_CAUSAL", "WHOLE_SHOT", "lib_path", "load_library",
           "launch_count"]
