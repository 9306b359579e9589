"""B200 (sm_100a) implementation of the CORE round (Common Random Reconstruction):
project -> aggregate -> reconstruct with common Gaussian vectors that are regenerated
on the fly, plus the least-squares CORE-GD step (Algorithms 1 and 2 of the paper).

The work is done by the CUDA library ``libcore_b200.so`` (C ABI in ``include/core.h``);
``binding`` marshals torch tensors into it.  ``python -m paper_2309_13307_b200.build``
compiles the library in-tree.
"""
from .binding import (CORE_BF16, CORE_ELIMIT, CORE_F32, Core, CoreError, LeastSquares, core_device_status,
                      core_project_static, exported_symbols, lib, library_path)

__all__ = ["Core", "LeastSquares", "CoreError", "CORE_F32", "CORE_BF16", "CORE_ELIMIT", "core_project_static",
           "core_device_status", "lib", "library_path", "exported_symbols"]
