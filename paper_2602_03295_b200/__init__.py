"""POP (Prefill-Only Pruning) pruned-prefill path for NVIDIA B200: Python binding of the C-ABI
CUDA library. All arithmetic runs in the library's kernels; this package only marshals arguments."""
from .binding import (PopError, PopLibrary, PopModel, lib, POP_OK, POP_E_INVALID, POP_E_NOSPACE, POP_E_CUDA,
                      POP_E_DEVICE_TIMEOUT, POP_E_MISSING)

__all__ = ["PopError", "PopLibrary", "PopModel", "lib", "POP_OK", "POP_E_INVALID", "POP_E_NOSPACE",
           "POP_E_CUDA", "POP_E_DEVICE_TIMEOUT", "POP_E_MISSING"]
