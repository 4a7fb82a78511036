"""B200-native verification hot path of multi-token assisted decoding (MTAD / MMTAD, arxiv 2407.09722).

The product is the C-ABI library built from csrc/ (see include/mtad.h); this package is its thin Python binding.
"""
from .binding import (Context, ModelDesc, MtadError, Result, ResultBuffers, load_library, log_tau, make_desc,
                      mtad_workspace_bytes, mtad_kernel_launches, EXPORTS, LIB_PATH,
                      KERNEL_CLASSES)

__all__ = ["Context", "ModelDesc", "MtadError", "Result", "ResultBuffers", "load_library", "log_tau", "make_desc",
           "mtad_workspace_bytes", "mtad_kernel_launches", "EXPORTS", "LIB_PATH", "KERNEL_CLASSES"]
