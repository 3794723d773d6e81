"""SDFP speculative-decode hot path for NVIDIA B200: a C-ABI CUDA library
(csrc/, include/sdfp.h) and this thin ctypes binding."""
from .binding import (FLAG_FMA_GEMM, FLAG_NO_GRAPH, FLAG_NO_DENSE, FLAG_NO_PASS_KERNEL, FLAG_NO_PDL, EXPORTS, GenOutput, Sdfp, SdfpError,
                      load_library, sdfp_fit_scores)
from .build import LIB_PATH, build_library

__all__ = ["Sdfp", "SdfpError", "GenOutput", "sdfp_fit_scores", "load_library", "build_library", "LIB_PATH", "EXPORTS",
           "FLAG_NO_GRAPH", "FLAG_NO_PDL", "FLAG_FMA_GEMM", "FLAG_NO_PASS_KERNEL", "FLAG_NO_DENSE"]
