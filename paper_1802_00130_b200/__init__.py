"""Subsampled Gauss-Newton products for fully-connected networks on one B200.

Thin ctypes binding over the C ABI of include/gn.h: argument marshalling only, every step of the
path runs in the library's CUDA kernels.  PyTorch supplies device memory and streams.
"""
from .binding import (GN_FP32_ACCURATE, GN_TF32, GnContext, GnError, NewtonParams, NewtonReport, exported_symbols, lib, lib_path,
                      plan_group, thin_m_gemm_noalloc)

__all__ = ["GnContext", "GnError", "GN_TF32", "GN_FP32_ACCURATE", "lib", "lib_path", "exported_symbols", "NewtonParams", "NewtonReport", "thin_m_gemm_noalloc", "plan_group"]
