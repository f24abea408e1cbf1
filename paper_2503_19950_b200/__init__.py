"""LogQuant decode hot path for B200 (sm_100a): thin ctypes binding over the C-ABI library.

Every step of the path runs in the CUDA kernels of ``liblogquant.so``; this package only marshals
arguments.  PyTorch is used by callers for device memory and streams.
"""
from .binding import (LQ_DEVICE_NONE, LQ_FLAG_OVERLAP_DECODE, LQ_FILTER_LOG, LQ_FILTER_RECENT, LQ_KERNEL_AUTO, LQ_KERNEL_MMA, LQ_KERNEL_UMMA,
                      LQ_KERNEL_SCALAR, LogQuantCache, LogQuantError, decode_attn_image_static, exported_symbols,
                      load_library)

__all__ = ["LogQuantCache", "LogQuantError", "load_library", "exported_symbols", "decode_attn_image_static",
           "LQ_DEVICE_NONE",
           "LQ_KERNEL_AUTO", "LQ_KERNEL_SCALAR", "LQ_KERNEL_MMA", "LQ_KERNEL_UMMA", "LQ_FILTER_LOG", "LQ_FILTER_RECENT", "LQ_FLAG_OVERLAP_DECODE"]
