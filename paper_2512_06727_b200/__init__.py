"""KV-CAR decode hot path for NVIDIA B200: Python binding of the CUDA library.

`binding` mirrors the C ABI (include/kvcar.h); `session` holds the torch-side
plumbing (device buffers, streams).  All arithmetic runs in libkvcar.so.
"""
from . import binding  # noqa: F401
from .binding import (BF16, F32, INCLUDE_CURRENT_EXACT, KERNEL_AUTO, KERNEL_GENERIC, KERNEL_TENSOR, K, V,  # noqa: F401
                      Context, KvcarError)
