"""Representation Shift hot path on B200: ctypes binding of the CUDA library.

The shared library is loaded on first use (see binding.load_library); importing
the package needs neither a GPU nor the built library, so the input generator
(`synth`) and the build script stay importable everywhere.
"""
from .binding import (Context, block_fwd_static, static_async_status, DeviceBlockWeights, PrunedViT, RsError, load_library, LIB_PATH,  # noqa: F401
                      EXPORTS, attn_kernel_choice)
