"""FlowCache hot path for NVIDIA B200: thin Python binding over the C-ABI library ``libfc.so``.

The four calls carry the names of the C entry points and only marshal arguments: every step of
the path runs in the library's CUDA kernels.  PyTorch is used for device memory and streams
only.  There is no CPU fallback: importing works anywhere (so that the library can be built
and its symbols checked without a GPU), but creating a :class:`Context` needs a B200.
"""
from .binding import (BF16, F32, Context, FcError, STATUS_BITS, exported_symbols, declared_symbols,
                      lib, lib_path)

__all__ = ["BF16", "F32", "Context", "FcError", "STATUS_BITS", "exported_symbols", "declared_symbols",
           "lib", "lib_path"]
