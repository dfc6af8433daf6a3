"""CriticalKV prefill-time KV-cache compression for NVIDIA B200: CUDA kernels behind a C ABI, plus this binding.

`binding` mirrors include/criticalkv.h one to one; `build.build_library()` compiles the kernels in-tree.
Importing the package does not load the shared library; the first call does, and fails if it is not built.
"""
from . import binding, build  # noqa: F401
from .binding import *  # noqa: F401,F403
from .session import ChunkedPrefillCompressor, CompressionSession, session_for, to_device, to_host  # noqa: F401,E402
