"""B200-native tree verification for speculative decoding of LLM-based speech recognition.

`binding` mirrors the C ABI of include/specasr.h one to one; `runtime` holds the torch-owned
device buffers the library borrows.  The CUDA library is built in-tree by `build.build()`.
"""
from . import binding
from .binding import SpecasrError

__all__ = ["binding", "SpecasrError"]
