"""B200-native verify step of HOLA's Hierarchical Speculative Decoding: thin binding over libhola_verify.so.

`workloads` (seeded synthetic inputs) imports nothing from the CUDA side; `binding` loads the C-ABI library and
fails loudly when it is missing or when no sm_100 device is present.  There is no CPU fallback.
"""
from . import workloads  # noqa: F401

__all__ = ["workloads", "binding", "build"]
