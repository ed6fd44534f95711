"""B200-native per-stage micro-batched training step (hand-written CUDA for sm_100a behind a C ABI).

The Python layer only marshals arguments to `lib/libasteroid.so`; every step of the path runs
in the library's kernels.  There is no CPU fallback: importing works without a GPU, calling
any compute entry point without the built library or without a CUDA device raises.
"""
from .binding import *          # noqa: F401,F403
from .build import build        # noqa: F401
