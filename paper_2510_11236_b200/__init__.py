"""B200-native decode attention over an XQuant (cross-layer, 1/2-bit) KV cache.

The compute lives in libxq.so (CUDA, sm_100a); `binding` forwards to its C
entry points, `workloads` generates the seeded synthetic inputs, `build`
compiles the library in-tree.
"""
from . import binding  # noqa: F401
from .binding import *  # noqa: F401,F403
