"""TopLoc proof hot path for NVIDIA B200: hand-written sm_100a kernels behind a C ABI.

`binding` mirrors the C entry points of include/toploc.h (argument marshalling only);
`synth` is the seeded input generator.  There is no CPU fallback: every call needs the
compiled CUDA library and fails loudly without it.
"""
from . import synth  # noqa: F401
from .binding import *  # noqa: F401,F403
