"""B200-native tensor-granular prefetch engine for oversubscribed transformer inference.

The hot path lives in libtgp.so (csrc/): registry, trace, roofline planner, copy engine and the
sm_100a kernels.  `binding` exposes its C ABI one to one; `session` wires a synthetic pool to it.
"""
from . import binding  # noqa: F401
