"""B200-native (sm_100a) 4-bit training hot path: amax, INT4 and LUQ-FP4
quantize-and-pack, and the forward / backward / update GEMMs on tcgen05.

The compute lives in the C-ABI library declared in ``include/luq.h``; this
package is a thin ctypes binding (``binding``), the in-tree build step
(``build``) and the seeded synthetic workloads (``inputs``).  There is no CPU
fallback: using the binding without the compiled library raises.
"""
from . import inputs  # noqa: F401

__all__ = ["inputs", "binding", "build"]
