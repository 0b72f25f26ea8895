"""B200-native (sm_100a) chunkwise training backward of the gated delta rule (GDN) recurrence.

The product is the C-ABI shared library `libgdn_b200.so` (declared in include/gdn.h); `binding`
marshals torch device tensors into it and `runner` offers allocation helpers around it.  `synth`
draws seeded synthetic workloads and contains none of the method's arithmetic.  Nothing in this
package imports the CPU oracle, and there is no CPU or framework fallback for the kernels.
"""
from . import synth  # noqa: F401  (numpy only)

__all__ = ["synth", "binding", "runner", "build"]
