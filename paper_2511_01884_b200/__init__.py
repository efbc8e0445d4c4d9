"""B200-native fused linear operator: Y = epilogue(act(X W^T + b)) with an optional row
reduction (sum, max, LayerNorm over N), one hand-written sm_100a kernel per call.

``binding`` mirrors the C interface in ``include/forge.h``; ``workloads`` holds the seeded
synthetic inputs; ``build`` compiles ``csrc/`` into ``libforge.so`` in-tree."""
from . import binding, workloads  # noqa: F401
from .binding import (FusedLinear, ForgeError, make_desc)  # noqa: F401
