"""B200-native clustered-MoE layer forward (hierarchical routing, shared-base +
INT4 low-rank expert FFNs, gated combine) behind a small C ABI.

`inputs` holds the seeded synthetic workloads; `binding` is the thin ctypes
layer over the CUDA library (imported lazily so that CPU-only tools can use the
generators without the extension)."""
from . import inputs  # noqa: F401

__all__ = ["inputs"]
