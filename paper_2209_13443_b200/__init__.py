"""B200-native hot path of batched early-exit CNN serving.

Stage-by-stage execution of an early-exit CNN under a batch that shrinks at
every exit and is refilled at stage boundaries (the problem statement of
"Fluid Batching", Methodology and Algorithm 1).  The product is the C-ABI
library declared in ``include/ee.h``; :mod:`.binding` is the thin ctypes layer
over it and :mod:`.workloads` holds the seeded synthetic inputs and network
shapes (no arithmetic of the method lives there).

Nothing is imported eagerly: ``workloads`` must stay importable without the
CUDA library so that CPU-only tooling can generate inputs.
"""

__all__ = ["binding", "workloads", "build"]
