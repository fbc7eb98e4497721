"""B200-native Token Filtering layer step (per-layer online pruning + pruned attention).

``paper_2512_07090_b200.binding`` is the thin ctypes layer over the C-ABI CUDA
library (``include/tf.h``); ``paper_2512_07090_b200.workloads`` makes the seeded
synthetic inputs.  There is no CPU fallback: using the binding without the
built CUDA library raises.
"""
__all__ = ["binding", "workloads"]
