"""B200-native MoE expert FFN (forward + backward) behind a C-ABI CUDA library.

`paper_2606_26453_b200.binding` is the thin ctypes layer over libmoe_b200.so (it raises if the
library has not been built); `paper_2606_26453_b200.workloads` draws the seeded synthetic inputs.
"""
__all__ = ["workloads"]
