"""B200-native decode hot path of TokenButler: projected-key cache, fused importance scoring +
top-B selection, neighbour fetching, prediction interval, and split-K sparse decode attention.

``paper_2503_07518_b200.binding`` is the ctypes layer over the C-ABI library (it fails loudly when
the CUDA library has not been built); ``paper_2503_07518_b200.workloads`` draws the synthetic
inputs and needs neither CUDA nor the library.
"""

__all__ = ["binding", "workloads", "build"]
