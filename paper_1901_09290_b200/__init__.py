"""B200-native hot path of PruneTrain (arxiv 1901.09290): conv fwd/dgrad/wgrad on ragged pruned
channel counts, the fused group-lasso + momentum-SGD step, zero-group detection and channel-union
compaction, as hand-written sm_100a CUDA kernels behind a small C ABI (``include/pt.h``).

``paper_1901_09290_b200.binding`` is the thin ctypes layer over the shared library;
``paper_1901_09290_b200.workloads`` holds shape tables and seeded input generators only.
Nothing here falls back to the CPU: calls raise if the CUDA library is missing.
"""
__all__ = ["binding", "workloads"]
