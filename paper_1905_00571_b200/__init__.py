"""B200 (sm_100a) sparse-CNN inference library: Python face of the C ABI in include/cadnn.h.

The CUDA library must be built first (``python -m paper_1905_00571_b200.build``);
importing ``paper_1905_00571_b200.binding`` without it raises ImportError.
"""
