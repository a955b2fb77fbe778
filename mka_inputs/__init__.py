"""Seeded synthetic inputs for the FastMKA hot path.

This package holds only the input recipe: a counter-based pseudo-random
generator and the tensor shapes of the benchmark configurations.  It contains
none of the attention / routing arithmetic, and it is the one module that both
the CPU oracle's tests and the CUDA path's tests and benchmark may import.
"""
from .generator import approx_normal, CONFIGS, WorkloadConfig, make_tensor, TENSOR_IDS  # noqa: F401
from .generator import PAGED_CONFIGS, PagedConfig, make_paged, paged_rows, paged_tables  # noqa: F401
from .generator import RECALL_CONFIGS, RecallConfig, make_recall  # noqa: F401
