"""Seeded synthetic inputs shared by the CPU oracle's tests and the CUDA path's tests.

This module holds segment layouts, random-gradient recipes and the index draws of random-k only.  None of the
method's arithmetic (compressors, aggregation, updates) lives here, so that the
oracle and the CUDA library can both be fed the same bytes without sharing code.
"""
from .layouts import (Layout, flat_layout, resnet18_layout, resnet50_layout,
                      gpt2_small_layout, scaled_layout, ragged_layout, topk_counts, equal_blocks_layout)
from .grads import (WORKLOADS, Workload, make_gradients, gradient_seed)
from .subsets import random_subsets, subset_seed

__all__ = [
    "Layout", "flat_layout", "resnet18_layout", "resnet50_layout", "gpt2_small_layout",
    "scaled_layout", "ragged_layout", "topk_counts", "equal_blocks_layout",
    "WORKLOADS", "Workload", "make_gradients", "gradient_seed", "random_subsets", "subset_seed",
]
