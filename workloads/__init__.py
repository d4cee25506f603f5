"""Seeded synthetic inputs for the FastOCR decode-attention hot path.

This package only manufactures bytes (K/V caches, queries, page tables, fixation
tracks). It contains none of the method's arithmetic (no attention, no scoring,
no selection) and is the only code shared by the CPU oracle's tests and the CUDA
path's tests/bench.
"""
from .generator import (  # noqa: F401
    stream_key, normal_bf16, make_kv, make_queries, fixation_track,
    make_page_table, scatter_to_pages, window_indices,
)
from .configs import WorkloadConfig, get_config, kept_count_hint  # noqa: F401
