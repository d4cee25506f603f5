"""CPU oracle for the FastOCR decode-attention hot path: TEST INFRASTRUCTURE ONLY.

Imported by tests/, the smoke check and the bench's cpu_baseline / reference arm; never by
the product package. The arithmetic lives in fastocr_oracle.cpp (plain C++); this module is
a ctypes wrapper plus the step schedule of Algorithm 1 written over those primitives.
"""
from .binding import (  # noqa: F401
    dense, probs, scores, topk, sparse, masked_dense, kept_count, focal_layers, attn_flops, attn_flops_pruned,
    set_threads, num_threads,
)
from .schedule import decode_step, warmup_step, StepTrace, profile_focal_layers  # noqa: F401
