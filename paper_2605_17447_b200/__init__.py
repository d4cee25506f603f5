"""FastOCR decode-step attention hot path for B200 (sm_100a): thin Python binding over the C ABI
declared in include/fastocr.h. Every step of the path runs in the CUDA library; this package only
marshals pointers. Importing it requires the built library (python -m paper_2605_17447_b200.build)."""
from .api import (  # noqa: F401
    Context, KVView, FastOCRError, kept_count, focal_layers, attn_flops, attn_flops_pruned, launch_count, cluster_launch_count,
    fastocr_dense_decode_attn, fastocr_focal_scores, fastocr_select_topk, fastocr_sparse_decode_attn,
    fastocr_decode_step, fastocr_warmup_step, fastocr_sparse_decode_attn_noalloc, noalloc_device_faults, StepPlan, PROF_CLASSES,
)
from .sharding import make_scores_exchange, mean_ratio_over_ranks, shard_heads, shard_sequences  # noqa: F401
