"""Loads libfastocr.so and declares the C signatures. There is no fallback: a missing library is
an error."""
from __future__ import annotations

import ctypes as C
import os

HERE = os.path.dirname(os.path.abspath(__file__))
# FASTOCR_LIB: development knob, another build of the same library (a debug or experimental variant)
LIB_PATH = os.environ.get("FASTOCR_LIB") or os.path.join(HERE, "libfastocr.so")


class KVViewStruct(C.Structure):
    _fields_ = [
        ("batch", C.c_int32), ("num_q_heads", C.c_int32), ("num_kv_heads", C.c_int32), ("head_dim", C.c_int32),
        ("page_size", C.c_int32), ("max_seq_len", C.c_int32),
        ("k", C.c_void_p), ("v", C.c_void_p),
        ("seq_stride_tokens", C.c_int64),
        ("block_table", C.c_void_p), ("max_pages", C.c_int32), ("num_pages", C.c_int32),
        ("seq_len", C.c_void_p), ("vis_start", C.c_void_p), ("vis_len", C.c_void_p),
        ("sm_scale", C.c_float),
    ]


# int (*)(float* scores, int32 batch, int32 n_stride, int32 layer, void* stream, void* user)
ScoresExchangeFn = C.CFUNCTYPE(C.c_int, C.c_void_p, C.c_int32, C.c_int32, C.c_int32, C.c_void_p, C.c_void_p)


class StepOptionsStruct(C.Structure):
    _fields_ = [("is_focal_seq", C.c_void_p), ("is_focal_seq_dev", C.c_void_p), ("union_sets", C.c_int32),
                ("scores_exchange", ScoresExchangeFn), ("scores_exchange_user", C.c_void_p)]


class LimitsStruct(C.Structure):
    _fields_ = [("max_batch", C.c_int32), ("num_q_heads", C.c_int32), ("num_kv_heads", C.c_int32),
                ("max_seq_len", C.c_int32), ("max_vis_len", C.c_int32)]


EXPORTS = {
    "fastocr_create": (C.c_int, [C.POINTER(C.c_void_p), C.c_int, C.POINTER(LimitsStruct)]),
    "fastocr_destroy": (None, [C.c_void_p]),
    "fastocr_last_error": (C.c_char_p, [C.c_void_p]),
    "fastocr_device_faults": (C.c_int64, [C.c_void_p]),
    "fastocr_kept_count": (C.c_int32, [C.c_int32, C.c_double]),
    "fastocr_dense_decode_attn": (C.c_int, [C.c_void_p, C.POINTER(KVViewStruct), C.c_void_p, C.c_void_p, C.c_int,
                                            C.c_void_p, C.c_int32, C.c_void_p, C.c_void_p]),
    "fastocr_focal_scores": (C.c_int, [C.c_void_p, C.POINTER(KVViewStruct), C.c_void_p, C.c_void_p, C.c_int32,
                                       C.c_void_p, C.c_void_p]),
    "fastocr_select_topk": (C.c_int, [C.c_void_p, C.c_void_p, C.c_int32, C.c_void_p, C.c_void_p, C.c_int32,
                                      C.c_int32, C.c_void_p, C.c_int32, C.c_void_p]),
    "fastocr_sparse_decode_attn": (C.c_int, [C.c_void_p, C.POINTER(KVViewStruct), C.c_void_p, C.c_void_p, C.c_void_p,
                                             C.c_int32, C.c_int32, C.c_void_p, C.c_int, C.c_void_p]),
    "fastocr_decode_step": (C.c_int, [C.c_void_p, C.c_int32, C.POINTER(KVViewStruct), C.c_void_p, C.c_void_p, C.c_int,
                                      C.c_void_p, C.c_void_p, C.c_void_p, C.c_int32, C.c_int, C.c_int32, C.c_int32,
                                      C.POINTER(C.c_int), C.c_void_p]),
    "fastocr_decode_step_ex": (C.c_int, [C.c_void_p, C.c_int32, C.POINTER(KVViewStruct), C.c_void_p, C.c_void_p, C.c_int,
                                         C.c_void_p, C.c_void_p, C.c_void_p, C.c_int32, C.c_int, C.c_int32, C.c_int32,
                                         C.POINTER(C.c_int), C.POINTER(StepOptionsStruct), C.c_void_p]),
    "fastocr_warmup_step": (C.c_int, [C.c_void_p, C.c_int32, C.POINTER(KVViewStruct), C.c_void_p, C.c_void_p, C.c_int,
                                      C.c_void_p, C.c_void_p]),
    "fastocr_focal_layers": (C.c_int32, [C.c_void_p, C.c_int32, C.c_double, C.c_int32, C.c_void_p]),
    "fastocr_attn_flops": (C.c_double, [C.c_double] * 4),
    "fastocr_attn_flops_pruned": (C.c_double, [C.c_double] * 6),
    "fastocr_sparse_decode_attn_noalloc": (C.c_int, [C.POINTER(KVViewStruct), C.c_void_p, C.c_void_p, C.c_void_p, C.c_int32,
                                                     C.c_void_p, C.c_int, C.c_void_p]),
    "fastocr_noalloc_last_error": (C.c_char_p, []),
    "fastocr_noalloc_device_faults": (C.c_int64, []),
    "fastocr_profile_begin": (C.c_int, [C.c_void_p, C.c_int32, C.c_int]),
    "fastocr_profile_end": (C.c_int, [C.c_void_p, C.c_void_p, C.c_void_p]),
    "fastocr_launch_count": (C.c_int64, []),
    "fastocr_cluster_launch_count": (C.c_int64, []),
}

_lib = None


def load() -> C.CDLL:
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise ImportError(
                f"{LIB_PATH} is missing: build it with `python -m paper_2605_17447_b200.build` "
                "(nvcc, sm_100a). There is no CPU or PyTorch fallback.")
        lib = C.CDLL(LIB_PATH)
        for name, (res, args) in EXPORTS.items():
            fn = getattr(lib, name)
            fn.restype = res
            fn.argtypes = args
        _lib = lib
    return _lib
