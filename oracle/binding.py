"""ctypes wrapper over libfastocr_oracle.so (test infrastructure; see fastocr_oracle.cpp).

Tensors are torch CPU tensors: q [H][d], K/V [S][Hkv][d] in bf16; outputs fp32.
"""
from __future__ import annotations

import ctypes as C
import os

import numpy as np
import torch

from . import build as _build

_lib = C.CDLL(_build.build())
try:
    _omp = C.CDLL("libgomp.so.1")
except OSError:  # pragma: no cover
    _omp = None

_u16p, _f32p, _i32p, _u8p, _f64p = (C.c_void_p,) * 5
_lib.fastocr_oracle_dense.argtypes = [_u16p, _u16p, _u16p, C.c_int, C.c_int, C.c_int, C.c_int, C.c_float, C.c_int, _f32p]
_lib.fastocr_oracle_probs.argtypes = [_u16p, _u16p, C.c_int, C.c_int, C.c_int, C.c_int, C.c_float, C.c_int, _f32p]
_lib.fastocr_oracle_scores.argtypes = [_u16p, _u16p, C.c_int, C.c_int, C.c_int, C.c_int, C.c_float, C.c_int, C.c_int, C.c_int, _f32p, _f32p]
_lib.fastocr_oracle_topk.argtypes = [_f32p, C.c_int, C.c_int, _i32p]
_lib.fastocr_oracle_sparse.argtypes = [_u16p, _u16p, _u16p, C.c_int, C.c_int, C.c_int, C.c_int, C.c_float, C.c_int, C.c_int, _i32p, C.c_int, C.c_int, _f32p]
_lib.fastocr_oracle_masked_dense.argtypes = [_u16p, _u16p, _u16p, C.c_int, C.c_int, C.c_int, C.c_int, C.c_float, _u8p, _f32p]
_lib.fastocr_oracle_kept_count.argtypes = [C.c_int, C.c_double]
_lib.fastocr_oracle_focal_layers.argtypes = [_f64p, C.c_int, C.c_double, C.c_int, _i32p]
_lib.fastocr_oracle_attn_flops.argtypes = [C.c_double] * 4
_lib.fastocr_oracle_attn_flops.restype = C.c_double
_lib.fastocr_oracle_attn_flops_pruned.argtypes = [C.c_double] * 6
_lib.fastocr_oracle_attn_flops_pruned.restype = C.c_double


def set_threads(n: int) -> None:
    if _omp is not None:
        _omp.omp_set_num_threads(int(n))


def num_threads() -> int:
    return int(_omp.omp_get_max_threads()) if _omp is not None else 1


def _bf16(t: torch.Tensor) -> torch.Tensor:
    assert t.dtype == torch.bfloat16 and t.device.type == "cpu"
    return t.contiguous()


def _check(rc: int, what: str) -> None:
    if rc != 0:
        raise ValueError(f"oracle {what}: invalid arguments (code {rc})")


def _shape(q, K):
    H, d = q.shape
    S, Hkv, d2 = K.shape
    assert d == d2
    return S, H, Hkv, d


def dense(q, K, V, sm_scale: float, acc64: bool = False) -> torch.Tensor:
    q, K, V = _bf16(q), _bf16(K), _bf16(V)
    S, H, Hkv, d = _shape(q, K)
    out = torch.empty(H, d, dtype=torch.float32)
    _check(_lib.fastocr_oracle_dense(q.data_ptr(), K.data_ptr(), V.data_ptr(), S, H, Hkv, d, sm_scale, int(acc64), out.data_ptr()), "dense")
    return out


def probs(q, K, sm_scale: float, acc64: bool = False) -> torch.Tensor:
    q, K = _bf16(q), _bf16(K)
    S, H, Hkv, d = _shape(q, K)
    out = torch.empty(H, S, dtype=torch.float32)
    _check(_lib.fastocr_oracle_probs(q.data_ptr(), K.data_ptr(), S, H, Hkv, d, sm_scale, int(acc64), out.data_ptr()), "probs")
    return out


def scores(q, K, sm_scale: float, vis_start: int, N: int, acc64: bool = False):
    """-> (scores [N] fp32, image_mass float)"""
    q, K = _bf16(q), _bf16(K)
    S, H, Hkv, d = _shape(q, K)
    out = torch.empty(max(N, 0), dtype=torch.float32)
    mass = C.c_float(0)
    _check(_lib.fastocr_oracle_scores(q.data_ptr(), K.data_ptr(), S, H, Hkv, d, sm_scale, vis_start, N, int(acc64), out.data_ptr(), C.addressof(mass)), "scores")
    return out, float(mass.value)


def topk(score: torch.Tensor, k: int) -> torch.Tensor:
    s = score.to(torch.float32).contiguous()
    out = torch.empty(max(k, 0), dtype=torch.int32)
    _check(_lib.fastocr_oracle_topk(s.data_ptr(), s.numel(), k, out.data_ptr()), "topk")
    return out


def sparse(q, K, V, sm_scale: float, vis_start: int, N: int, idx: torch.Tensor, acc64: bool = False) -> torch.Tensor:
    q, K, V = _bf16(q), _bf16(K), _bf16(V)
    S, H, Hkv, d = _shape(q, K)
    idx = idx.to(torch.int32).contiguous()
    out = torch.empty(H, d, dtype=torch.float32)
    _check(_lib.fastocr_oracle_sparse(q.data_ptr(), K.data_ptr(), V.data_ptr(), S, H, Hkv, d, sm_scale, vis_start, N, idx.data_ptr(), idx.numel(), int(acc64), out.data_ptr()), "sparse")
    return out


def masked_dense(q, K, V, sm_scale: float, keep: torch.Tensor) -> torch.Tensor:
    q, K, V = _bf16(q), _bf16(K), _bf16(V)
    S, H, Hkv, d = _shape(q, K)
    keep = keep.to(torch.uint8).contiguous()
    assert keep.numel() == S
    out = torch.empty(H, d, dtype=torch.float32)
    _check(_lib.fastocr_oracle_masked_dense(q.data_ptr(), K.data_ptr(), V.data_ptr(), S, H, Hkv, d, sm_scale, keep.data_ptr(), out.data_ptr()), "masked_dense")
    return out


def kept_count(N: int, tau: float) -> int:
    return int(_lib.fastocr_oracle_kept_count(int(N), float(tau)))


def focal_layers(mean_ratio, rho: float, gap: int):
    r = np.ascontiguousarray(np.asarray(mean_ratio, dtype=np.float64))
    out = np.empty(max(len(r), 1), dtype=np.int32)
    n = _lib.fastocr_oracle_focal_layers(r.ctypes.data, len(r), float(rho), int(gap), out.ctypes.data)
    return [int(x) for x in out[:n]]


def attn_flops(b, l, h, s) -> float:
    return float(_lib.fastocr_oracle_attn_flops(float(b), float(l), float(h), float(s)))


def attn_flops_pruned(b, l, h, s, full_layers, s_kept) -> float:
    return float(_lib.fastocr_oracle_attn_flops_pruned(float(b), float(l), float(h), float(s), float(full_layers), float(s_kept)))
