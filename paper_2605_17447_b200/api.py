"""Python names for the C entry points of include/fastocr.h (argument marshalling only).

Tensors are torch CUDA tensors used as device buffers; the functions pass their data pointers and
the current torch stream to the library and return nothing (results land in the output tensors,
asynchronously on that stream).
"""
from __future__ import annotations

import ctypes as C
from dataclasses import dataclass
from typing import Optional, Sequence

import numpy as np
import torch

from . import _lib

_STATUS = {1: "invalid argument", 2: "unsupported", 3: "workspace limits exceeded", 4: "CUDA error"}


PROF_CLASSES = ("attn_dense", "attn_keys", "attn_sparse", "scores_finalize", "select_topk", "image_mass")


class FastOCRError(RuntimeError):
    def __init__(self, code: int, msg: str):
        super().__init__(f"fastocr: {_STATUS.get(code, code)}: {msg}")
        self.code = code


def _ptr(t: Optional[torch.Tensor]):
    return None if t is None else C.c_void_p(t.data_ptr())


def _stream(stream=None):
    s = torch.cuda.current_stream() if stream is None else stream
    return C.c_void_p(s.cuda_stream)


def _dev(t: torch.Tensor, dtype, what: str) -> torch.Tensor:
    if not t.is_cuda or t.dtype != dtype or not t.is_contiguous():
        raise TypeError(f"{what}: need a contiguous CUDA tensor of {dtype}")
    return t


@dataclass
class KVView:
    """One layer's cache for a batch (see fastocr_kv_view). k/v: bf16 CUDA tensors, contiguous
    [B][seq_stride][Hkv][128] or paged [num_pages][page_size][Hkv][128]."""
    k: torch.Tensor
    v: Optional[torch.Tensor]
    seq_len: torch.Tensor          # int32 CUDA [B]
    vis_start: torch.Tensor        # int32 CUDA [B]
    vis_len: torch.Tensor          # int32 CUDA [B]
    num_q_heads: int
    max_seq_len: int
    sm_scale: float
    block_table: Optional[torch.Tensor] = None   # int32 CUDA [B][max_pages] when paged
    num_pages: int = -1            # paged: pages in the pools (block-table entries are clamped to it); -1: k.shape[0]

    def struct(self) -> _lib.KVViewStruct:
        _dev(self.k, torch.bfloat16, "k")
        if self.v is not None:
            _dev(self.v, torch.bfloat16, "v")
        for name in ("seq_len", "vis_start", "vis_len"):
            _dev(getattr(self, name), torch.int32, name)
        s = _lib.KVViewStruct()
        s.batch = int(self.seq_len.numel())
        s.num_q_heads = int(self.num_q_heads)
        s.num_kv_heads = int(self.k.shape[2])
        s.head_dim = int(self.k.shape[3])
        s.max_seq_len = int(self.max_seq_len)
        s.k = self.k.data_ptr()
        s.v = self.v.data_ptr() if self.v is not None else None
        if self.block_table is not None:
            _dev(self.block_table, torch.int32, "block_table")
            s.page_size = int(self.k.shape[1])
            s.block_table = self.block_table.data_ptr()
            s.max_pages = int(self.block_table.shape[1])
            s.num_pages = int(self.k.shape[0]) if self.num_pages < 0 else int(self.num_pages)
            s.seq_stride_tokens = 0
        else:
            s.page_size = 0
            s.seq_stride_tokens = int(self.k.shape[1])
        s.seq_len = self.seq_len.data_ptr()
        s.vis_start = self.vis_start.data_ptr()
        s.vis_len = self.vis_len.data_ptr()
        s.sm_scale = float(self.sm_scale)
        return s


class Context:
    """Owns a fastocr_ctx (workspace on one device)."""

    def __init__(self, max_batch: int, num_q_heads: int, num_kv_heads: int, max_seq_len: int, max_vis_len: int,
                 device: Optional[int] = None):
        self._lib = _lib.load()
        if not torch.cuda.is_available():
            raise RuntimeError("fastocr needs a CUDA device (B200, sm_100a); there is no CPU path")
        self.device = torch.cuda.current_device() if device is None else int(device)
        lim = _lib.LimitsStruct(max_batch, num_q_heads, num_kv_heads, max_seq_len, max_vis_len)
        h = C.c_void_p()
        rc = self._lib.fastocr_create(C.byref(h), self.device, C.byref(lim))
        if rc != 0:
            raise FastOCRError(rc, "fastocr_create failed")
        self._h = h
        self.max_vis_len = max_vis_len

    def close(self):
        if getattr(self, "_h", None):
            self._lib.fastocr_destroy(self._h)
            self._h = None

    def __del__(self):  # pragma: no cover
        try:
            self.close()
        except Exception:
            pass

    def check(self, rc: int):
        if rc != 0:
            raise FastOCRError(rc, self._lib.fastocr_last_error(self._h).decode())

    def device_faults(self) -> int:
        return int(self._lib.fastocr_device_faults(self._h))

    def profile_begin(self, max_launches: int, coalesce_runs: bool = False) -> None:
        """coalesce_runs: time maximal runs of same-class launches as one interval (in-situ durations)
        instead of every launch on its own (isolated durations)."""
        self.check(self._lib.fastocr_profile_begin(self._h, int(max_launches), int(bool(coalesce_runs))))

    def profile_end(self):
        """-> {class name: (total ms, launches)} for the launches since profile_begin."""
        ms = (C.c_double * len(PROF_CLASSES))()
        n = (C.c_int64 * len(PROF_CLASSES))()
        self.check(self._lib.fastocr_profile_end(self._h, ms, n))
        return {name: (float(ms[i]), int(n[i])) for i, name in enumerate(PROF_CLASSES)}


def kept_count(n_vis: int, tau: float) -> int:
    return int(_lib.load().fastocr_kept_count(int(n_vis), float(tau)))


def focal_layers(mean_ratio: Sequence[float], rho: float, gap: int):
    r = np.ascontiguousarray(np.asarray(mean_ratio, dtype=np.float64))
    out = np.zeros(max(len(r), 1), dtype=np.int32)
    n = _lib.load().fastocr_focal_layers(r.ctypes.data, len(r), float(rho), int(gap), out.ctypes.data)
    if n < 0:
        raise FastOCRError(1, "fastocr_focal_layers: invalid arguments")
    return [int(x) for x in out[:n]]


def attn_flops(batch, layers, hidden, seq_len) -> float:
    return float(_lib.load().fastocr_attn_flops(float(batch), float(layers), float(hidden), float(seq_len)))


def attn_flops_pruned(batch, layers, hidden, seq_len, full_layers, kept_len) -> float:
    return float(_lib.load().fastocr_attn_flops_pruned(float(batch), float(layers), float(hidden), float(seq_len),
                                                       float(full_layers), float(kept_len)))


def launch_count() -> int:
    return int(_lib.load().fastocr_launch_count())


def cluster_launch_count() -> int:
    return int(_lib.load().fastocr_cluster_launch_count())


def fastocr_dense_decode_attn(ctx: Context, kv: KVView, q: torch.Tensor, out: torch.Tensor,
                              scores_out: Optional[torch.Tensor] = None, image_mass_out: Optional[torch.Tensor] = None,
                              stream=None) -> None:
    _dev(q, torch.bfloat16, "q")
    st = kv.struct()
    n_stride = int(scores_out.shape[-1]) if scores_out is not None else 0
    if scores_out is not None:
        _dev(scores_out, torch.float32, "scores_out")
    if image_mass_out is not None:
        _dev(image_mass_out, torch.float32, "image_mass_out")
    ctx.check(ctx._lib.fastocr_dense_decode_attn(ctx._h, C.byref(st), _ptr(q), _ptr(out), int(out.dtype == torch.float32),
                                                 _ptr(scores_out), n_stride, _ptr(image_mass_out), _stream(stream)))


def fastocr_focal_scores(ctx: Context, kv: KVView, q: torch.Tensor, scores_out: torch.Tensor,
                         image_mass_out: Optional[torch.Tensor] = None, stream=None) -> None:
    _dev(q, torch.bfloat16, "q")
    _dev(scores_out, torch.float32, "scores_out")
    st = kv.struct()
    ctx.check(ctx._lib.fastocr_focal_scores(ctx._h, C.byref(st), _ptr(q), _ptr(scores_out), int(scores_out.shape[-1]),
                                            _ptr(image_mass_out), _stream(stream)))


def fastocr_select_topk(ctx: Context, scores: torch.Tensor, vis_len: torch.Tensor, k: torch.Tensor,
                        idx_out: torch.Tensor, max_vis_len: int, stream=None) -> None:
    _dev(scores, torch.float32, "scores")
    _dev(vis_len, torch.int32, "vis_len")
    _dev(k, torch.int32, "k")
    _dev(idx_out, torch.int32, "idx_out")
    ctx.check(ctx._lib.fastocr_select_topk(ctx._h, _ptr(scores), int(scores.shape[-1]), _ptr(vis_len), _ptr(k),
                                           int(vis_len.numel()), int(max_vis_len), _ptr(idx_out),
                                           int(idx_out.shape[-1]), _stream(stream)))


def fastocr_sparse_decode_attn(ctx: Context, kv: KVView, q: torch.Tensor, idx: torch.Tensor, k: torch.Tensor,
                               out: torch.Tensor, max_kept: int = 0, stream=None) -> None:
    _dev(q, torch.bfloat16, "q")
    _dev(idx, torch.int32, "idx")
    _dev(k, torch.int32, "k")
    st = kv.struct()
    ctx.check(ctx._lib.fastocr_sparse_decode_attn(ctx._h, C.byref(st), _ptr(q), _ptr(idx), _ptr(k), int(idx.shape[-1]),
                                                  int(max_kept), _ptr(out), int(out.dtype == torch.float32),
                                                  _stream(stream)))


def fastocr_sparse_decode_attn_noalloc(kv: KVView, q: torch.Tensor, idx: torch.Tensor, k: torch.Tensor,
                                       out: torch.Tensor, stream=None) -> None:
    """Pruned attention for callers that may not allocate: no Context, the library's built-in scratch
    array is used (batch * num_kv_heads <= 256; calls on one device must not overlap on the GPU)."""
    _dev(q, torch.bfloat16, "q")
    _dev(idx, torch.int32, "idx")
    _dev(k, torch.int32, "k")
    lib = _lib.load()
    st = kv.struct()
    rc = lib.fastocr_sparse_decode_attn_noalloc(C.byref(st), _ptr(q), _ptr(idx), _ptr(k), int(idx.shape[-1]), _ptr(out),
                                                int(out.dtype == torch.float32), _stream(stream))
    if rc != 0:
        raise FastOCRError(rc, lib.fastocr_noalloc_last_error().decode())


class _DeviceFloats:
    """A span of device fp32 memory owned by the library, described through the CUDA array interface."""

    def __init__(self, ptr: int, shape):
        self.__cuda_array_interface__ = {"shape": tuple(int(x) for x in shape), "typestr": "<f4", "data": (int(ptr), False),
                                         "strides": None, "version": 2}


class _StepArgs:
    """Marshalled arguments of fastocr_decode_step_ex that do not change between steps."""

    def __init__(self, layers: Sequence[KVView], is_focal, k: torch.Tensor, fixation: torch.Tensor, max_vis_len: int,
                 max_kept: int, union_sets: bool, scores_exchange=None):
        self.L = len(layers)
        self.keep = (list(layers), k, fixation)
        self.arr = (_lib.KVViewStruct * self.L)(*[kv.struct() for kv in layers])
        focal = np.ascontiguousarray(np.asarray(is_focal, dtype=np.uint8))
        self.opt = _lib.StepOptionsStruct(None, None, int(bool(union_sets)))
        self.exchange_error = None
        if scores_exchange is not None:
            device = k.device

            def hook(ptr, batch, n_stride, layer, stream, user):
                # the library's score workspace as a tensor (no copy); the callable enqueues on the current stream
                try:
                    scores = torch.as_tensor(_DeviceFloats(ptr, (batch, n_stride)), device=device)
                    scores_exchange(scores, layer)
                    return 0
                except BaseException as e:      # must not propagate through the C frames
                    self.exchange_error = e
                    return 1

            self._hook = _lib.ScoresExchangeFn(hook)   # kept alive with the arguments
            self.opt.scores_exchange = self._hook
        self.focal = focal
        self.focal_ptr = focal.ctypes.data
        if focal.ndim == 2:                       # per-sequence focal layer sets [L][B]: host copy + device copy
            if focal.shape != (self.L, int(k.numel())):
                raise ValueError("per-sequence focal sets must be [layers][batch]")
            self.focal_dev = torch.from_numpy(focal).to(k.device)
            self.opt.is_focal_seq = focal.ctypes.data
            self.opt.is_focal_seq_dev = self.focal_dev.data_ptr()
            self.focal_ptr = None
        elif focal.shape != (self.L,):
            raise ValueError("is_focal must have one entry per layer")
        self.k = _ptr(_dev(k, torch.int32, "k"))
        self.fix = _ptr(_dev(fixation, torch.int32, "fixation"))
        self.k_stride = int(fixation.shape[-1])
        self.max_vis, self.max_kept = int(max_vis_len), int(max_kept)
        self.have = C.c_int(0)

    def run(self, ctx: Context, q: torch.Tensor, out: torch.Tensor, has_fixation: bool, stream=None) -> bool:
        rc = ctx._lib.fastocr_decode_step_ex(ctx._h, self.L, self.arr, C.c_void_p(q.data_ptr()), C.c_void_p(out.data_ptr()),
                                             int(out.dtype == torch.float32), self.focal_ptr, self.k, self.fix,
                                             self.k_stride, int(bool(has_fixation)), self.max_vis, self.max_kept,
                                             C.byref(self.have), C.byref(self.opt), _stream(stream))
        if self.exchange_error is not None:             # what the exchange callable raised, not the library's summary of it
            e, self.exchange_error = self.exchange_error, None
            raise e
        ctx.check(rc)
        return bool(self.have.value)


def noalloc_device_faults() -> int:
    """Values the allocation-free entry point's kernels have had to force into range on the current device."""
    return int(_lib.load().fastocr_noalloc_device_faults())


def fastocr_decode_step(ctx: Context, layers: Sequence[KVView], q: torch.Tensor, out: torch.Tensor,
                        is_focal, k: torch.Tensor, fixation: torch.Tensor, has_fixation: bool,
                        max_vis_len: int, max_kept: int = 0, union_sets: bool = False, stream=None,
                        scores_exchange=None) -> bool:
    """q/out: [L][B][H][128]. is_focal: [L] (one focal layer set for the batch) or [L][B] (per-sequence
    sets). scores_exchange: for heads sharded over processes, a callable (scores [B][n_stride] device
    fp32, layer) that sums the scores over the ranks in place on the current stream (see
    sharding.make_scores_exchange); the step must then run on the current stream. Returns whether
    `fixation` is valid after the step."""
    _dev(q, torch.bfloat16, "q")
    return _StepArgs(layers, is_focal, k, fixation, max_vis_len, max_kept, union_sets, scores_exchange).run(
        ctx, q, out, has_fixation, stream)


def fastocr_warmup_step(ctx: Context, layers: Sequence[KVView], q: torch.Tensor, out: torch.Tensor,
                        ratio_out: torch.Tensor, stream=None) -> None:
    """One warm-up step: every layer dense, Eq. 1's ratio of layer l and sequence b into ratio_out[l][b]."""
    _dev(q, torch.bfloat16, "q")
    _dev(ratio_out, torch.float32, "ratio_out")
    L = len(layers)
    arr = (_lib.KVViewStruct * L)(*[kv.struct() for kv in layers])
    ctx.check(ctx._lib.fastocr_warmup_step(ctx._h, L, arr, _ptr(q), _ptr(out), int(out.dtype == torch.float32),
                                           _ptr(ratio_out), _stream(stream)))


class StepPlan:
    """fastocr_decode_step with everything that does not change between steps marshalled once
    (the per-step Python cost is then a single foreign call)."""

    def __init__(self, ctx: Context, layers: Sequence[KVView], is_focal, k: torch.Tensor,
                 fixation: torch.Tensor, max_vis_len: int, max_kept: int = 0, union_sets: bool = False,
                 scores_exchange=None):
        self.ctx = ctx
        self.L = len(layers)
        self._args = _StepArgs(layers, is_focal, k, fixation, max_vis_len, max_kept, union_sets, scores_exchange)

    def run(self, q: torch.Tensor, out: torch.Tensor, has_fixation: bool, stream=None) -> bool:
        return self._args.run(self.ctx, q, out, has_fixation, stream)
