"""ctypes binding of libheadcast.so: argument marshalling only.

Every method mirrors the C entry point of the same name in include/headcast.h; tensors are torch
CUDA tensors whose ``data_ptr()`` is handed to the library, and the current torch stream is passed
along.  There is no fallback: if the library is missing or a call fails, an exception is raised.
"""
from __future__ import annotations

import ctypes as C
import os
from typing import Optional, Sequence

from . import build as _build

SINK, DUMMY, SPATIAL, GLOBAL = 0, 1, 2, 3
N_SCORES = 10
ERRORS = {0: "HC_OK", -1: "HC_ERR_INVALID_ARG", -2: "HC_ERR_STATE", -3: "HC_ERR_CUDA", -4: "HC_ERR_NOMEM",
          -5: "HC_ERR_UNSUPPORTED", -6: "HC_ERR_TIMEOUT"}

EXPORTS = ("headcast_default_config", "headcast_create", "headcast_destroy", "headcast_append",
           "headcast_full_attend", "headcast_classify", "headcast_set_labels", "headcast_get_labels",
           "headcast_split_cache", "headcast_attend", "headcast_export_cache", "headcast_n_filled",
           "headcast_launch_count", "headcast_attend_flops", "headcast_check", "headcast_last_error",
           "headcast_set_kernel_timing", "headcast_last_attention_kernel_ms", "headcast_set_tracing",
           "headcast_read_trace", "headcast_dense_attend_noalloc", "headcast_noalloc_status",
           "headcast_noalloc_last_error", "headcast_plan_schedule", "headcast_selftest_bounded_wait", "headcast_overwrite_last",
           "headcast_append_host", "headcast_attend_host")


class Config(C.Structure):
    _fields_ = [("n_heads", C.c_int32), ("head_dim", C.c_int32), ("grid_h", C.c_int32), ("grid_w", C.c_int32),
                ("frames_per_block", C.c_int32), ("n_blocks", C.c_int32), ("cell_h", C.c_int32),
                ("cell_w", C.c_int32), ("row_edges_host", C.POINTER(C.c_int32)), ("n_row_edges", C.c_int32),
                ("col_edges_host", C.POINTER(C.c_int32)), ("n_col_edges", C.c_int32),
                ("proxy_radius", C.c_int32), ("theta_sink", C.c_float), ("theta_dummy", C.c_float),
                ("theta_spatial", C.c_float), ("theta_score", C.c_float), ("gamma", C.c_float),
                ("softmax_scale", C.c_float), ("keep_monolithic", C.c_int32), ("sd_mode", C.c_int32),
                ("rule", C.c_int32), ("mass_tau", C.c_float)]

RULE_COSINE, RULE_MASS = 0, 1


class HeadCastError(RuntimeError):
    def __init__(self, code: int, message: str):
        super().__init__(f"{ERRORS.get(code, code)}: {message}")
        self.code = code


_lib = None


def load_library(path: Optional[str] = None) -> C.CDLL:
    """Loads (building first if the sources are newer) libheadcast.so and declares the prototypes."""
    global _lib
    if _lib is not None and path is None:
        return _lib
    lib = C.CDLL(path or _build.build())
    vp, i32p, f32p = C.c_void_p, C.POINTER(C.c_int32), C.POINTER(C.c_float)
    lib.headcast_default_config.argtypes = [C.POINTER(Config)]
    lib.headcast_default_config.restype = None
    lib.headcast_create.argtypes = [C.POINTER(Config), C.POINTER(vp)]
    lib.headcast_destroy.argtypes = [vp]
    lib.headcast_append.argtypes = [vp, vp, vp, vp]
    lib.headcast_full_attend.argtypes = [vp, vp, vp, vp]
    lib.headcast_overwrite_last.argtypes = [vp, vp, vp, vp]
    lib.headcast_classify.argtypes = [vp, vp, i32p, f32p, vp]
    lib.headcast_set_labels.argtypes = [vp, i32p]
    lib.headcast_get_labels.argtypes = [vp, i32p]
    lib.headcast_split_cache.argtypes = [vp, vp]
    lib.headcast_attend.argtypes = [vp, vp, vp, vp]
    lib.headcast_append_host.argtypes = [vp, vp, vp, vp]
    lib.headcast_attend_host.argtypes = [vp, vp, vp, vp]
    lib.headcast_export_cache.argtypes = [vp, C.c_int32, vp, vp, i32p, vp]
    lib.headcast_n_filled.argtypes = [vp]
    lib.headcast_launch_count.argtypes = [vp]
    lib.headcast_launch_count.restype = C.c_int64
    lib.headcast_attend_flops.argtypes = [vp, C.c_int32]
    lib.headcast_attend_flops.restype = C.c_double
    lib.headcast_check.argtypes = [vp, vp]
    lib.headcast_set_kernel_timing.argtypes = [vp, C.c_int32]
    lib.headcast_last_attention_kernel_ms.argtypes = [vp, f32p]
    lib.headcast_set_tracing.argtypes = [vp, C.c_int32]
    lib.headcast_read_trace.argtypes = [vp, C.POINTER(C.c_int64), C.c_int32, i32p]
    lib.headcast_dense_attend_noalloc.argtypes = [vp, vp, vp, vp, C.c_int32, C.c_int32, C.c_int32, C.c_int32, C.c_float, vp]
    lib.headcast_noalloc_status.argtypes = [vp]
    lib.headcast_selftest_bounded_wait.argtypes = [vp, C.c_int32, vp]
    lib.headcast_plan_schedule.argtypes = [C.POINTER(Config), i32p, C.c_int32, C.c_int32, C.c_int32, i32p, C.c_int32, i32p, i32p]
    lib.headcast_noalloc_last_error.argtypes = []
    lib.headcast_noalloc_last_error.restype = C.c_char_p
    lib.headcast_last_error.argtypes = [vp]
    lib.headcast_last_error.restype = C.c_char_p
    if path is None:
        _lib = lib
    return lib


def default_config(**kw) -> Config:
    cfg = Config()
    load_library().headcast_default_config(C.byref(cfg))
    for k, v in kw.items():
        setattr(cfg, k, v)
    return cfg


def _stream() -> int:
    import torch
    return torch.cuda.current_stream().cuda_stream


def _validate(t, name: str, shape, cuda: bool = True) -> None:
    """Rejects, before the library sees a pointer, any tensor that would make a kernel read or write outside the
    caller's buffer: wrong dtype, rank, shape, device or a non-contiguous view.  ``shape`` entries of None are free."""
    import torch
    if not isinstance(t, torch.Tensor):
        raise ValueError(f"{name}: expected a torch tensor, got {type(t).__name__}")
    if t.dtype != torch.bfloat16:
        raise ValueError(f"{name}: dtype must be bfloat16, got {t.dtype}")
    if t.dim() != len(shape) or any(want is not None and int(got) != int(want) for got, want in zip(t.shape, shape)):
        raise ValueError(f"{name}: shape must be {tuple(shape)}, got {tuple(t.shape)}")
    if not t.is_contiguous():
        raise ValueError(f"{name}: must be contiguous")
    if cuda:
        if not t.is_cuda:
            raise ValueError(f"{name}: must be a CUDA tensor")
        if t.device.index != torch.cuda.current_device():
            raise ValueError(f"{name}: lives on cuda:{t.device.index}, the current device is cuda:{torch.cuda.current_device()}")
    elif t.is_cuda:
        raise ValueError(f"{name}: the host entry points take CPU tensors")


def _ptr(t, name: str = "tensor", shape=None) -> int:
    if shape is not None:
        _validate(t, name, shape)
    elif not (t.is_cuda and t.is_contiguous()):
        raise ValueError(f"{name}: tensors handed to the library must be contiguous CUDA tensors")
    return t.data_ptr()


def _host_ptr(t, name: str = "tensor", shape=None) -> int:
    if shape is not None:
        _validate(t, name, shape, cuda=False)
    elif t.is_cuda or not t.is_contiguous():
        raise ValueError(f"{name}: host entry points take contiguous CPU tensors")
    return t.data_ptr()


ITEM_FIELDS = ("head", "cell", "q_start0", "q_start1", "q_count0", "q_count1", "kv_map", "kv_x0", "kv_row0", "seg_stride",
               "seg_len", "tiles_per_seg", "tile_begin", "tile_end", "out_mode", "out_slot")


def plan_schedule(cfg: Config, labels: Optional[Sequence[int]], n_filled: int, n_ctas: int = 148, dense: bool = False):
    """Host-only: the work list of headcast_attend / headcast_full_attend as (items [n, 16] int32 with columns
    ITEM_FIELDS, cta_first [n_ctas + 1] int32)."""
    import numpy as np
    lib = load_library()
    lab = None if labels is None else (C.c_int32 * cfg.n_heads)(*[int(v) for v in labels])
    n = C.c_int32()
    rc = lib.headcast_plan_schedule(C.byref(cfg), lab, n_filled, n_ctas, int(dense), None, 0, C.byref(n), None)
    if rc != 0:
        raise HeadCastError(rc, "headcast_plan_schedule")
    items = np.zeros((max(n.value, 1), 16), dtype=np.int32)
    first = np.zeros(n_ctas + 1, dtype=np.int32)
    rc = lib.headcast_plan_schedule(C.byref(cfg), lab, n_filled, n_ctas, int(dense), items.ctypes.data_as(C.POINTER(C.c_int32)),
                                    n.value, C.byref(n), first.ctypes.data_as(C.POINTER(C.c_int32)))
    if rc != 0:
        raise HeadCastError(rc, "headcast_plan_schedule")
    return items[: n.value], first


def dense_attend_noalloc(q, k, v, out, softmax_scale: float = 0.0) -> None:
    """Dense attention of q [Lq, H, d] over k, v [Lk, H, d] into out [Lq, H, d] (bf16 CUDA tensors) through the
    library's allocation-free entry point: for hosts that cannot let the library allocate device memory (a server
    whose own pool owns the GPU, a loop that cannot take an allocation's device-wide synchronisation).  Calls on
    one GPU share a fixed scratch array inside the library: keep them on one stream.  Sizes beyond
    n_heads * ceil(Lq / 256) <= 2048 are rejected."""
    lib = load_library()
    if getattr(q, "ndim", 0) != 3 or getattr(k, "ndim", 0) != 3:
        raise ValueError("q and k must be [rows, heads, head_dim]")
    n_q, h, d = q.shape
    n_k = k.shape[0]
    rc = lib.headcast_dense_attend_noalloc(_ptr(q, "q", (n_q, h, d)), _ptr(k, "k", (n_k, h, d)), _ptr(v, "v", (n_k, h, d)),
                                           _ptr(out, "out", (n_q, h, d)), n_q, n_k, h, d, float(softmax_scale), _stream())
    if rc != 0:
        raise HeadCastError(rc, lib.headcast_noalloc_last_error().decode())


def noalloc_status() -> None:
    """Synchronises the current stream and raises if the allocation-free kernel reported a bounded-wait expiry."""
    lib = load_library()
    rc = lib.headcast_noalloc_status(_stream())
    if rc != 0:
        raise HeadCastError(rc, lib.headcast_noalloc_last_error().decode())


class HeadCast:
    """One attention layer's HeadCast context (wraps headcast_ctx*)."""

    def __init__(self, n_heads: int, head_dim: int, grid_h: int, grid_w: int, n_blocks: int,
                 frames_per_block: int = 3, cell_h: int = 10, cell_w: int = 10, keep_monolithic: bool = False,
                 row_edges: Optional[Sequence[int]] = None, col_edges: Optional[Sequence[int]] = None, **overrides):
        self.lib = load_library()
        cfg = default_config(n_heads=n_heads, head_dim=head_dim, grid_h=grid_h, grid_w=grid_w, n_blocks=n_blocks,
                             frames_per_block=frames_per_block, cell_h=cell_h, cell_w=cell_w,
                             keep_monolithic=int(keep_monolithic), **overrides)
        keep = []
        if row_edges is not None:
            arr = (C.c_int32 * len(row_edges))(*row_edges)
            keep.append(arr)
            cfg.row_edges_host, cfg.n_row_edges = arr, len(row_edges)
        if col_edges is not None:
            arr = (C.c_int32 * len(col_edges))(*col_edges)
            keep.append(arr)
            cfg.col_edges_host, cfg.n_col_edges = arr, len(col_edges)
        self.cfg = cfg
        self.n_heads, self.head_dim = n_heads, head_dim
        self.block_tokens = frames_per_block * grid_h * grid_w
        self.n_blocks = n_blocks
        self._ctx = C.c_void_p()
        rc = self.lib.headcast_create(C.byref(cfg), C.byref(self._ctx))
        if rc != 0:
            self._ctx = C.c_void_p()
            raise HeadCastError(rc, "headcast_create failed")

    @classmethod
    def from_workload(cls, w, **kw) -> "HeadCast":
        return cls(w.n_heads, w.head_dim, w.grid_h, w.grid_w, w.n_blocks, w.frames_per_block, w.cell_h, w.cell_w, **kw)

    @property
    def _block(self):
        return (self.block_tokens, self.n_heads, self.head_dim)

    def _check(self, rc: int) -> None:
        if rc != 0:
            raise HeadCastError(rc, self.lib.headcast_last_error(self._ctx).decode())

    def destroy(self) -> None:
        if self._ctx:
            self.lib.headcast_destroy(self._ctx)
            self._ctx = C.c_void_p()

    def __del__(self):
        try:
            self.destroy()
        except Exception:
            pass

    def append(self, k_new, v_new) -> None:
        self._check(self.lib.headcast_append(self._ctx, _ptr(k_new, "k_new", self._block), _ptr(v_new, "v_new", self._block), _stream()))

    def overwrite_last(self, k_new, v_new) -> None:
        self._check(self.lib.headcast_overwrite_last(self._ctx, _ptr(k_new, "k_new", self._block), _ptr(v_new, "v_new", self._block), _stream()))

    def full_attend(self, q, out) -> None:
        self._check(self.lib.headcast_full_attend(self._ctx, _ptr(q, "q", self._block), _ptr(out, "out", self._block), _stream()))

    def classify(self, q):
        import numpy as np
        labels = (C.c_int32 * self.n_heads)()
        scores = (C.c_float * (self.n_heads * N_SCORES))()
        self._check(self.lib.headcast_classify(self._ctx, _ptr(q, "q", self._block), labels, scores, _stream()))
        return (np.array(labels[:], dtype=np.int32),
                np.array(scores[:], dtype=np.float32).reshape(self.n_heads, N_SCORES))

    def set_labels(self, labels: Sequence[int]) -> None:
        if len(labels) != self.n_heads:
            raise ValueError(f"labels: expected {self.n_heads} entries, got {len(labels)}")
        arr = (C.c_int32 * self.n_heads)(*[int(v) for v in labels])
        self._check(self.lib.headcast_set_labels(self._ctx, arr))

    def get_labels(self):
        arr = (C.c_int32 * self.n_heads)()
        self._check(self.lib.headcast_get_labels(self._ctx, arr))
        return list(arr)

    def split_cache(self) -> None:
        self._check(self.lib.headcast_split_cache(self._ctx, _stream()))

    def attend(self, q, out) -> None:
        self._check(self.lib.headcast_attend(self._ctx, _ptr(q, "q", self._block), _ptr(out, "out", self._block), _stream()))

    def append_host(self, k_host, v_host) -> None:
        """k_host / v_host: CPU tensors (pinned for overlap) of shape [L, H, d], bf16."""
        self._check(self.lib.headcast_append_host(self._ctx, _host_ptr(k_host, "k_host", self._block), _host_ptr(v_host, "v_host", self._block), _stream()))

    def attend_host(self, q_host, out_host) -> None:
        """q_host / out_host: CPU tensors (pinned for overlap); out_host is complete after the stream is synchronised."""
        self._check(self.lib.headcast_attend_host(self._ctx, _host_ptr(q_host, "q_host", self._block), _host_ptr(out_host, "out_host", self._block), _stream()))

    def export_cache_device(self, head: int):
        """Returns (K, V) bf16 device tensors [n_tokens, d] of what the cache keeps for ``head``, logical order."""
        import torch
        n = C.c_int32()
        k = torch.empty((self.n_blocks * self.block_tokens, self.head_dim), dtype=torch.bfloat16, device="cuda")
        v = torch.empty_like(k)
        self._check(self.lib.headcast_export_cache(self._ctx, head, _ptr(k), _ptr(v), C.byref(n), _stream()))
        torch.cuda.current_stream().synchronize()
        return k[: n.value], v[: n.value]

    def export_cache(self, head: int):
        """Returns (K, V) uint16 CPU arrays [n_tokens, d] of what the cache keeps for ``head``."""
        import torch
        k, v = self.export_cache_device(head)
        to_bits = lambda t: t.view(torch.int16).cpu().numpy().view("uint16")
        return to_bits(k), to_bits(v)

    def n_filled(self) -> int:
        return self.lib.headcast_n_filled(self._ctx)

    def launch_count(self) -> int:
        return self.lib.headcast_launch_count(self._ctx)

    def attend_flops(self, dense: bool = False) -> float:
        return self.lib.headcast_attend_flops(self._ctx, int(dense))

    def set_kernel_timing(self, enable: bool) -> None:
        self._check(self.lib.headcast_set_kernel_timing(self._ctx, int(enable)))

    def last_attention_kernel_ms(self) -> float:
        ms = C.c_float()
        self._check(self.lib.headcast_last_attention_kernel_ms(self._ctx, C.byref(ms)))
        return ms.value

    def set_tracing(self, enable: bool) -> None:
        self._check(self.lib.headcast_set_tracing(self._ctx, int(enable)))

    def read_trace(self):
        """[n_items, 8] int64: cta, head, cell, query rows, key tiles, output mode, start ns, end ns."""
        import numpy as np
        n = C.c_int32()
        self._check(self.lib.headcast_read_trace(self._ctx, None, 0, C.byref(n)))
        rows = np.zeros((max(n.value, 1), 8), dtype=np.int64)
        self._check(self.lib.headcast_read_trace(self._ctx, rows.ctypes.data_as(C.POINTER(C.c_int64)), n.value, C.byref(n)))
        return rows[: n.value]

    def selftest_bounded_wait(self, limit_ms: int = 50) -> int:
        """Returns the library's status code (HC_ERR_TIMEOUT = -6 is the expected outcome)."""
        return self.lib.headcast_selftest_bounded_wait(self._ctx, int(limit_ms), _stream())

    def check(self) -> None:
        self._check(self.lib.headcast_check(self._ctx, _stream()))
