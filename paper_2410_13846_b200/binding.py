"""ctypes binding of liblt.so.  Same names as the C ABI minus the ``lt_`` prefix.

Tensors are torch CUDA tensors used only as device memory: the binding passes
``data_ptr()`` and the current CUDA stream.  Layer tables are Python lists of
tensors (or None entries).  Nothing here computes anything.
"""
from __future__ import annotations

import ctypes as C
import os
from dataclasses import dataclass

LT_F32, LT_BF16 = 0, 1
LT_MAX_LAYERS = 128
_PKG_DIR = os.path.dirname(os.path.abspath(__file__))
_LIB = None


class LtError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        super().__init__(f"{where}: lt_status {status} ({status_string(status)})")


class _CShape(C.Structure):
    _fields_ = [(n, C.c_int32) for n in
                ("n_layers", "batch", "n_q_heads", "n_kv_heads", "head_dim", "n_sink", "n_recent",
                 "full_capacity", "dtype")] + [("softmax_scale", C.c_float), ("per_sequence_mask", C.c_int32),
                                                ("recent_per_row", C.c_int32), ("page_size", C.c_int32),
                                                ("pages_per_seq", C.c_int32), ("n_pages", C.c_int32),
                                                ("reserved_", C.c_int32), ("block_table", C.c_void_p),
                                                ("kv_fp8", C.c_int32), ("reserved2_", C.c_int32),
                                                ("kv_scales", C.c_void_p)]


@dataclass
class Shape:
    n_layers: int
    batch: int
    n_q_heads: int
    n_kv_heads: int
    head_dim: int
    n_sink: int
    n_recent: int
    full_capacity: int
    dtype: int = LT_BF16
    softmax_scale: float = 0.0
    per_sequence_mask: int = 0
    recent_per_row: int = 0
    page_size: int = 0           # > 0: paged full caches (see lt_shape in include/lt.h)
    pages_per_seq: int = 0
    n_pages: int = 0
    block_table: object = None   # int32 CUDA tensor [batch][pages_per_seq]
    kv_fp8: int = 0              # 1: caches hold FP8 E4M3 bytes with per-layer scales
    kv_scales: object = None     # float32 CUDA tensor [n_layers][2]

    def c(self) -> _CShape:
        bt = None
        if self.block_table is not None:
            t = self.block_table
            if not (t.is_cuda and t.is_contiguous() and t.element_size() == 4):
                raise ValueError("block_table must be a contiguous int32 CUDA tensor")
            bt = t.data_ptr()
        return _CShape(self.n_layers, self.batch, self.n_q_heads, self.n_kv_heads, self.head_dim, self.n_sink,
                       self.n_recent, self.full_capacity, self.dtype, self.softmax_scale, self.per_sequence_mask,
                       self.recent_per_row, self.page_size, self.pages_per_seq, self.n_pages, 0, bt, self.kv_fp8, 0,
                       self._scales_ptr())

    def _scales_ptr(self):
        t = self.kv_scales
        if t is None:
            return None
        import torch
        if not (t.is_cuda and t.is_contiguous() and t.dtype == torch.float32):
            raise ValueError("kv_scales must be a contiguous float32 CUDA tensor")
        return t.data_ptr()

    @property
    def stream_capacity(self) -> int:
        return self.n_sink + self.n_recent


def lib_path() -> str:
    return os.path.join(_PKG_DIR, "liblt.so")


def lib() -> C.CDLL:
    """Load liblt.so (once).  Raises if it has not been built."""
    global _LIB
    if _LIB is not None:
        return _LIB
    path = lib_path()
    if not os.path.exists(path):
        raise RuntimeError(f"{path} is missing: build it with `python -m paper_2410_13846_b200.build` "
                           "(there is no fallback path)")
    L = C.CDLL(path)
    vp, i32, sz = C.c_void_p, C.c_int32, C.c_size_t
    shp = C.POINTER(_CShape)
    tab = C.POINTER(C.c_void_p)
    L.lt_status_string.restype = C.c_char_p
    L.lt_status_string.argtypes = [i32]
    L.lt_version.restype = i32
    L.lt_version.argtypes = []
    L.lt_ring_slot.restype = i32
    L.lt_ring_slot.argtypes = [i32, i32, i32]
    L.lt_workspace_bytes.restype = i32
    L.lt_workspace_bytes.argtypes = [shp, i32, i32, C.POINTER(sz)]
    L.lt_workspace_init.restype = i32
    L.lt_workspace_init.argtypes = [vp, sz, vp]
    L.lt_check.restype = i32
    L.lt_check.argtypes = [vp, C.POINTER(C.c_uint32), vp]
    L.lt_lazy_scores.restype = i32
    L.lt_lazy_scores.argtypes = [shp, vp, tab, i32, i32, i32, i32, vp, vp, sz, vp]
    L.lt_lazy_scores_with_lse.restype = i32
    L.lt_lazy_scores_with_lse.argtypes = [shp, vp, tab, i32, i32, i32, i32, vp, vp, vp, sz, vp]
    L.lt_lazy_scores_lse.restype = i32
    L.lt_lazy_scores_lse.argtypes = [shp, vp, tab, vp, i32, i32, i32, i32, vp, vp, sz, vp]
    L.lt_select_lazy.restype = i32
    L.lt_select_lazy.argtypes = [vp, i32, i32, i32, i32, vp, vp, vp]
    L.lt_select_lazy_per_seq.restype = i32
    L.lt_select_lazy_per_seq.argtypes = [vp, i32, i32, i32, i32, vp, vp, vp]
    L.lt_select_lazy_frequency.restype = i32
    L.lt_select_lazy_frequency.argtypes = [vp, i32, i32, i32, vp, vp, vp]
    L.lt_select_lazy_push.restype = i32
    L.lt_select_lazy_push.argtypes = [vp, i32, i32, i32, i32, i32, vp, vp, vp, vp]
    L.lt_stream_init_layer.restype = i32
    L.lt_stream_init_layer.argtypes = [shp, vp, vp, tab, tab, vp, tab, tab, vp, vp]
    L.lt_stream_init.restype = i32
    L.lt_stream_init.argtypes = [shp, vp, tab, tab, vp, tab, tab, vp, vp]
    L.lt_kv_append.restype = i32
    L.lt_kv_append.argtypes = [shp, vp, vp, vp, vp, tab, tab, tab, tab, i32, i32, i32, vp, vp]
    L.lt_hybrid_decode_attn.restype = i32
    L.lt_hybrid_decode_attn.argtypes = [shp, vp, tab, tab, tab, tab, vp, vp, vp, i32, i32, i32, i32, vp, sz, vp]
    L.lt_decode_step.restype = i32
    L.lt_decode_step.argtypes = [shp, vp, vp, vp, tab, tab, tab, tab, vp, vp, vp, i32, i32, i32, i32, vp, sz, vp]
    L.lt_decode_step_host.restype = i32
    L.lt_decode_step_layers.restype = i32
    L.lt_workspace_bytes_layers.restype = i32
    L.lt_decode_step_layers.argtypes = [shp, vp, vp, vp, tab, tab, tab, tab, vp, vp, vp, i32, i32, i32, i32, i32, vp, sz,
                                        vp]
    L.lt_workspace_bytes_layers.argtypes = [shp, i32, i32, C.POINTER(sz)]
    L.lt_decode_step_host.argtypes = [shp, vp, vp, vp, vp, vp, vp, vp, vp, tab, tab, tab, tab, vp, vp, i32, vp, sz, vp]
    _LIB = L
    return L


def status_string(status: int) -> str:
    return lib().lt_status_string(int(status)).decode()


def version() -> int:
    return int(lib().lt_version())


def ring_slot(pos: int, n_sink: int, n_recent: int) -> int:
    return int(lib().lt_ring_slot(pos, n_sink, n_recent))


# ---- marshalling helpers ----------------------------------------------------
def _ptr(t):
    if t is None:
        return None
    if not t.is_cuda:
        raise ValueError("liblt works on CUDA tensors only (no CPU path)")
    if not t.is_contiguous():
        raise ValueError("tensor must be contiguous")
    return C.c_void_p(t.data_ptr())


def _table(tensors, n_layers):
    """Host array of device pointers from a list of tensors / None; None -> NULL table."""
    if tensors is None:
        return None
    if len(tensors) != n_layers:
        raise ValueError("layer table must have n_layers entries")
    arr = (C.c_void_p * n_layers)()
    for i, t in enumerate(tensors):
        if t is None:
            arr[i] = None
        else:
            if not t.is_cuda or not t.is_contiguous():
                raise ValueError("layer table entries must be contiguous CUDA tensors")
            arr[i] = t.data_ptr()
    return arr


def _stream(stream):
    import torch
    s = stream if stream is not None else torch.cuda.current_stream()
    return C.c_void_p(s.cuda_stream)


def _ok(status: int, where: str):
    if status != 0:
        raise LtError(status, where)


class LayerTables:
    """Pre-marshalled host tables for one set of caches (build once, reuse every step)."""

    def __init__(self, shape: Shape, k_full=None, v_full=None, k_stream=None, v_stream=None):
        L = shape.n_layers
        self.keep = (k_full, v_full, k_stream, v_stream)     # keep the tensors alive
        self.k_full, self.v_full = _table(k_full, L), _table(v_full, L)
        self.k_stream, self.v_stream = _table(k_stream, L), _table(v_stream, L)


# ---- the calls --------------------------------------------------------------
def workspace_bytes(shape: Shape, n_ctx_max: int = 0, w_last_max: int = 0) -> int:
    out = C.c_size_t(0)
    _ok(lib().lt_workspace_bytes(C.byref(shape.c()), n_ctx_max, w_last_max, C.byref(out)), "lt_workspace_bytes")
    return int(out.value)


def workspace_init(ws, stream=None):
    _ok(lib().lt_workspace_init(_ptr(ws), ws.numel() * ws.element_size(), _stream(stream)), "lt_workspace_init")


def check(ws, stream=None, raise_on_error: bool = True) -> int:
    flags = C.c_uint32(0)
    st = lib().lt_check(_ptr(ws), C.byref(flags), _stream(stream))
    if st != 0 and (raise_on_error or st not in (5, 6)):
        raise LtError(st, f"lt_check (flags={flags.value:#x})")
    return int(flags.value)


def lazy_scores(shape: Shape, q_tail, k_full, n_ctx: int, w_last: int, scores, ws, layer_begin: int = 0,
                layer_count: int | None = None, stream=None):
    tab = k_full.k_full if isinstance(k_full, LayerTables) else _table(k_full, shape.n_layers)
    cnt = shape.n_layers - layer_begin if layer_count is None else layer_count
    _ok(lib().lt_lazy_scores(C.byref(shape.c()), _ptr(q_tail), tab, n_ctx, w_last, layer_begin, cnt, _ptr(scores),
                             _ptr(ws), ws.numel() * ws.element_size(), _stream(stream)), "lt_lazy_scores")


def lazy_scores_with_lse(shape: Shape, q_tail, k_full, n_ctx: int, w_last: int, scores, lse_out, ws, layer_begin: int = 0,
                         layer_count: int | None = None, stream=None):
    """lt_lazy_scores_with_lse: Eq. 1 plus the tail rows' log-sum-exp that the same pass computed."""
    tab = k_full.k_full if isinstance(k_full, LayerTables) else _table(k_full, shape.n_layers)
    cnt = shape.n_layers - layer_begin if layer_count is None else layer_count
    _ok(lib().lt_lazy_scores_with_lse(C.byref(shape.c()), _ptr(q_tail), tab, n_ctx, w_last, layer_begin, cnt,
                                      _ptr(scores), _ptr(lse_out), _ptr(ws), ws.numel() * ws.element_size(),
                                      _stream(stream)), "lt_lazy_scores_with_lse")


def lazy_scores_lse(shape: Shape, q_tail, k_full, lse, n_ctx: int, w_last: int, scores, ws, layer_begin: int = 0,
                    layer_count: int | None = None, stream=None):
    """lt_lazy_scores_lse: Eq. 1 from the prefill's log-sum-exp and the kept keys only."""
    tab = k_full.k_full if isinstance(k_full, LayerTables) else _table(k_full, shape.n_layers)
    cnt = shape.n_layers - layer_begin if layer_count is None else layer_count
    _ok(lib().lt_lazy_scores_lse(C.byref(shape.c()), _ptr(q_tail), tab, _ptr(lse), n_ctx, w_last, layer_begin, cnt,
                                 _ptr(scores), _ptr(ws), ws.numel() * ws.element_size(), _stream(stream)),
        "lt_lazy_scores_lse")


def select_lazy(scores, n_layers: int, batch: int, n_q_heads: int, n_lazy: int, layer_mask, layer_ratio=None,
                stream=None):
    _ok(lib().lt_select_lazy(_ptr(scores), n_layers, batch, n_q_heads, n_lazy, _ptr(layer_mask),
                             _ptr(layer_ratio), _stream(stream)), "lt_select_lazy")


def select_lazy_per_seq(scores, n_layers: int, batch: int, n_q_heads: int, n_lazy: int, layer_mask, layer_ratio=None,
                        stream=None):
    _ok(lib().lt_select_lazy_per_seq(_ptr(scores), n_layers, batch, n_q_heads, n_lazy, _ptr(layer_mask),
                                     _ptr(layer_ratio), _stream(stream)), "lt_select_lazy_per_seq")


def select_lazy_frequency(sample_masks, n_samples: int, n_layers: int, n_lazy: int, layer_mask, layer_counts=None,
                          stream=None):
    _ok(lib().lt_select_lazy_frequency(_ptr(sample_masks), n_samples, n_layers, n_lazy, _ptr(layer_mask),
                                       _ptr(layer_counts), _stream(stream)), "lt_select_lazy_frequency")


def select_lazy_push(layer_scores, layer: int, n_layers: int, batch: int, n_q_heads: int, n_full: int, queue_state,
                     layer_mask, popped_layer=None, stream=None):
    _ok(lib().lt_select_lazy_push(_ptr(layer_scores), layer, n_layers, batch, n_q_heads, n_full, _ptr(queue_state),
                                  _ptr(layer_mask), _ptr(popped_layer), _stream(stream)), "lt_select_lazy_push")


def stream_init_layer(shape: Shape, layer_mask, layer, tables: LayerTables, seq_lens, ws=None, stream=None):
    _ok(lib().lt_stream_init_layer(C.byref(shape.c()), _ptr(layer_mask), _ptr(layer), tables.k_full, tables.v_full,
                                   _ptr(seq_lens), tables.k_stream, tables.v_stream, _ptr(ws), _stream(stream)),
        "lt_stream_init_layer")


def stream_init(shape: Shape, layer_mask, tables: LayerTables, seq_lens, ws=None, stream=None):
    _ok(lib().lt_stream_init(C.byref(shape.c()), _ptr(layer_mask), tables.k_full, tables.v_full, _ptr(seq_lens),
                             tables.k_stream, tables.v_stream, _ptr(ws), _stream(stream)), "lt_stream_init")


def kv_append(shape: Shape, layer_mask, k_new, v_new, seq_lens, tables: LayerTables, layer_begin: int = 0,
              layer_count: int | None = None, advance_seq_lens: bool = True, ws=None, stream=None):
    cnt = shape.n_layers - layer_begin if layer_count is None else layer_count
    _ok(lib().lt_kv_append(C.byref(shape.c()), _ptr(layer_mask), _ptr(k_new), _ptr(v_new), _ptr(seq_lens),
                           tables.k_full, tables.v_full, tables.k_stream, tables.v_stream, layer_begin, cnt,
                           1 if advance_seq_lens else 0, _ptr(ws), _stream(stream)), "lt_kv_append")


def hybrid_decode_attn(shape: Shape, q, tables: LayerTables, layer_mask, seq_lens, out, ws, out_dtype: int | None = None,
                       max_seq_len_hint: int = 0, layer_begin: int = 0, layer_count: int | None = None, stream=None):
    import torch
    if out_dtype is None:
        out_dtype = LT_F32 if out.dtype == torch.float32 else LT_BF16
    cnt = shape.n_layers - layer_begin if layer_count is None else layer_count
    _ok(lib().lt_hybrid_decode_attn(C.byref(shape.c()), _ptr(q), tables.k_full, tables.v_full, tables.k_stream,
                                    tables.v_stream, _ptr(layer_mask), _ptr(seq_lens), _ptr(out), out_dtype,
                                    max_seq_len_hint, layer_begin, cnt, _ptr(ws), ws.numel() * ws.element_size(),
                                    _stream(stream)), "lt_hybrid_decode_attn")


def decode_step(shape: Shape, q, k_new, v_new, tables: LayerTables, layer_mask, seq_lens, out, ws,
                out_dtype: int | None = None, layer_begin: int = 0, layer_count: int | None = None,
                advance_seq_lens: bool = True, stream=None):
    """lt_decode_step: KV append + hybrid attention (+ seq_lens advance) in one launch."""
    import torch
    if out_dtype is None:
        out_dtype = LT_F32 if out.dtype == torch.float32 else LT_BF16
    cnt = shape.n_layers - layer_begin if layer_count is None else layer_count
    _ok(lib().lt_decode_step(C.byref(shape.c()), _ptr(q), _ptr(k_new), _ptr(v_new), tables.k_full, tables.v_full,
                             tables.k_stream, tables.v_stream, _ptr(layer_mask), _ptr(seq_lens), _ptr(out), out_dtype,
                             layer_begin, cnt, 1 if advance_seq_lens else 0, _ptr(ws),
                             ws.numel() * ws.element_size(), _stream(stream)), "lt_decode_step")


def decode_step_layers(shape: Shape, q, k_new, v_new, tables: LayerTables, layer_mask, seq_lens, out, ws,
                       layer_begin: int, layer_count: int = 1, advance_seq_lens: bool = False,
                       independent_of_previous: bool = False, out_dtype: int | None = None, stream=None):
    """lt_decode_step_layers: one launch of a step that comes as several launches over disjoint layer ranges."""
    import torch
    if out_dtype is None:
        out_dtype = LT_F32 if out.dtype == torch.float32 else LT_BF16
    _ok(lib().lt_decode_step_layers(C.byref(shape.c()), _ptr(q), _ptr(k_new), _ptr(v_new), tables.k_full,
                                    tables.v_full, tables.k_stream, tables.v_stream, _ptr(layer_mask), _ptr(seq_lens),
                                    _ptr(out), out_dtype, layer_begin, layer_count, 1 if advance_seq_lens else 0,
                                    1 if independent_of_previous else 0, _ptr(ws), ws.numel() * ws.element_size(),
                                    _stream(stream)), "lt_decode_step_layers")


def workspace_bytes_layers(shape: Shape, n_ctx_max: int = 0, w_last_max: int = 0) -> int:
    out = C.c_size_t(0)
    _ok(lib().lt_workspace_bytes_layers(C.byref(shape.c()), n_ctx_max, w_last_max, C.byref(out)),
        "lt_workspace_bytes_layers")
    return out.value


def decode_step_host(shape: Shape, q_host, k_new_host, v_new_host, out_host, q_dev, k_new_dev, v_new_dev, out_dev,
                     tables: LayerTables, layer_mask, seq_lens, ws, stream=None):
    """lt_decode_step_host: the whole-stack step with HOST inputs and output (host tensors, ideally pinned)
    through caller-owned device staging tensors.  Asynchronous on the stream."""
    import torch
    for t in (q_host, k_new_host, v_new_host, out_host):
        if t.is_cuda or not t.is_contiguous():
            raise ValueError("host tensors must be contiguous CPU tensors")
    out_dtype = LT_F32 if out_dev.dtype == torch.float32 else LT_BF16
    hp = lambda t: C.c_void_p(t.data_ptr())  # noqa: E731
    _ok(lib().lt_decode_step_host(C.byref(shape.c()), hp(q_host), hp(k_new_host), hp(v_new_host), hp(out_host),
                                  _ptr(q_dev), _ptr(k_new_dev), _ptr(v_new_dev), _ptr(out_dev), tables.k_full,
                                  tables.v_full, tables.k_stream, tables.v_stream, _ptr(layer_mask), _ptr(seq_lens),
                                  out_dtype, _ptr(ws), ws.numel() * ws.element_size(), _stream(stream)),
        "lt_decode_step_host")


STATIC_SCRATCH_BYTES = 16 << 20


def hybrid_decode_attn_static(shape: Shape, q, tables: LayerTables, layer_mask, seq_lens, out, out_dtype: int | None = None,
                              max_seq_len_hint: int = 0, layer_begin: int = 0, layer_count: int | None = None,
                              dev_error=None, stream=None):
    """lt_hybrid_decode_attn_static: the decode step for callers that cannot
    allocate device memory (the scratch is a fixed array inside the library).
    ``dev_error`` is an optional uint32/int32 CUDA tensor of one element that
    receives the call's error word."""
    import torch
    L = lib()
    if not hasattr(L.lt_hybrid_decode_attn_static, "_lt_typed"):
        vp, i32 = C.c_void_p, C.c_int32
        tab = C.POINTER(C.c_void_p)
        L.lt_hybrid_decode_attn_static.restype = i32
        L.lt_hybrid_decode_attn_static.argtypes = [C.POINTER(_CShape), vp, tab, tab, tab, tab, vp, vp, vp, i32, i32,
                                                   i32, i32, vp, vp]
        L.lt_hybrid_decode_attn_static._lt_typed = True
    if out_dtype is None:
        out_dtype = LT_F32 if out.dtype == torch.float32 else LT_BF16
    cnt = shape.n_layers - layer_begin if layer_count is None else layer_count
    _ok(L.lt_hybrid_decode_attn_static(C.byref(shape.c()), _ptr(q), tables.k_full, tables.v_full, tables.k_stream,
                                       tables.v_stream, _ptr(layer_mask), _ptr(seq_lens), _ptr(out), out_dtype,
                                       max_seq_len_hint, layer_begin, cnt, _ptr(dev_error), _stream(stream)),
        "lt_hybrid_decode_attn_static")
