"""ctypes binding of the C ABI in include/seer.h: same names, argument marshalling only.

Tensors are torch CUDA tensors used purely as device buffers; every step of the
path runs inside libseer.so.  There is no CPU fallback: if the shared library
has not been built, or no B200 is present, the calls raise.
"""
from __future__ import annotations

import ctypes as C
import os
from typing import Optional, Sequence

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libseer.so")

SEER_OK = 0
SEER_TOPK_RATIO, SEER_TOPK_COUNT, SEER_THRESHOLD = 0, 1, 2
SEER_FORCE_DIAG, SEER_FORCE_SINK = 1, 2
SEER_POOL_AVG, SEER_POOL_MAX, SEER_POOL_MIN = 1, 2, 4
STATUS_NAMES = ["SEER_OK", "SEER_ERR_INVALID_ARG", "SEER_ERR_UNSUPPORTED", "SEER_ERR_WORKSPACE", "SEER_ERR_CAPACITY",
                "SEER_ERR_INVALID_INDEX", "SEER_ERR_TIMEOUT", "SEER_ERR_CUDA"]

# every symbol include/seer.h declares
EXPORTS = ["seer_create", "seer_destroy", "seer_status_string", "seer_workspace_bytes", "seer_scores_elems",
           "seer_mask_rows", "seer_causal_blocks", "seer_gate_scores", "seer_block_mask", "seer_sparse_attn",
           "seer_gate_project", "seer_set_attn_impl", "seer_debug_lost_wait", "seer_poll_device_status", "seer_launch_count", "seer_prefill_host_arena_bytes",
           "seer_prefill_host", "seer_set_trace_buffer", "seer_gate_scores_static", "seer_gate_scores_ex",
           "seer_attn_block_max", "seer_gate_mask_workspace_bytes", "seer_gate_block_mask",
           "seer_expand_block_lists"]


class SeerError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        name = STATUS_NAMES[status] if 0 <= status < len(STATUS_NAMES) else str(status)
        super().__init__(f"{where}: {name}")


class seer_shape(C.Structure):
    _fields_ = [("batch", C.c_int32), ("cu_seqlens_host", C.POINTER(C.c_int32)), ("num_q_heads", C.c_int32),
                ("num_kv_heads", C.c_int32), ("head_dim", C.c_int32), ("block", C.c_int32), ("gate_dim", C.c_int32),
                ("softmax_scale", C.c_float), ("cu_seqlens_q_host", C.POINTER(C.c_int32))]


class seer_mask_params(C.Structure):
    _fields_ = [("mode", C.c_int32), ("keep_num", C.c_int32), ("keep_den", C.c_int32), ("k", C.c_int32),
                ("threshold", C.c_float), ("flags", C.c_uint32), ("dense_tail_blocks", C.c_int32)]


class seer_gate_options(C.Structure):
    _fields_ = [("pool_q", C.c_uint32), ("pool_k", C.c_uint32), ("rope_theta", C.c_float)]


_lib = None


def load_library() -> C.CDLL:
    """Loads libseer.so (built in-tree by `python -m paper_2410_13276_b200.build`)."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(LIB_PATH):
        raise ImportError(f"{LIB_PATH} is missing: build it with `python -m paper_2410_13276_b200.build` "
                          "(there is no fallback path)")
    lib = C.CDLL(LIB_PATH)
    vp, sz, i64, i32 = C.c_void_p, C.c_size_t, C.c_int64, C.c_int32
    shp = C.POINTER(seer_shape)
    lib.seer_create.argtypes = [C.POINTER(vp), C.c_int]
    lib.seer_create.restype = C.c_int
    lib.seer_destroy.argtypes = [vp]
    lib.seer_destroy.restype = None
    lib.seer_status_string.argtypes = [C.c_int]
    lib.seer_status_string.restype = C.c_char_p
    lib.seer_workspace_bytes.argtypes = [shp]
    lib.seer_workspace_bytes.restype = sz
    lib.seer_scores_elems.argtypes = [shp]
    lib.seer_scores_elems.restype = sz
    lib.seer_mask_rows.argtypes = [shp]
    lib.seer_mask_rows.restype = i64
    lib.seer_causal_blocks.argtypes = [shp]
    lib.seer_causal_blocks.restype = i64
    lib.seer_gate_scores.argtypes = [vp, shp, vp, vp, vp, vp, vp, vp, sz, vp]
    lib.seer_gate_scores.restype = C.c_int
    lib.seer_gate_project.argtypes = [vp, shp, vp, vp, vp, vp, vp, sz, vp]
    lib.seer_gate_project.restype = C.c_int
    lib.seer_block_mask.argtypes = [vp, shp, vp, C.POINTER(seer_mask_params), vp, vp, i64, vp, vp, sz, vp]
    lib.seer_block_mask.restype = C.c_int
    lib.seer_sparse_attn.argtypes = [vp, shp, vp, vp, vp, vp, vp, vp, vp, vp, sz, vp]
    lib.seer_sparse_attn.restype = C.c_int
    lib.seer_set_attn_impl.argtypes = [vp, C.c_int]
    lib.seer_set_attn_impl.restype = C.c_int
    lib.seer_debug_lost_wait.argtypes = [vp, C.c_uint32, C.c_int32]
    lib.seer_debug_lost_wait.restype = C.c_int
    lib.seer_poll_device_status.argtypes = [vp, vp]
    lib.seer_poll_device_status.restype = C.c_int
    lib.seer_launch_count.argtypes = [vp]
    lib.seer_launch_count.restype = i64
    lib.seer_prefill_host_arena_bytes.argtypes = [shp]
    lib.seer_prefill_host_arena_bytes.restype = sz
    lib.seer_prefill_host.argtypes = [vp, shp, vp, vp, vp, vp, vp, C.POINTER(seer_mask_params), vp, vp, vp, sz, vp]
    lib.seer_prefill_host.restype = C.c_int
    lib.seer_gate_scores_static.argtypes = [shp, vp, vp, vp, vp, vp, vp]
    lib.seer_gate_scores_static.restype = C.c_int
    lib.seer_gate_scores_ex.argtypes = [vp, shp, C.POINTER(seer_gate_options), vp, vp, vp, vp, vp, vp, sz, vp]
    lib.seer_gate_scores_ex.restype = C.c_int
    lib.seer_attn_block_max.argtypes = [vp, shp, vp, vp, vp, vp, vp, vp, vp]
    lib.seer_attn_block_max.restype = C.c_int
    lib.seer_gate_mask_workspace_bytes.argtypes = [shp, sz]
    lib.seer_gate_mask_workspace_bytes.restype = sz
    lib.seer_gate_block_mask.argtypes = [vp, shp, C.POINTER(seer_gate_options), vp, vp, vp, vp, C.POINTER(seer_mask_params),
                                         vp, vp, i64, vp, vp, sz, vp]
    lib.seer_gate_block_mask.restype = C.c_int
    lib.seer_expand_block_lists.argtypes = [vp, shp, vp, vp, vp, vp, i64, vp, vp]
    lib.seer_expand_block_lists.restype = C.c_int
    lib.seer_set_trace_buffer.argtypes = [vp, vp]
    lib.seer_set_trace_buffer.restype = C.c_int
    _lib = lib
    return lib


def _ptr(t) -> Optional[int]:
    """Device (or host) address of a tensor / raw int / None."""
    if t is None:
        return None
    if isinstance(t, int):
        return t
    return t.data_ptr()


def _stream(stream) -> Optional[int]:
    if stream is None:
        import torch
        return torch.cuda.current_stream().cuda_stream
    if isinstance(stream, int):
        return stream
    return stream.cuda_stream


def _check(status: int, where: str) -> None:
    if status != SEER_OK:
        raise SeerError(status, where)


def make_shape(cu_seqlens: Sequence[int], num_q_heads: int, num_kv_heads: int, *, head_dim: int = 128,
               block: int = 64, gate_dim: int = 128, softmax_scale: float = 0.0, cu_seqlens_q=None) -> seer_shape:
    """cu_seqlens_q (optional): chunked prefill, the queries are the last cu_q[b+1] - cu_q[b] positions of sequence b."""
    cu = np.ascontiguousarray(np.asarray(cu_seqlens, dtype=np.int32))
    cuq = None if cu_seqlens_q is None else np.ascontiguousarray(np.asarray(cu_seqlens_q, dtype=np.int32))
    if cuq is not None and len(cuq) != len(cu):
        raise ValueError("cu_seqlens_q must have batch + 1 entries")
    s = seer_shape(len(cu) - 1, cu.ctypes.data_as(C.POINTER(C.c_int32)), num_q_heads, num_kv_heads, head_dim, block,
                   gate_dim, softmax_scale, None if cuq is None else cuq.ctypes.data_as(C.POINTER(C.c_int32)))
    s._keepalive = (cu, cuq)   # the struct points into these arrays
    return s


def make_mask_params(mode: int, *, keep_num: int = 1, keep_den: int = 1, k: int = 0, threshold: float = 0.0,
                     flags: int = SEER_FORCE_DIAG, dense_tail: int = 0) -> seer_mask_params:
    return seer_mask_params(mode, keep_num, keep_den, k, threshold, flags, dense_tail)


def seer_workspace_bytes(shape: seer_shape) -> int:
    return int(load_library().seer_workspace_bytes(C.byref(shape)))


def seer_scores_elems(shape: seer_shape) -> int:
    return int(load_library().seer_scores_elems(C.byref(shape)))


def seer_mask_rows(shape: seer_shape) -> int:
    return int(load_library().seer_mask_rows(C.byref(shape)))


def seer_causal_blocks(shape: seer_shape) -> int:
    return int(load_library().seer_causal_blocks(C.byref(shape)))


def seer_status_string(status: int) -> str:
    return load_library().seer_status_string(status).decode()


class Context:
    """Owns a seer_ctx on one device."""

    def __init__(self, device: int = 0):
        self._lib = load_library()
        self._h = C.c_void_p()
        _check(self._lib.seer_create(C.byref(self._h), device), "seer_create")
        self.device = device

    def close(self):
        if getattr(self, "_h", None) is not None and self._h:
            self._lib.seer_destroy(self._h)
            self._h = C.c_void_p()

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    @property
    def handle(self):
        return self._h


def seer_gate_scores(ctx: Context, shape: seer_shape, q, k, wq, wk, scores, ws, stream=None) -> None:
    ws_bytes = 0 if ws is None else ws.numel() * ws.element_size()
    _check(ctx._lib.seer_gate_scores(ctx.handle, C.byref(shape), _ptr(q), _ptr(k), _ptr(wq), _ptr(wk), _ptr(scores),
                                     _ptr(ws), ws_bytes, _stream(stream)), "seer_gate_scores")


def seer_gate_project(ctx: Context, shape: seer_shape, q, k, wq, wk, ws, stream=None) -> None:
    ws_bytes = 0 if ws is None else ws.numel() * ws.element_size()
    _check(ctx._lib.seer_gate_project(ctx.handle, C.byref(shape), _ptr(q), _ptr(k), _ptr(wq), _ptr(wk), _ptr(ws), ws_bytes,
                                      _stream(stream)), "seer_gate_project")


def seer_gate_scores_ex(ctx: Context, shape: seer_shape, options: seer_gate_options, q, k, wq, wk, scores, ws,
                        stream=None) -> None:
    ws_bytes = 0 if ws is None else ws.numel() * ws.element_size()
    _check(ctx._lib.seer_gate_scores_ex(ctx.handle, C.byref(shape), C.byref(options), _ptr(q), _ptr(k), _ptr(wq),
                                        _ptr(wk), _ptr(scores), _ptr(ws), ws_bytes, _stream(stream)),
           "seer_gate_scores_ex")


def seer_gate_mask_workspace_bytes(shape: seer_shape, band_bytes: int) -> int:
    return int(load_library().seer_gate_mask_workspace_bytes(C.byref(shape), band_bytes))


def seer_gate_block_mask(ctx: Context, shape: seer_shape, options: Optional[seer_gate_options], q, k, wq, wk,
                         params: seer_mask_params, row_ptr, col_idx, col_capacity: Optional[int], nnz_out, ws,
                         stream=None) -> None:
    if col_capacity is None:
        col_capacity = 0 if col_idx is None else col_idx.numel()
    ws_bytes = 0 if ws is None else ws.numel() * ws.element_size()
    opt = None if options is None else C.byref(options)
    _check(ctx._lib.seer_gate_block_mask(ctx.handle, C.byref(shape), opt, _ptr(q), _ptr(k), _ptr(wq), _ptr(wk),
                                         C.byref(params), _ptr(row_ptr), _ptr(col_idx), col_capacity, _ptr(nnz_out),
                                         _ptr(ws), ws_bytes, _stream(stream)), "seer_gate_block_mask")


def seer_expand_block_lists(ctx: Context, shape: seer_shape, row_ptr, col_idx, row_ptr64, col_idx64,
                            col_capacity64: Optional[int] = None, nnz_out=None, stream=None) -> None:
    if col_capacity64 is None:
        col_capacity64 = 0 if col_idx64 is None else col_idx64.numel()
    _check(ctx._lib.seer_expand_block_lists(ctx.handle, C.byref(shape), _ptr(row_ptr), _ptr(col_idx), _ptr(row_ptr64),
                                            _ptr(col_idx64), col_capacity64, _ptr(nnz_out), _stream(stream)),
           "seer_expand_block_lists")


def seer_attn_block_max(ctx: Context, shape: seer_shape, q, k, row_ptr, col_idx, lse, block_max, stream=None) -> None:
    _check(ctx._lib.seer_attn_block_max(ctx.handle, C.byref(shape), _ptr(q), _ptr(k), _ptr(row_ptr), _ptr(col_idx),
                                        _ptr(lse), _ptr(block_max), _stream(stream)), "seer_attn_block_max")


def seer_block_mask(ctx: Context, shape: seer_shape, scores, params: seer_mask_params, row_ptr, col_idx,
                    col_capacity: Optional[int] = None, nnz_out=None, ws=None, stream=None) -> None:
    if col_capacity is None:
        col_capacity = 0 if col_idx is None else col_idx.numel()
    ws_bytes = 0 if ws is None else ws.numel() * ws.element_size()
    _check(ctx._lib.seer_block_mask(ctx.handle, C.byref(shape), _ptr(scores), C.byref(params), _ptr(row_ptr),
                                    _ptr(col_idx), col_capacity, _ptr(nnz_out), _ptr(ws), ws_bytes, _stream(stream)),
           "seer_block_mask")


def seer_sparse_attn(ctx: Context, shape: seer_shape, q, k, v, row_ptr, col_idx, o, lse=None, ws=None,
                     stream=None) -> None:
    ws_bytes = 0 if ws is None else ws.numel() * ws.element_size()
    _check(ctx._lib.seer_sparse_attn(ctx.handle, C.byref(shape), _ptr(q), _ptr(k), _ptr(v), _ptr(row_ptr),
                                     _ptr(col_idx), _ptr(o), _ptr(lse), _ptr(ws), ws_bytes, _stream(stream)),
           "seer_sparse_attn")


def seer_set_attn_impl(ctx: Context, impl: int) -> None:
    _check(ctx._lib.seer_set_attn_impl(ctx.handle, impl), "seer_set_attn_impl")


def seer_debug_lost_wait(ctx: Context, wait_limit_us: int = 2_000_000, lose_v_copy_of_tile: int = -1) -> None:
    _check(ctx._lib.seer_debug_lost_wait(ctx.handle, wait_limit_us, lose_v_copy_of_tile), "seer_debug_lost_wait")


def seer_poll_device_status(ctx: Context, stream=None) -> int:
    return int(ctx._lib.seer_poll_device_status(ctx.handle, _stream(stream)))


def seer_launch_count(ctx: Context) -> int:
    return int(ctx._lib.seer_launch_count(ctx.handle))


def seer_prefill_host_arena_bytes(shape: seer_shape) -> int:
    return int(load_library().seer_prefill_host_arena_bytes(C.byref(shape)))


def seer_prefill_host(ctx: Context, shape: seer_shape, q_host, k_host, v_host, wq_host, wk_host,
                      params: seer_mask_params, o_host, lse_host, arena, stream=None) -> None:
    """Host tensors (ideally pinned) in, host tensors out; `arena` is a device tensor."""
    _check(ctx._lib.seer_prefill_host(ctx.handle, C.byref(shape), _ptr(q_host), _ptr(k_host), _ptr(v_host),
                                      _ptr(wq_host), _ptr(wk_host), C.byref(params), _ptr(o_host), _ptr(lse_host),
                                      _ptr(arena), arena.numel() * arena.element_size(), _stream(stream)),
           "seer_prefill_host")


def seer_set_trace_buffer(ctx: Context, device_buffer) -> None:
    _check(ctx._lib.seer_set_trace_buffer(ctx.handle, _ptr(device_buffer)), "seer_set_trace_buffer")


SEER_STATIC_SCRATCH_BYTES = 8 << 20
SEER_STATIC_MAX_BATCH = 256


def seer_gate_scores_static(shape: seer_shape, q, k, wq, wk, scores, stream=None) -> None:
    """Gate scores for callers that must not allocate: no context, no workspace; the intermediates live in a fixed
    array inside the library (at most SEER_STATIC_SCRATCH_BYTES per call, else SEER_ERR_WORKSPACE).  Runs on the
    current device.  Calls on one device share that array, so keep them on one stream."""
    _check(load_library().seer_gate_scores_static(C.byref(shape), _ptr(q), _ptr(k), _ptr(wq), _ptr(wk), _ptr(scores),
                                                  _stream(stream)), "seer_gate_scores_static")
