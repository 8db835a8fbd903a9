"""ctypes binding of libpowerattn.so: argument marshalling only.

Every function has the name and meaning of its C entry point in include/powerattn.h.  Torch
tensors are used as device buffers (data_ptr) and for the current CUDA stream; all computation
happens inside the library's kernels.  Importing this module without a built library fails.
"""
from __future__ import annotations

import ctypes
import os
from typing import Optional, Tuple

import torch

_PKG = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_PKG, "libpowerattn.so")

PA_OK = 0
PA_BF16, PA_F32 = 0, 1
STATUS_NAMES = ["PA_OK", "PA_ERR_INVALID_ARG", "PA_ERR_SHAPE", "PA_ERR_ALIGNMENT", "PA_ERR_LAYOUT",
                "PA_ERR_WORKSPACE", "PA_ERR_UNSUPPORTED", "PA_ERR_CUDA", "PA_ERR_TIMEOUT"]

EXPORTS = ["pa_status_string", "pa_last_error_message", "pa_version", "pa_reload_environment",
           "pa_set_wait_limit_cycles", "pa_layout_size", "pa_build_layout", "pa_window_layout_size",
           "pa_build_window_layout", "pa_reach_counts", "pa_tile_layout_size",
           "pa_build_tile_layout", "pa_prefill_workspace_bytes", "pa_prefill", "pa_prefill_varlen", "pa_prefill_status",
           "pa_prefill_backward_workspace_bytes", "pa_prefill_backward",
           "pa_decode_workspace_bytes", "pa_decode", "pa_decode_status", "pa_decode_block_list",
           "pa_decode_row_block_set", "pa_decode_paged_workspace_bytes", "pa_decode_paged", "pa_kv_append",
           "pa_decode_static"]


class PaError(RuntimeError):
    def __init__(self, status: int, message: str):
        self.status = status
        name = STATUS_NAMES[status] if 0 <= status < len(STATUS_NAMES) else str(status)
        super().__init__(f"{name}: {message}")


class pa_strides(ctypes.Structure):
    _fields_ = [("batch", ctypes.c_int64), ("seq", ctypes.c_int64), ("head", ctypes.c_int64)]


class pa_prefill_params(ctypes.Structure):
    _fields_ = [("batch", ctypes.c_int32), ("n_q_heads", ctypes.c_int32), ("n_kv_heads", ctypes.c_int32),
                ("head_dim", ctypes.c_int32), ("seq_len", ctypes.c_int64), ("block", ctypes.c_int32),
                ("softmax_scale", ctypes.c_float), ("q", pa_strides), ("k", pa_strides),
                ("v", pa_strides), ("o", pa_strides), ("o_dtype", ctypes.c_int)]


class pa_decode_params(ctypes.Structure):
    _fields_ = [("batch", ctypes.c_int32), ("n_q_heads", ctypes.c_int32), ("n_kv_heads", ctypes.c_int32),
                ("head_dim", ctypes.c_int32), ("block", ctypes.c_int32), ("window_blocks", ctypes.c_int32),
                ("sink_blocks", ctypes.c_int32), ("max_len", ctypes.c_int64),
                ("softmax_scale", ctypes.c_float), ("k", pa_strides), ("v", pa_strides),
                ("o_dtype", ctypes.c_int)]


class pa_paged_params(ctypes.Structure):
    _fields_ = [("batch", ctypes.c_int32), ("n_q_heads", ctypes.c_int32), ("n_kv_heads", ctypes.c_int32),
                ("head_dim", ctypes.c_int32), ("block", ctypes.c_int32), ("window_blocks", ctypes.c_int32),
                ("sink_blocks", ctypes.c_int32), ("n_pages", ctypes.c_int32),
                ("max_blocks_per_seq", ctypes.c_int32), ("softmax_scale", ctypes.c_float),
                ("k", pa_strides), ("v", pa_strides), ("o_dtype", ctypes.c_int)]


def _load() -> ctypes.CDLL:
    if not os.path.exists(LIB_PATH):
        raise ImportError(f"{LIB_PATH} is missing: build it with `python paper_2503_03588_b200/build.py` "
                          "(there is no fallback path)")
    lib = ctypes.CDLL(LIB_PATH)
    vp, i32, i64 = ctypes.c_void_p, ctypes.c_int32, ctypes.c_int64
    lib.pa_status_string.restype = ctypes.c_char_p
    lib.pa_status_string.argtypes = [ctypes.c_int]
    lib.pa_last_error_message.restype = ctypes.c_char_p
    lib.pa_last_error_message.argtypes = []
    lib.pa_version.restype = ctypes.c_int
    lib.pa_layout_size.restype = ctypes.c_int
    lib.pa_layout_size.argtypes = [i64, i32, i32, i32, ctypes.POINTER(i32), ctypes.POINTER(i64)]
    lib.pa_build_layout.restype = ctypes.c_int
    lib.pa_build_layout.argtypes = [i64, i32, i32, i32, vp, vp, i64, vp]
    lib.pa_window_layout_size.restype = ctypes.c_int
    lib.pa_window_layout_size.argtypes = [i64, i32, i32, i32, ctypes.POINTER(i32), ctypes.POINTER(i64)]
    lib.pa_build_window_layout.restype = ctypes.c_int
    lib.pa_build_window_layout.argtypes = [i64, i32, i32, i32, vp, vp, i64, vp]
    lib.pa_reach_counts.restype = ctypes.c_int
    lib.pa_reach_counts.argtypes = [vp, vp, i32, i32, i32, vp]
    lib.pa_tile_layout_size.restype = ctypes.c_int
    lib.pa_tile_layout_size.argtypes = [i64, i32, i32, i32, i32, ctypes.POINTER(i32), ctypes.POINTER(i64)]
    lib.pa_build_tile_layout.restype = ctypes.c_int
    lib.pa_build_tile_layout.argtypes = [i64, i32, i32, i32, i32, vp, vp, i64, vp]
    lib.pa_prefill_workspace_bytes.restype = ctypes.c_size_t
    lib.pa_prefill_workspace_bytes.argtypes = [ctypes.POINTER(pa_prefill_params)]
    lib.pa_prefill.restype = ctypes.c_int
    lib.pa_prefill.argtypes = [ctypes.POINTER(pa_prefill_params), vp, vp, vp, vp, vp, i64, vp, vp, vp,
                               ctypes.c_size_t, vp]
    lib.pa_prefill_varlen.restype = ctypes.c_int
    lib.pa_prefill_varlen.argtypes = [ctypes.POINTER(pa_prefill_params), vp, vp, vp, vp, i64, vp, vp, i64, vp, vp, vp,
                                      ctypes.c_size_t, vp]
    lib.pa_prefill_backward_workspace_bytes.restype = ctypes.c_size_t
    lib.pa_prefill_backward_workspace_bytes.argtypes = [ctypes.POINTER(pa_prefill_params), i64]
    lib.pa_prefill_backward.restype = ctypes.c_int
    lib.pa_prefill_backward.argtypes = [ctypes.POINTER(pa_prefill_params), vp, vp, vp, vp, vp, vp, vp, vp, i64, vp, vp,
                                        vp, vp, ctypes.c_size_t, vp]
    lib.pa_prefill_status.restype = ctypes.c_int
    lib.pa_prefill_status.argtypes = [vp, vp, ctypes.POINTER(i32)]
    lib.pa_decode_workspace_bytes.restype = ctypes.c_size_t
    lib.pa_decode_workspace_bytes.argtypes = [ctypes.POINTER(pa_decode_params)]
    lib.pa_decode.restype = ctypes.c_int
    lib.pa_decode.argtypes = [ctypes.POINTER(pa_decode_params), vp, vp, vp, vp, vp, vp, vp,
                              ctypes.c_size_t, vp]
    lib.pa_decode_block_list.restype = ctypes.c_int
    lib.pa_decode_block_list.argtypes = [i64, i32, i32, i32, vp, vp, i32, vp]
    lib.pa_decode_static.restype = ctypes.c_int
    lib.pa_decode_static.argtypes = [ctypes.POINTER(pa_decode_params), vp, vp, vp, vp, vp, vp, vp]
    lib.pa_reload_environment.restype = None
    lib.pa_reload_environment.argtypes = []
    lib.pa_set_wait_limit_cycles.restype = None
    lib.pa_set_wait_limit_cycles.argtypes = [i64]
    lib.pa_decode_status.restype = ctypes.c_int
    lib.pa_decode_status.argtypes = [vp, vp, ctypes.POINTER(i32)]
    lib.pa_decode_row_block_set.restype = ctypes.c_int
    lib.pa_decode_row_block_set.argtypes = [i64, i32, i32, i32, vp, vp, i32, vp]
    lib.pa_decode_paged_workspace_bytes.restype = ctypes.c_size_t
    lib.pa_decode_paged_workspace_bytes.argtypes = [ctypes.POINTER(pa_paged_params)]
    lib.pa_decode_paged.restype = ctypes.c_int
    lib.pa_decode_paged.argtypes = [ctypes.POINTER(pa_paged_params), vp, vp, vp, vp, vp, vp, vp, vp,
                                    ctypes.c_size_t, vp]
    lib.pa_kv_append.restype = ctypes.c_int
    lib.pa_kv_append.argtypes = [ctypes.POINTER(pa_paged_params), vp, vp, vp, vp, vp, vp, vp]
    return lib


lib = _load()


def _check(status: int) -> None:
    if status != PA_OK:
        raise PaError(status, lib.pa_last_error_message().decode())


def _stream() -> ctypes.c_void_p:
    return ctypes.c_void_p(torch.cuda.current_stream().cuda_stream)


def _ptr(t: Optional[torch.Tensor]) -> ctypes.c_void_p:
    return ctypes.c_void_p(0 if t is None else t.data_ptr())


def _strides4(t: torch.Tensor) -> pa_strides:
    assert t.dim() == 4 and t.stride(3) == 1, "expected [batch, seq, head, head_dim] with contiguous head_dim"
    return pa_strides(t.stride(0), t.stride(1), t.stride(2))


def pa_version() -> int:
    return int(lib.pa_version())


def pa_status_string(status: int) -> str:
    return lib.pa_status_string(status).decode()


def pa_reload_environment() -> None:
    lib.pa_reload_environment()


def pa_set_wait_limit_cycles(cycles: int) -> None:
    lib.pa_set_wait_limit_cycles(int(cycles))


def pa_layout_size(seq_len: int, block: int, window_blocks: int, sink_blocks: int) -> Tuple[int, int]:
    nqb, nnz = ctypes.c_int32(0), ctypes.c_int64(0)
    _check(lib.pa_layout_size(seq_len, block, window_blocks, sink_blocks, ctypes.byref(nqb), ctypes.byref(nnz)))
    return int(nqb.value), int(nnz.value)


def pa_build_layout(seq_len: int, block: int, window_blocks: int, sink_blocks: int,
                    row_ptr: Optional[torch.Tensor] = None, col_idx: Optional[torch.Tensor] = None,
                    device="cuda"):
    """Returns (row_ptr, col_idx) int32 device tensors (allocated here when not passed in)."""
    nqb, nnz = pa_layout_size(seq_len, block, window_blocks, sink_blocks)
    if row_ptr is None:
        row_ptr = torch.empty(nqb + 1, dtype=torch.int32, device=device)
    if col_idx is None:
        col_idx = torch.empty(nnz, dtype=torch.int32, device=device)
    assert row_ptr.dtype == torch.int32 and col_idx.dtype == torch.int32 and row_ptr.numel() >= nqb + 1
    _check(lib.pa_build_layout(seq_len, block, window_blocks, sink_blocks, _ptr(row_ptr), _ptr(col_idx),
                               col_idx.numel(), _stream()))
    return row_ptr, col_idx


def pa_window_layout_size(seq_len: int, block: int, window_blocks: int, sink_blocks: int) -> Tuple[int, int]:
    nqb, nnz = ctypes.c_int32(0), ctypes.c_int64(0)
    _check(lib.pa_window_layout_size(seq_len, block, window_blocks, sink_blocks, ctypes.byref(nqb), ctypes.byref(nnz)))
    return int(nqb.value), int(nnz.value)


def pa_build_window_layout(seq_len: int, block: int, window_blocks: int, sink_blocks: int,
                           row_ptr: Optional[torch.Tensor] = None, col_idx: Optional[torch.Tensor] = None,
                           device="cuda"):
    """Sliding-window layout (window + sink blocks, no power-of-two term) as int32 device tensors."""
    nqb, nnz = pa_window_layout_size(seq_len, block, window_blocks, sink_blocks)
    if row_ptr is None:
        row_ptr = torch.empty(nqb + 1, dtype=torch.int32, device=device)
    if col_idx is None:
        col_idx = torch.empty(nnz, dtype=torch.int32, device=device)
    _check(lib.pa_build_window_layout(seq_len, block, window_blocks, sink_blocks, _ptr(row_ptr), _ptr(col_idx),
                                      col_idx.numel(), _stream()))
    return row_ptr, col_idx


def pa_reach_counts(row_ptr, col_idx, start: int, max_steps: int):
    """|B_k| for k = 1..max_steps from a HOST CSR (numpy int32 arrays or CPU tensors)."""
    import numpy as np

    rp = np.ascontiguousarray(np.asarray(row_ptr, dtype=np.int32))
    ci = np.ascontiguousarray(np.asarray(col_idx, dtype=np.int32))
    out = np.zeros(max_steps, dtype=np.int64)
    _check(lib.pa_reach_counts(rp.ctypes.data_as(ctypes.c_void_p), ci.ctypes.data_as(ctypes.c_void_p), len(rp) - 1,
                               start, max_steps, out.ctypes.data_as(ctypes.c_void_p)))
    return out.tolist()


def pa_tile_layout_size(seq_len: int, block: int, window_blocks: int, sink_blocks: int,
                        tile: int = 64) -> Tuple[int, int]:
    nqt, nnz = ctypes.c_int32(0), ctypes.c_int64(0)
    _check(lib.pa_tile_layout_size(seq_len, block, window_blocks, sink_blocks, tile, ctypes.byref(nqt),
                                   ctypes.byref(nnz)))
    return int(nqt.value), int(nnz.value)


def pa_build_tile_layout(seq_len: int, block: int, window_blocks: int, sink_blocks: int, tile: int = 64,
                         row_ptr: Optional[torch.Tensor] = None, col_idx: Optional[torch.Tensor] = None,
                         device="cuda"):
    """Returns (row_ptr, col_idx) int32 device tensors of the mask with `block`-token blocks listed by
    `tile`-token tiles (allocated here when not passed in)."""
    nqt, nnz = pa_tile_layout_size(seq_len, block, window_blocks, sink_blocks, tile)
    if row_ptr is None:
        row_ptr = torch.empty(nqt + 1, dtype=torch.int32, device=device)
    if col_idx is None:
        col_idx = torch.empty(nnz, dtype=torch.int32, device=device)
    assert row_ptr.dtype == torch.int32 and col_idx.dtype == torch.int32 and row_ptr.numel() >= nqt + 1
    _check(lib.pa_build_tile_layout(seq_len, block, window_blocks, sink_blocks, tile, _ptr(row_ptr),
                                    _ptr(col_idx), col_idx.numel(), _stream()))
    return row_ptr, col_idx


def prefill_params(q, k, v, o, block: int = 64, softmax_scale: float = 0.0) -> pa_prefill_params:
    batch, seq, hq, d = q.shape
    return pa_prefill_params(batch, hq, k.shape[2], d, seq, block, float(softmax_scale), _strides4(q),
                             _strides4(k), _strides4(v), _strides4(o),
                             PA_F32 if o.dtype == torch.float32 else PA_BF16)


def pa_prefill_workspace_bytes(params: pa_prefill_params) -> int:
    return int(lib.pa_prefill_workspace_bytes(ctypes.byref(params)))


def pa_prefill(q, k, v, row_ptr, col_idx, o=None, lse=None, workspace=None, block: int = 64,
               softmax_scale: float = 0.0, o_dtype=torch.bfloat16, nnz: Optional[int] = None):
    """q [batch, N, Hq, D], k, v [batch, N, Hkv, D] bf16 device tensors; CSR int32 device tensors.
    Returns (o, lse, workspace); outputs and scratch are allocated here when not passed in."""
    batch, seq, hq, d = q.shape
    if o is None:
        o = torch.empty((batch, seq, hq, d), dtype=o_dtype, device=q.device)
    if lse is None:
        lse = torch.empty((batch, hq, seq), dtype=torch.float32, device=q.device)
    params = prefill_params(q, k, v, o, block, softmax_scale)
    if workspace is None:
        workspace = torch.empty(max(pa_prefill_workspace_bytes(params), 16), dtype=torch.uint8, device=q.device)
    _check(lib.pa_prefill(ctypes.byref(params), _ptr(q), _ptr(k), _ptr(v), _ptr(row_ptr), _ptr(col_idx),
                          col_idx.numel() if nnz is None else nnz, _ptr(o), _ptr(lse), _ptr(workspace),
                          workspace.numel(), _stream()))
    return o, lse, workspace


def pa_prefill_varlen(q, k, v, cu_seqlens, max_seq_len: int, row_ptr, col_idx, o=None, lse=None, workspace=None,
                      block: int = 64, softmax_scale: float = 0.0, o_dtype=torch.bfloat16):
    """Packed sequences: q [total, Hq, D], k, v [total, Hkv, D] bf16, cu_seqlens int32 [batch + 1] on the
    device.  Returns (o [total, Hq, D], lse [Hq, total], workspace)."""
    total, hq, d = q.shape
    assert q.stride(2) == 1 and k.stride(2) == 1 and v.stride(2) == 1 and cu_seqlens.dtype == torch.int32
    if o is None:
        o = torch.empty((total, hq, d), dtype=o_dtype, device=q.device)
    if lse is None:
        lse = torch.empty((hq, total), dtype=torch.float32, device=q.device)
    st = lambda t: pa_strides(0, t.stride(0), t.stride(1))
    params = pa_prefill_params(cu_seqlens.numel() - 1, hq, k.shape[1], d, max_seq_len, block, float(softmax_scale),
                               st(q), st(k), st(v), st(o), PA_F32 if o.dtype == torch.float32 else PA_BF16)
    if workspace is None:
        workspace = torch.empty(max(pa_prefill_workspace_bytes(params), 16), dtype=torch.uint8, device=q.device)
    _check(lib.pa_prefill_varlen(ctypes.byref(params), _ptr(q), _ptr(k), _ptr(v), _ptr(cu_seqlens), total,
                                 _ptr(row_ptr), _ptr(col_idx), col_idx.numel(), _ptr(o), _ptr(lse), _ptr(workspace),
                                 workspace.numel(), _stream()))
    return o, lse, workspace


def pa_prefill_backward(q, k, v, o, lse, d_o, row_ptr, col_idx, dq=None, dk=None, dv=None, workspace=None,
                        block: int = 64, softmax_scale: float = 0.0):
    """Gradients of pa_prefill: q, k, v, o (bf16) and lse as in the forward call, d_o bf16 with o's
    strides.  Returns (dq, dk, dv, workspace), fp32 contiguous, allocated here when not passed in."""
    batch, seq, hq, d = q.shape
    hkv = k.shape[2]
    assert d_o.stride() == o.stride() and o.dtype == torch.bfloat16 and d_o.dtype == torch.bfloat16
    if dq is None:
        dq = torch.empty((batch, seq, hq, d), dtype=torch.float32, device=q.device)
    if dk is None:
        dk = torch.empty((batch, seq, hkv, d), dtype=torch.float32, device=q.device)
    if dv is None:
        dv = torch.empty((batch, seq, hkv, d), dtype=torch.float32, device=q.device)
    params = prefill_params(q, k, v, o, block, softmax_scale)
    nnz = col_idx.numel()
    if workspace is None:
        workspace = torch.empty(int(lib.pa_prefill_backward_workspace_bytes(ctypes.byref(params), nnz)) + 256,
                                dtype=torch.uint8, device=q.device)
    ws_ptr = (workspace.data_ptr() + 255) & ~255
    _check(lib.pa_prefill_backward(ctypes.byref(params), _ptr(q), _ptr(k), _ptr(v), _ptr(o), _ptr(lse), _ptr(d_o),
                                   _ptr(row_ptr), _ptr(col_idx), nnz, _ptr(dq), _ptr(dk), _ptr(dv),
                                   ctypes.c_void_p(ws_ptr), workspace.numel() - (ws_ptr - workspace.data_ptr()), _stream()))
    return dq, dk, dv, workspace


def pa_prefill_status(workspace: torch.Tensor) -> int:
    """Synchronises the current stream; raises PaError if the kernel recorded a timeout."""
    detail = ctypes.c_int32(0)
    _check(lib.pa_prefill_status(_ptr(workspace), _stream(), ctypes.byref(detail)))
    return int(detail.value)


def decode_params(q, k_cache, v_cache, window_blocks: int, sink_blocks: int, block: int = 64,
                  softmax_scale: float = 0.0, o_dtype=torch.bfloat16) -> pa_decode_params:
    batch, hq, d = q.shape
    return pa_decode_params(batch, hq, k_cache.shape[2], d, block, window_blocks, sink_blocks,
                            k_cache.shape[1], float(softmax_scale), _strides4(k_cache), _strides4(v_cache),
                            PA_F32 if o_dtype == torch.float32 else PA_BF16)


def pa_decode_workspace_bytes(params: pa_decode_params) -> int:
    return int(lib.pa_decode_workspace_bytes(ctypes.byref(params)))


def pa_decode(q, k_cache, v_cache, cache_lens, window_blocks: int, sink_blocks: int, o=None, lse=None,
              workspace=None, block: int = 64, softmax_scale: float = 0.0, o_dtype=torch.bfloat16):
    """q [batch, Hq, D] bf16, caches [batch, max_len, Hkv, D] bf16, cache_lens int32 [batch], all on
    the device.  Returns (o, lse, workspace)."""
    batch, hq, d = q.shape
    if o is None:
        o = torch.empty((batch, hq, d), dtype=o_dtype, device=q.device)
    if lse is None:
        lse = torch.empty((batch, hq), dtype=torch.float32, device=q.device)
    params = decode_params(q, k_cache, v_cache, window_blocks, sink_blocks, block, softmax_scale, o.dtype)
    if workspace is None:
        workspace = torch.empty(max(pa_decode_workspace_bytes(params), 16), dtype=torch.uint8, device=q.device)
    assert cache_lens.dtype == torch.int32 and q.is_contiguous() and o.is_contiguous()
    _check(lib.pa_decode(ctypes.byref(params), _ptr(q), _ptr(k_cache), _ptr(v_cache), _ptr(cache_lens),
                         _ptr(o), _ptr(lse), _ptr(workspace), workspace.numel(), _stream()))
    return o, lse, workspace


def pa_decode_block_list(cache_len: int, block: int, window_blocks: int, sink_blocks: int,
                         capacity: int = 256, device="cuda") -> torch.Tensor:
    out = torch.full((capacity,), -1, dtype=torch.int32, device=device)
    cnt = torch.zeros(1, dtype=torch.int32, device=device)
    _check(lib.pa_decode_block_list(cache_len, block, window_blocks, sink_blocks, _ptr(out), _ptr(cnt),
                                    capacity, _stream()))
    n = int(cnt.item())
    return out[:n].clone()


def pa_decode_status(workspace: torch.Tensor) -> int:
    """Synchronises the current stream; raises PaError if the decode kernel recorded a timeout."""
    detail = ctypes.c_int32(0)
    _check(lib.pa_decode_status(_ptr(workspace), _stream(), ctypes.byref(detail)))
    return int(detail.value)


def pa_decode_row_block_set(cache_len: int, block: int, window_blocks: int, sink_blocks: int,
                            device="cuda") -> torch.Tensor:
    """The single-launch decode kernel's (unsorted) key-block set for one cache length."""
    out = torch.full((32,), -1, dtype=torch.int32, device=device)
    cnt = torch.zeros(1, dtype=torch.int32, device=device)
    _check(lib.pa_decode_row_block_set(cache_len, block, window_blocks, sink_blocks, _ptr(out), _ptr(cnt), 32,
                                       _stream()))
    n = int(cnt.item())
    return out[:n].clone()


def paged_params(q, k_pool, v_pool, block_table, window_blocks: int, sink_blocks: int, block: int = 64,
                 softmax_scale: float = 0.0, o_dtype=torch.bfloat16) -> pa_paged_params:
    """q [batch, Hq, D]; pools [n_pages, block, Hkv, D]; block_table int32 [batch, max_blocks]."""
    batch, hq, d = q.shape
    assert k_pool.shape[1] == block and block_table.dtype == torch.int32 and block_table.is_contiguous()
    return pa_paged_params(batch, hq, k_pool.shape[2], d, block, window_blocks, sink_blocks, k_pool.shape[0],
                           block_table.shape[1], float(softmax_scale), _strides4(k_pool), _strides4(v_pool),
                           PA_F32 if o_dtype == torch.float32 else PA_BF16)


def pa_decode_paged_workspace_bytes(params: pa_paged_params) -> int:
    return int(lib.pa_decode_paged_workspace_bytes(ctypes.byref(params)))


def pa_decode_paged(q, k_pool, v_pool, block_table, cache_lens, window_blocks: int, sink_blocks: int, o=None,
                    lse=None, workspace=None, block: int = 64, softmax_scale: float = 0.0, o_dtype=torch.bfloat16):
    """pa_decode against a pool of 64-token pages.  Returns (o, lse, workspace)."""
    batch, hq, d = q.shape
    if o is None:
        o = torch.empty((batch, hq, d), dtype=o_dtype, device=q.device)
    if lse is None:
        lse = torch.empty((batch, hq), dtype=torch.float32, device=q.device)
    params = paged_params(q, k_pool, v_pool, block_table, window_blocks, sink_blocks, block, softmax_scale, o.dtype)
    if workspace is None:
        workspace = torch.empty(max(pa_decode_paged_workspace_bytes(params), 16), dtype=torch.uint8, device=q.device)
    assert cache_lens.dtype == torch.int32 and q.is_contiguous() and o.is_contiguous()
    _check(lib.pa_decode_paged(ctypes.byref(params), _ptr(q), _ptr(k_pool), _ptr(v_pool), _ptr(block_table),
                               _ptr(cache_lens), _ptr(o), _ptr(lse), _ptr(workspace), workspace.numel(), _stream()))
    return o, lse, workspace


def pa_kv_append(k_new, v_new, k_pool, v_pool, block_table, cache_lens, block: int = 64) -> None:
    """k_new, v_new [batch, Hkv, D] go to position cache_lens[b] of each sequence; cache_lens grows by one."""
    batch, hkv, d = k_new.shape
    assert k_new.is_contiguous() and v_new.is_contiguous() and cache_lens.dtype == torch.int32
    params = pa_paged_params(batch, hkv, hkv, d, block, 0, 0, k_pool.shape[0], block_table.shape[1], 0.0,
                             _strides4(k_pool), _strides4(v_pool), PA_BF16)
    _check(lib.pa_kv_append(ctypes.byref(params), _ptr(k_new), _ptr(v_new), _ptr(k_pool), _ptr(v_pool),
                            _ptr(block_table), _ptr(cache_lens), _stream()))


PA_DECODE_STATIC_SCRATCH_BYTES = 4 << 20


def pa_decode_static(q, k_cache, v_cache, cache_lens, window_blocks: int, sink_blocks: int, o, lse,
                     block: int = 64, softmax_scale: float = 0.0):
    """pa_decode for callers that may not allocate: the split-K scratch lives inside the library.

    Unlike the other wrappers this one never creates a tensor: `o` [batch, Hq, D] and `lse`
    [batch, Hq] must be passed in.  Problems whose scratch would exceed
    PA_DECODE_STATIC_SCRATCH_BYTES raise PaError(PA_ERR_WORKSPACE).  Calls that overlap on the GPU
    share (and would corrupt) the one built-in scratch array: keep them on one stream.
    """
    assert cache_lens.dtype == torch.int32 and q.is_contiguous() and o.is_contiguous()
    params = decode_params(q, k_cache, v_cache, window_blocks, sink_blocks, block, softmax_scale, o.dtype)
    _check(lib.pa_decode_static(ctypes.byref(params), _ptr(q), _ptr(k_cache), _ptr(v_cache), _ptr(cache_lens),
                                _ptr(o), _ptr(lse), _stream()))
    return o, lse
