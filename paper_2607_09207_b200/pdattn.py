"""ctypes binding of libpdattn (include/pdattn.h): argument marshalling only.

Every step of the decode path runs in the library's CUDA kernels.  torch is used for device
memory and streams.  There is no CPU fallback: if the library has not been built, importing
`lib()` raises.
"""
from __future__ import annotations

import ctypes
import os
from typing import Optional

import numpy as np
import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "lib", "libpdattn.so")

OK = 0
INVALID_ARG = -1
UNSUPPORTED = -2
WORKSPACE_TOO_SMALL = -3
MISALIGNED = -4
NOT_BOUND = -5
CUDA_ERROR = -6
BAD_PAGE_INDEX = -7
DEVICE_TIMEOUT = -8

EXPORTS = [
    "pdattn_workspace_size", "pdattn_workspace_init", "pdattn_decode_ex", "pdattn_bind", "pdattn_decode",
    "pdattn_decode_host_fp8", "pdattn_decode_grouped_fp8",
    "pdattn_host_staging_size", "pdattn_decode_host", "pdattn_plan_host", "pdattn_check",
    "pdattn_last_launch_count", "pdattn_status_string", "pdattn_last_cuda_error", "pdattn_profile_events",
    "pdattn_gather_probe", "pdattn_stream_read_probe", "pdattn_wait_limit_probe", "pdattn_set_dynamic_spans",
    "pdattn_set_merge_mode", "pdattn_set_prefix_engine", "pdattn_set_host_zero_copy", "pdattn_set_short_piece_path",
    "pdattn_decode_static_scratch", "pdattn_append_kv",
    "pdattn_grouped_workspace_size", "pdattn_decode_grouped",
    "pdattn_multi_workspace_size", "pdattn_decode_multi", "pdattn_decode_fp8", "pdattn_append_kv_fp8", "pdattn_decode_fp8_multi",
]


class PdattnError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        L = lib()
        msg = L.pdattn_status_string(status).decode()
        if status == CUDA_ERROR:
            msg += ": " + L.pdattn_last_cuda_error().decode()
        super().__init__(f"{where}: {msg} ({status})")


class Args(ctypes.Structure):
    _fields_ = [
        ("q", ctypes.c_void_p), ("k_cache", ctypes.c_void_p), ("v_cache", ctypes.c_void_p),
        ("out", ctypes.c_void_p), ("block_table", ctypes.c_void_p), ("context_lens", ctypes.c_void_p),
        ("context_lens_host", ctypes.c_void_p),
        ("num_seqs", ctypes.c_int), ("num_q_heads", ctypes.c_int), ("num_kv_heads", ctypes.c_int),
        ("head_dim", ctypes.c_int), ("block_size", ctypes.c_int),
        ("max_blocks_per_seq", ctypes.c_int), ("num_blocks", ctypes.c_int),
        ("kv_block_stride", ctypes.c_int64), ("kv_head_stride", ctypes.c_int64), ("kv_token_stride", ctypes.c_int64),
        ("scale", ctypes.c_float),
        ("workspace", ctypes.c_void_p), ("workspace_bytes", ctypes.c_size_t),
    ]


class Plan(ctypes.Structure):
    _fields_ = [("n_static", ctypes.c_int), ("n_dynamic", ctypes.c_int), ("total_tiles", ctypes.c_int)]


_lib = None


def lib():
    """The loaded C-ABI library.  Raises if it has not been built (see build.py)."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise RuntimeError(
                f"{LIB_PATH} is missing: build it with `python -m paper_2607_09207_b200.build` "
                "(there is no fallback path)")
        L = ctypes.CDLL(LIB_PATH)
        vp, i32, i64, f32, sz = ctypes.c_void_p, ctypes.c_int, ctypes.c_int64, ctypes.c_float, ctypes.c_size_t
        L.pdattn_workspace_size.argtypes = [i32] * 6 + [ctypes.POINTER(sz), ctypes.POINTER(sz)]
        L.pdattn_workspace_init.argtypes = [vp, sz, vp]
        L.pdattn_decode_ex.argtypes = [ctypes.POINTER(Args), vp]
        L.pdattn_bind.argtypes = [i32, i32, vp, sz, vp]
        L.pdattn_decode.argtypes = [vp, vp, vp, vp, vp, i32, i32, i32, i32, i32, f32, vp, vp]
        L.pdattn_host_staging_size.argtypes = [i32, i32, i32, i32, ctypes.POINTER(sz)]
        L.pdattn_decode_host.argtypes = [vp, vp, vp, vp, vp, vp, i32, i32, i32, i32, i32, i32, i32, f32,
                                         vp, sz, vp, sz, vp]
        L.pdattn_plan_host.argtypes = [vp, i32, i32, i32, i32, i32, vp, ctypes.POINTER(Plan)]
        L.pdattn_set_dynamic_spans.argtypes = [i32]
        L.pdattn_set_merge_mode.argtypes = [i32]
        L.pdattn_set_prefix_engine.argtypes = [i32]
        L.pdattn_set_short_piece_path.argtypes = [i32]
        L.pdattn_set_host_zero_copy.argtypes = [i32]
        L.pdattn_decode_static_scratch.argtypes = [ctypes.POINTER(Args), vp, vp]
        L.pdattn_grouped_workspace_size.argtypes = [i32, i32, i32, i32, i32, ctypes.POINTER(sz)]
        L.pdattn_decode_grouped.argtypes = [ctypes.POINTER(Args), i32, vp, vp, vp]
        L.pdattn_decode_grouped_fp8.argtypes = [ctypes.POINTER(Args), i32, vp, vp, vp, vp, vp]
        L.pdattn_decode_host_fp8.argtypes = [vp, vp, vp, vp, vp, vp, vp, vp, i32, i32, i32, i32, i32, i32, i32, f32,
                                             vp, sz, vp, sz, vp]
        L.pdattn_multi_workspace_size.argtypes = [i32, i32, i32, i32, i32, i32, ctypes.POINTER(sz)]
        L.pdattn_decode_multi.argtypes = [ctypes.POINTER(Args), i32, vp]
        L.pdattn_decode_fp8.argtypes = [ctypes.POINTER(Args), vp, vp, vp]
        L.pdattn_decode_fp8_multi.argtypes = [ctypes.POINTER(Args), i32, vp, vp, vp]
        L.pdattn_append_kv_fp8.argtypes = [vp, vp, vp, vp, vp, vp, vp, vp, i32, i32, i32, i32, i32, i32, vp, vp]
        L.pdattn_append_kv.argtypes = [vp, vp, vp, vp, vp, vp, i32, i32, i32, i32, i32, i32, i64, i64, i64, vp, vp]
        L.pdattn_check.argtypes = [vp, vp]
        L.pdattn_profile_events.argtypes = [vp, vp]
        L.pdattn_gather_probe.argtypes = [ctypes.POINTER(Args), vp]
        L.pdattn_stream_read_probe.argtypes = [vp, sz, vp, vp]
        L.pdattn_wait_limit_probe.argtypes = [vp, i32, vp]
        L.pdattn_last_launch_count.argtypes = []
        L.pdattn_status_string.argtypes = [i32]
        L.pdattn_status_string.restype = ctypes.c_char_p
        L.pdattn_last_cuda_error.argtypes = []
        L.pdattn_last_cuda_error.restype = ctypes.c_char_p
        _lib = L
    return _lib


def _stream_ptr(stream) -> int:
    if stream is None:
        stream = torch.cuda.current_stream()
    return int(stream.cuda_stream)


def workspace_size(num_seqs, num_q_heads, num_kv_heads, head_dim, block_size=16, max_context_len=0) -> int:
    dev, pin = ctypes.c_size_t(0), ctypes.c_size_t(0)
    st = lib().pdattn_workspace_size(num_seqs, num_q_heads, num_kv_heads, head_dim, block_size, max_context_len,
                                     ctypes.byref(dev), ctypes.byref(pin))
    if st != OK:
        raise PdattnError(st, "pdattn_workspace_size")
    return dev.value


def alloc_workspace(num_seqs, num_q_heads, num_kv_heads, head_dim, block_size=16, device="cuda", stream=None):
    """torch-owned workspace, error word cleared."""
    n = workspace_size(num_seqs, num_q_heads, num_kv_heads, head_dim, block_size)
    ws = torch.empty(n, dtype=torch.uint8, device=device)
    st = lib().pdattn_workspace_init(ws.data_ptr(), n, _stream_ptr(stream))
    if st != OK:
        raise PdattnError(st, "pdattn_workspace_init")
    return ws


def decode_ex(q, k_cache, v_cache, block_table, context_lens, scale, out, workspace,
              context_lens_host: Optional[np.ndarray] = None, num_blocks: Optional[int] = None,
              stream=None, check: bool = True, probe: bool = False) -> int:
    """pdattn_decode_ex.  k_cache / v_cache: bf16 tensors indexed [page, kv_head, slot, dim] with any
    strides whose last dimension is contiguous.  Returns the status (raises unless check=False)."""
    S, Hq, d = q.shape
    NB, Hkv, bs, _ = k_cache.shape
    a = Args()
    a.q, a.k_cache, a.v_cache, a.out = q.data_ptr(), k_cache.data_ptr(), v_cache.data_ptr(), out.data_ptr()
    a.block_table, a.context_lens = block_table.data_ptr(), context_lens.data_ptr()
    keep = None
    if context_lens_host is not None:
        keep = np.ascontiguousarray(context_lens_host, dtype=np.int32)
        a.context_lens_host = keep.ctypes.data
    else:
        a.context_lens_host = None
    a.num_seqs, a.num_q_heads, a.num_kv_heads, a.head_dim, a.block_size = S, Hq, Hkv, d, bs
    a.max_blocks_per_seq = block_table.shape[1] if block_table.dim() == 2 else 0
    a.num_blocks = NB if num_blocks is None else num_blocks
    a.kv_block_stride, a.kv_head_stride, a.kv_token_stride = k_cache.stride(0), k_cache.stride(1), k_cache.stride(2)
    a.scale = float(scale)
    a.workspace, a.workspace_bytes = workspace.data_ptr(), workspace.numel()
    fn = lib().pdattn_gather_probe if probe else lib().pdattn_decode_ex
    st = fn(ctypes.byref(a), _stream_ptr(stream))
    if check and st != OK:
        raise PdattnError(st, "pdattn_gather_probe" if probe else "pdattn_decode_ex")
    return st


def decode_static_scratch(q, k_cache, v_cache, block_table, context_lens, scale, out,
                          context_lens_host: Optional[np.ndarray] = None, status_out: Optional[torch.Tensor] = None,
                          stream=None, check: bool = True) -> int:
    """pdattn_decode_static_scratch: the decode step on the library's built-in scratch array, for callers
    that can neither provide a workspace nor let the library allocate one.  status_out: optional int32
    device tensor of one element that receives this call's error bits."""
    S, Hq, d = q.shape
    NB, Hkv, bs, _ = k_cache.shape
    a = Args()
    a.q, a.k_cache, a.v_cache, a.out = q.data_ptr(), k_cache.data_ptr(), v_cache.data_ptr(), out.data_ptr()
    a.block_table, a.context_lens = block_table.data_ptr(), context_lens.data_ptr()
    keep = None
    if context_lens_host is not None:
        keep = np.ascontiguousarray(context_lens_host, dtype=np.int32)
        a.context_lens_host = keep.ctypes.data
    a.num_seqs, a.num_q_heads, a.num_kv_heads, a.head_dim, a.block_size = S, Hq, Hkv, d, bs
    a.max_blocks_per_seq = block_table.shape[1] if block_table.dim() == 2 else 0
    a.num_blocks = NB
    a.kv_block_stride, a.kv_head_stride, a.kv_token_stride = k_cache.stride(0), k_cache.stride(1), k_cache.stride(2)
    a.scale = float(scale)
    st = lib().pdattn_decode_static_scratch(ctypes.byref(a), status_out.data_ptr() if status_out is not None else None,
                                            _stream_ptr(stream))
    if check and st != OK:
        raise PdattnError(st, "pdattn_decode_static_scratch")
    return st


def grouped_workspace_size(num_seqs, num_q_heads, num_kv_heads, head_dim, block_size=16) -> int:
    n = ctypes.c_size_t(0)
    st = lib().pdattn_grouped_workspace_size(num_seqs, num_q_heads, num_kv_heads, head_dim, block_size, ctypes.byref(n))
    if st != OK:
        raise PdattnError(st, "pdattn_grouped_workspace_size")
    return n.value


def alloc_grouped_workspace(num_seqs, num_q_heads, num_kv_heads, head_dim, block_size=16, device="cuda", stream=None):
    n = grouped_workspace_size(num_seqs, num_q_heads, num_kv_heads, head_dim, block_size)
    ws = torch.empty(n, dtype=torch.uint8, device=device)
    st = lib().pdattn_workspace_init(ws.data_ptr(), n, _stream_ptr(stream))
    if st != OK:
        raise PdattnError(st, "pdattn_workspace_init")
    return ws


def decode_grouped(q, k_cache, v_cache, block_table, context_lens, scale, out, workspace, context_lens_host,
                   group_size, prefix_tiles, prefix_tiles_host, stream=None, check: bool = True) -> int:
    """pdattn_decode_grouped: sequences come in groups of `group_size` whose first prefix_tiles[g] * 64 tokens
    are the same physical pages (GRPO samples of one prompt); those tiles are read once per group."""
    S, Hq, d = q.shape
    NB, Hkv, bs, _ = k_cache.shape
    a = Args()
    a.q, a.k_cache, a.v_cache, a.out = q.data_ptr(), k_cache.data_ptr(), v_cache.data_ptr(), out.data_ptr()
    a.block_table, a.context_lens = block_table.data_ptr(), context_lens.data_ptr()
    lens = np.ascontiguousarray(context_lens_host, dtype=np.int32)
    a.context_lens_host = lens.ctypes.data
    a.num_seqs, a.num_q_heads, a.num_kv_heads, a.head_dim, a.block_size = S, Hq, Hkv, d, bs
    a.max_blocks_per_seq = block_table.shape[1]
    a.num_blocks = NB
    a.kv_block_stride, a.kv_head_stride, a.kv_token_stride = k_cache.stride(0), k_cache.stride(1), k_cache.stride(2)
    a.scale = float(scale)
    a.workspace, a.workspace_bytes = workspace.data_ptr(), workspace.numel()
    pth = np.ascontiguousarray(prefix_tiles_host, dtype=np.int32)
    st = lib().pdattn_decode_grouped(ctypes.byref(a), int(group_size), prefix_tiles.data_ptr(), pth.ctypes.data,
                                     _stream_ptr(stream))
    if check and st != OK:
        raise PdattnError(st, "pdattn_decode_grouped")
    return st


def multi_workspace_size(num_seqs, num_q_heads, num_kv_heads, head_dim, block_size, num_query_tokens) -> int:
    n = ctypes.c_size_t(0)
    st = lib().pdattn_multi_workspace_size(num_seqs, num_q_heads, num_kv_heads, head_dim, block_size,
                                           num_query_tokens, ctypes.byref(n))
    if st != OK:
        raise PdattnError(st, "pdattn_multi_workspace_size")
    return n.value


def alloc_multi_workspace(num_seqs, num_q_heads, num_kv_heads, head_dim, block_size, num_query_tokens,
                          device="cuda", stream=None):
    n = multi_workspace_size(num_seqs, num_q_heads, num_kv_heads, head_dim, block_size, num_query_tokens)
    ws = torch.empty(n, dtype=torch.uint8, device=device)
    st = lib().pdattn_workspace_init(ws.data_ptr(), n, _stream_ptr(stream))
    if st != OK:
        raise PdattnError(st, "pdattn_workspace_init")
    return ws


def decode_multi(q, k_cache, v_cache, block_table, context_lens, scale, out, workspace, context_lens_host=None,
                 stream=None, check: bool = True) -> int:
    """pdattn_decode_multi: q and out are [num_seqs, T, num_q_heads, head_dim]; the last T tokens of every
    sequence are new and each attends to the keys up to its own position."""
    S, T, Hq, d = q.shape
    NB, Hkv, bs, _ = k_cache.shape
    a = Args()
    a.q, a.k_cache, a.v_cache, a.out = q.data_ptr(), k_cache.data_ptr(), v_cache.data_ptr(), out.data_ptr()
    a.block_table, a.context_lens = block_table.data_ptr(), context_lens.data_ptr()
    lens = None
    if context_lens_host is not None:
        lens = np.ascontiguousarray(context_lens_host, dtype=np.int32)
        a.context_lens_host = lens.ctypes.data
    a.num_seqs, a.num_q_heads, a.num_kv_heads, a.head_dim, a.block_size = S, Hq, Hkv, d, bs
    a.max_blocks_per_seq = block_table.shape[1]
    a.num_blocks = NB
    a.kv_block_stride, a.kv_head_stride, a.kv_token_stride = k_cache.stride(0), k_cache.stride(1), k_cache.stride(2)
    a.scale = float(scale)
    a.workspace, a.workspace_bytes = workspace.data_ptr(), workspace.numel()
    st = lib().pdattn_decode_multi(ctypes.byref(a), int(T), _stream_ptr(stream))
    if check and st != OK:
        raise PdattnError(st, "pdattn_decode_multi")
    return st


def decode_fp8(q, k8, v8, k_scale, v_scale, block_table, context_lens, scale, out, workspace,
               context_lens_host=None, stream=None, check: bool = True) -> int:
    """pdattn_decode_fp8: k8 uint8 [pages, Hkv, block_size, d], v8 uint8 [pages, Hkv, d, block_size] (e4m3 codes),
    k_scale / v_scale fp32 [Hkv] on the device."""
    T = q.shape[1] if q.dim() == 4 else 0          # [S, T, Hq, d]: several new tokens per sequence
    S, Hq, d = q.shape[0], q.shape[-2], q.shape[-1]
    NB, Hkv, bs, _ = k8.shape
    assert k8.dtype == torch.uint8 and v8.dtype == torch.uint8 and tuple(v8.shape) == (NB, Hkv, d, bs)
    assert k8.is_contiguous() and v8.is_contiguous() and k_scale.dtype == torch.float32 and v_scale.dtype == torch.float32
    a = Args()
    a.q, a.k_cache, a.v_cache, a.out = q.data_ptr(), k8.data_ptr(), v8.data_ptr(), out.data_ptr()
    a.block_table, a.context_lens = block_table.data_ptr(), context_lens.data_ptr()
    lens = None
    if context_lens_host is not None:
        lens = np.ascontiguousarray(context_lens_host, dtype=np.int32)
        a.context_lens_host = lens.ctypes.data
    a.num_seqs, a.num_q_heads, a.num_kv_heads, a.head_dim, a.block_size = S, Hq, Hkv, d, bs
    a.max_blocks_per_seq = block_table.shape[1]
    a.num_blocks = NB
    a.kv_block_stride, a.kv_head_stride, a.kv_token_stride = Hkv * bs * d, bs * d, d
    a.scale = float(scale)
    a.workspace, a.workspace_bytes = workspace.data_ptr(), workspace.numel()
    if T:
        st = lib().pdattn_decode_fp8_multi(ctypes.byref(a), T, k_scale.data_ptr(), v_scale.data_ptr(), _stream_ptr(stream))
    else:
        st = lib().pdattn_decode_fp8(ctypes.byref(a), k_scale.data_ptr(), v_scale.data_ptr(), _stream_ptr(stream))
    if check and st != OK:
        raise PdattnError(st, "pdattn_decode_fp8")
    return st


def decode_grouped_fp8(q, k8, v8, k_scale, v_scale, block_table, context_lens, scale, out, workspace,
                       context_lens_host, group_size, prefix_tiles, prefix_tiles_host, stream=None,
                       check: bool = True) -> int:
    """pdattn_decode_grouped_fp8: decode_grouped over the e4m3 code pools of decode_fp8."""
    S, Hq, d = q.shape
    NB, Hkv, bs, _ = k8.shape
    assert k8.dtype == torch.uint8 and v8.dtype == torch.uint8 and tuple(v8.shape) == (NB, Hkv, d, bs)
    assert k8.is_contiguous() and v8.is_contiguous()
    a = Args()
    a.q, a.k_cache, a.v_cache, a.out = q.data_ptr(), k8.data_ptr(), v8.data_ptr(), out.data_ptr()
    a.block_table, a.context_lens = block_table.data_ptr(), context_lens.data_ptr()
    lens = np.ascontiguousarray(context_lens_host, dtype=np.int32)
    a.context_lens_host = lens.ctypes.data
    a.num_seqs, a.num_q_heads, a.num_kv_heads, a.head_dim, a.block_size = S, Hq, Hkv, d, bs
    a.max_blocks_per_seq = block_table.shape[1]
    a.num_blocks = NB
    a.kv_block_stride, a.kv_head_stride, a.kv_token_stride = Hkv * bs * d, bs * d, d
    a.scale = float(scale)
    a.workspace, a.workspace_bytes = workspace.data_ptr(), workspace.numel()
    pth = np.ascontiguousarray(prefix_tiles_host, dtype=np.int32)
    st = lib().pdattn_decode_grouped_fp8(ctypes.byref(a), int(group_size), prefix_tiles.data_ptr(), pth.ctypes.data,
                                         k_scale.data_ptr(), v_scale.data_ptr(), _stream_ptr(stream))
    if check and st != OK:
        raise PdattnError(st, "pdattn_decode_grouped_fp8")
    return st


def decode_host_fp8(q_host, block_table_host, context_lens_host, out_host, k8, v8, k_scale, v_scale, scale, staging,
                    workspace, stream=None, check: bool = True) -> int:
    """pdattn_decode_host_fp8: q / block_table / context_lens / out are HOST tensors (pinned), code pools and scales
    on the device."""
    S, Hq, d = q_host.shape
    NB, Hkv, bs, _ = k8.shape
    st = lib().pdattn_decode_host_fp8(q_host.data_ptr(), block_table_host.data_ptr(), context_lens_host.data_ptr(),
                                      out_host.data_ptr(), k8.data_ptr(), v8.data_ptr(), k_scale.data_ptr(),
                                      v_scale.data_ptr(), S, Hq, Hkv, d, bs, block_table_host.shape[1], NB, float(scale),
                                      staging.data_ptr(), staging.numel(), workspace.data_ptr(), workspace.numel(),
                                      _stream_ptr(stream))
    if check and st != OK:
        raise PdattnError(st, "pdattn_decode_host_fp8")
    return st


def append_kv_fp8(k_new, v_new, k8, v8, k_scale, v_scale, block_table, context_lens, workspace=None, stream=None,
                  check: bool = True) -> int:
    """pdattn_append_kv_fp8: quantise the new K/V rows into the fp8 cache and advance context_lens (device, in place)."""
    S, Hkv, d = k_new.shape
    NB, _, bs, _ = k8.shape
    st = lib().pdattn_append_kv_fp8(k_new.data_ptr(), v_new.data_ptr(), k8.data_ptr(), v8.data_ptr(), k_scale.data_ptr(),
                                    v_scale.data_ptr(), block_table.data_ptr(), context_lens.data_ptr(), S, Hkv, d, bs,
                                    block_table.shape[1], NB, workspace.data_ptr() if workspace is not None else None,
                                    _stream_ptr(stream))
    if check and st != OK:
        raise PdattnError(st, "pdattn_append_kv_fp8")
    return st


def append_kv(k_new, v_new, k_cache, v_cache, block_table, context_lens, workspace=None, stream=None,
              check: bool = True) -> int:
    """pdattn_append_kv: write this step's K/V rows ([S, Hkv, d]) into the paged caches and advance
    context_lens (device tensor, in place)."""
    S, Hkv, d = k_new.shape
    NB, _, bs, _ = k_cache.shape
    st = lib().pdattn_append_kv(k_new.data_ptr(), v_new.data_ptr(), k_cache.data_ptr(), v_cache.data_ptr(),
                                block_table.data_ptr(), context_lens.data_ptr(), S, Hkv, d, bs, block_table.shape[1],
                                NB, k_cache.stride(0), k_cache.stride(1), k_cache.stride(2),
                                workspace.data_ptr() if workspace is not None else None, _stream_ptr(stream))
    if check and st != OK:
        raise PdattnError(st, "pdattn_append_kv")
    return st


def stream_read_probe(src: torch.Tensor, sink: torch.Tensor, stream=None):
    st = lib().pdattn_stream_read_probe(src.data_ptr(), src.numel() * src.element_size(), sink.data_ptr(),
                                        _stream_ptr(stream))
    if st != OK:
        raise PdattnError(st, "pdattn_stream_read_probe")


def bind(max_blocks_per_seq, num_blocks, workspace, context_lens_host: Optional[np.ndarray] = None):
    """pdattn_bind.  The caller keeps `workspace` and `context_lens_host` alive while bound."""
    hp = context_lens_host.ctypes.data if context_lens_host is not None else None
    st = lib().pdattn_bind(max_blocks_per_seq, num_blocks, workspace.data_ptr(), workspace.numel(), hp)
    if st != OK:
        raise PdattnError(st, "pdattn_bind")


def decode(q, k_cache, v_cache, block_table, context_lens, num_seqs, num_q_heads, num_kv_heads, head_dim,
           block_size, scale, out, stream=None, check: bool = True) -> int:
    """pdattn_decode (13-argument form, dense [NB, Hkv, bs, d] caches, uses the thread's binding)."""
    st = lib().pdattn_decode(q.data_ptr(), k_cache.data_ptr(), v_cache.data_ptr(), block_table.data_ptr(),
                             context_lens.data_ptr(), num_seqs, num_q_heads, num_kv_heads, head_dim, block_size,
                             float(scale), out.data_ptr(), _stream_ptr(stream))
    if check and st != OK:
        raise PdattnError(st, "pdattn_decode")
    return st


def host_staging_size(num_seqs, num_q_heads, head_dim, max_blocks_per_seq) -> int:
    n = ctypes.c_size_t(0)
    st = lib().pdattn_host_staging_size(num_seqs, num_q_heads, head_dim, max_blocks_per_seq, ctypes.byref(n))
    if st != OK:
        raise PdattnError(st, "pdattn_host_staging_size")
    return n.value


def decode_host(q_host, block_table_host, context_lens_host, out_host, k_cache, v_cache, scale, staging, workspace,
                stream=None, check: bool = True) -> int:
    """pdattn_decode_host: q / block_table / context_lens / out are HOST tensors (pinned), caches on device."""
    S, Hq, d = q_host.shape
    NB, Hkv, bs, _ = k_cache.shape
    st = lib().pdattn_decode_host(q_host.data_ptr(), block_table_host.data_ptr(), context_lens_host.data_ptr(),
                                  out_host.data_ptr(), k_cache.data_ptr(), v_cache.data_ptr(), S, Hq, Hkv, d, bs,
                                  block_table_host.shape[1], NB, float(scale), staging.data_ptr(), staging.numel(),
                                  workspace.data_ptr(), workspace.numel(), _stream_ptr(stream))
    if check and st != OK:
        raise PdattnError(st, "pdattn_decode_host")
    return st


class HostStep:
    """pdattn_decode_host for a decode loop that reuses its buffers: the engine rewrites q_host, block_table_host
    and context_lens_host in place every step and reads out_host after synchronising the stream.  The arguments
    are marshalled once, so a step is a single foreign call (argument marshalling only; same entry point, same
    results as decode_host)."""

    def __init__(self, q_host, block_table_host, context_lens_host, out_host, k_cache, v_cache, scale, staging,
                 workspace, stream=None):
        S, Hq, d = q_host.shape
        NB, Hkv, bs, _ = k_cache.shape
        self._keep = (q_host, block_table_host, context_lens_host, out_host, k_cache, v_cache, staging, workspace)
        vp, ci = ctypes.c_void_p, ctypes.c_int
        self._args = (vp(q_host.data_ptr()), vp(block_table_host.data_ptr()), vp(context_lens_host.data_ptr()),
                      vp(out_host.data_ptr()), vp(k_cache.data_ptr()), vp(v_cache.data_ptr()), ci(S), ci(Hq), ci(Hkv),
                      ci(d), ci(bs), ci(block_table_host.shape[1]), ci(NB), ctypes.c_float(float(scale)),
                      vp(staging.data_ptr()), ctypes.c_size_t(staging.numel()), vp(workspace.data_ptr()),
                      ctypes.c_size_t(workspace.numel()), vp(_stream_ptr(stream)))
        self._fn = lib().pdattn_decode_host

    def __call__(self, check: bool = True) -> int:
        st = self._fn(*self._args)
        if check and st != OK:
            raise PdattnError(st, "pdattn_decode_host")
        return st


def set_dynamic_spans(per_cta: int):
    st = lib().pdattn_set_dynamic_spans(per_cta)
    if st != OK:
        raise PdattnError(st, "pdattn_set_dynamic_spans")


def set_merge_mode(mode: int):
    """-1: default (1 for batches of long sequences with host lengths, else 2); 0: barrier merge + combine kernel; 1: chained merge + final merge of cut units inside the
    decode kernel; 2: chained merge + combine kernel."""
    st = lib().pdattn_set_merge_mode(mode)
    if st != OK:
        raise PdattnError(st, "pdattn_set_merge_mode")


def set_short_piece_path(mode: int):
    """-1: the short-piece kernel instantiation for batches below 1.5 tiles per unit on average (default); 0: never; 1: whenever
    it applies (chained merge, bf16 cache, at most 8 query rows per KV head, host lengths)."""
    st = lib().pdattn_set_short_piece_path(mode)
    if st != OK:
        raise PdattnError(st, "pdattn_set_short_piece_path")


def set_prefix_engine(engine: int):
    """-1: default (tcgen05); 0: warp-level MMAs; 1: tcgen05 with tensor-memory accumulators."""
    st = lib().pdattn_set_prefix_engine(engine)
    if st != OK:
        raise PdattnError(st, "pdattn_set_prefix_engine")


def set_host_zero_copy(mode: int):
    """-1 / 1: decode_host uses pinned, mapped q and out in place; 0: always through the staging copies."""
    st = lib().pdattn_set_host_zero_copy(mode)
    if st != OK:
        raise PdattnError(st, "pdattn_set_host_zero_copy")


def wait_limit_probe(workspace, limit_us: int, stream=None) -> int:
    """One warp waits limit_us microseconds on a barrier nothing arrives on, then raises the timeout bit."""
    return lib().pdattn_wait_limit_probe(workspace.data_ptr(), int(limit_us), _stream_ptr(stream))


def plan_host(context_lens_host, num_kv_heads, n_ctas, dynamic_per_cta=0, max_spans=None):
    """pdattn_plan_host -> (spans[n_spans + 1, 4], Plan).  Row i is (unit, tile, flat, 0); span i holds
    spans[i + 1, 2] - spans[i, 2] tiles.  Needs no GPU."""
    lens = np.ascontiguousarray(context_lens_host, dtype=np.int32)
    if max_spans is None:
        max_spans = n_ctas * 9
    spans = np.zeros((max_spans + 1, 4), dtype=np.int32)
    plan = Plan()
    st = lib().pdattn_plan_host(lens.ctypes.data if lens.size else None, lens.size, num_kv_heads, n_ctas,
                                dynamic_per_cta, max_spans, spans.ctypes.data, ctypes.byref(plan))
    if st != OK:
        raise PdattnError(st, "pdattn_plan_host")
    return spans[: plan.n_static + plan.n_dynamic + 1].copy(), plan


def check(workspace, stream=None) -> int:
    """pdattn_check: synchronises, returns OK / BAD_PAGE_INDEX / DEVICE_TIMEOUT and clears the word."""
    return lib().pdattn_check(workspace.data_ptr(), _stream_ptr(stream))


def last_launch_count() -> int:
    return lib().pdattn_last_launch_count()


def decode_workload(w, out=None, workspace=None, use_host_lens: bool = True, stream=None):
    """Convenience for tests and the benchmark: run one step on a workloads.Workload living on the GPU."""
    if out is None:
        out = torch.empty_like(w.q)
    if workspace is None:
        workspace = alloc_workspace(w.num_seqs, w.num_q_heads, w.num_kv_heads, w.head_dim, w.block_size,
                                    device=w.q.device)
    decode_ex(w.q, w.k_cache, w.v_cache, w.block_table, w.context_lens, w.scale, out, workspace,
              context_lens_host=w.context_lens_host if use_host_lens else None, stream=stream)
    return out
