"""Thin Python binding of libpagedkv.so: argument marshalling only.

Every function has the name and the meaning of the C entry point it forwards to (see
include/pagedkv.h).  Tensors are torch tensors used as plain device (or pinned host)
buffers; nothing is computed here, and there is no fallback: if the CUDA library cannot be
loaded, importing the functions' results fails loudly.
"""
from __future__ import annotations

import ctypes
import os
from typing import Optional

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libpagedkv.so")

PA_OK = 0
PA_BF16 = 1
PA_FLAG_REUSE_PLAN = 1
PA_STATUS_BAD_SEQ_LEN = 1
PA_STATUS_BAD_BLOCK_ID = 2
PA_STATUS_TIMEOUT = 4
PA_STATUS_WORKSPACE = 8
ERR = {"NULL": -1, "SHAPE": -2, "ALIGN": -3, "WORKSPACE": -4, "HOSTBUF": -5, "BLOCK_ID": -6,
       "CUDA": -7, "ARG": -8, "STATIC_LIMIT": -9}
PA_STATIC_WORKSPACE_BYTES = 64 << 20

EXPORTS = ["pa_workspace_bytes", "pa_decode", "pa_decode_strided", "pa_host_io_bytes", "pa_decode_host",
           "kv_block_bytes", "kv_swap_out", "kv_swap_in", "pa_status_string",
           "pa_last_cuda_error", "pa_launch_count", "pa_profile_enable", "pa_profile_read",
           "pa_decode_static", "kv_append", "pa_partial_floats", "pa_decode_partial",
           "pa_merge_partials",
           "pa_prefill_workspace_bytes", "pa_prefill", "pa_prefill_split",
           "pa_prefill_split_workspace_bytes", "pa_prefill_last_launch", "pa_prefill_select_launch", "pa_selftest_wait_expiry", "pa_probe_read", "pa_probe_tma_issue"]


class PaShape(ctypes.Structure):
    _fields_ = [("num_q_heads", ctypes.c_int32), ("num_kv_heads", ctypes.c_int32),
                ("head_dim", ctypes.c_int32), ("block_size", ctypes.c_int32),
                ("num_blocks", ctypes.c_int32), ("dtype", ctypes.c_int32),
                ("stride_block", ctypes.c_int64), ("stride_head", ctypes.c_int64),
                ("stride_tok", ctypes.c_int64)]


class KvPoolDesc(ctypes.Structure):
    _fields_ = [("num_layers", ctypes.c_int32), ("reserved", ctypes.c_int32),
                ("layer_stride_k", ctypes.c_int64), ("layer_stride_v", ctypes.c_int64)]


class PagedKVError(RuntimeError):
    def __init__(self, code: int, where: str):
        self.code = code
        msg = lib().pa_status_string(code).decode()
        if code == ERR["CUDA"]:
            msg += f" [cuda error {lib().pa_last_cuda_error()}]"
        super().__init__(f"{where}: {msg} ({code})")


_lib = None


def lib() -> ctypes.CDLL:
    """Load libpagedkv.so (built in-tree by paper_2602_07878_b200.build).  No fallback."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise RuntimeError(f"{LIB_PATH} is missing: run `python -m paper_2602_07878_b200.build`")
        L = ctypes.CDLL(LIB_PATH)
        vp, i32, i64, sz = ctypes.c_void_p, ctypes.c_int32, ctypes.c_int64, ctypes.c_size_t
        psz = ctypes.POINTER(ctypes.c_size_t)
        pshape, ppool = ctypes.POINTER(PaShape), ctypes.POINTER(KvPoolDesc)
        L.pa_workspace_bytes.argtypes = [pshape, i32, i64, i32, psz]
        L.pa_decode.argtypes = [pshape, vp, vp, vp, vp, i32, vp, i32, ctypes.c_float, vp, vp, sz,
                                i32, i32, vp, vp]
        L.pa_decode_static.argtypes = [pshape, vp, vp, vp, vp, i32, vp, i32, i64, ctypes.c_float,
                                       vp, i32, vp, vp]
        L.pa_decode_static.restype = ctypes.c_int
        L.pa_partial_floats.argtypes = [pshape, i32, psz]
        L.pa_partial_floats.restype = ctypes.c_int
        L.pa_decode_partial.argtypes = [pshape, vp, vp, vp, vp, i32, vp, i32, ctypes.c_float, vp,
                                        vp, sz, i32, vp, vp]
        L.pa_decode_partial.restype = ctypes.c_int
        L.pa_merge_partials.argtypes = [ctypes.POINTER(vp), i32, i32, i32, vp, vp]
        L.pa_merge_partials.restype = ctypes.c_int
        L.pa_prefill_workspace_bytes.argtypes = [i32, psz]
        L.pa_prefill_workspace_bytes.restype = ctypes.c_int
        L.pa_prefill.argtypes = [pshape, vp, vp, vp, vp, i32, vp, vp, i32, i32, ctypes.c_float, vp,
                                 vp, sz, vp, vp]
        L.pa_prefill.restype = ctypes.c_int
        L.pa_prefill_split.argtypes = [pshape, vp, vp, vp, vp, i32, vp, vp, i32, i32,
                                       ctypes.c_float, vp, vp, sz, i32, vp, vp]
        L.pa_prefill_split.restype = ctypes.c_int
        L.pa_prefill_split_workspace_bytes.argtypes = [pshape, i32, i32, i32, psz]
        L.pa_prefill_split_workspace_bytes.restype = ctypes.c_int
        pi32 = ctypes.POINTER(ctypes.c_int32)
        L.pa_prefill_last_launch.argtypes = [pi32, pi32, pi32]
        L.pa_prefill_last_launch.restype = ctypes.c_int
        L.pa_prefill_select_launch.argtypes = [pshape, i32, i32, i32, sz, i32, i32, pi32, pi32, pi32]
        L.pa_prefill_select_launch.restype = ctypes.c_int
        L.pa_selftest_wait_expiry.argtypes = [i32, vp, vp]
        L.pa_selftest_wait_expiry.restype = ctypes.c_int
        L.pa_probe_read.argtypes = [vp, sz, i32, ctypes.c_uint32, vp, vp, vp]
        L.pa_probe_read.restype = ctypes.c_int
        L.pa_probe_tma_issue.argtypes = [vp, sz, i32, i32, i32, ctypes.POINTER(ctypes.c_int64), vp, vp]
        L.pa_probe_tma_issue.restype = ctypes.c_int
        L.kv_append.argtypes = [pshape, vp, vp, vp, vp, vp, i32, vp, vp]
        L.kv_append.restype = ctypes.c_int
        L.pa_decode_strided.argtypes = [pshape, vp, ctypes.c_int64, vp, vp, vp, i32, vp, i32,
                                        ctypes.c_float, vp, ctypes.c_int64, vp, sz, i32, i32, vp, vp]
        L.pa_decode_strided.restype = ctypes.c_int
        L.pa_host_io_bytes.argtypes = [pshape, i32, i32, psz]
        L.pa_decode_host.argtypes = [pshape, vp, vp, vp, vp, i32, vp, i32, ctypes.c_float, vp, vp,
                                     sz, vp, sz, i32, vp, vp]
        L.kv_block_bytes.argtypes = [ppool, pshape, psz]
        L.kv_swap_out.argtypes = [ppool, pshape, vp, vp, vp, i32, vp, sz, vp, sz, vp]
        L.kv_swap_in.argtypes = [ppool, pshape, vp, vp, vp, sz, vp, i32, vp, sz, vp]
        for name in ("pa_workspace_bytes", "pa_decode", "pa_host_io_bytes", "pa_decode_host",
                     "kv_block_bytes", "kv_swap_out", "kv_swap_in", "pa_last_cuda_error"):
            getattr(L, name).restype = ctypes.c_int
        L.pa_status_string.argtypes = [ctypes.c_int]
        L.pa_status_string.restype = ctypes.c_char_p
        pd = ctypes.POINTER(ctypes.c_double)
        L.pa_profile_enable.argtypes = [ctypes.c_int]
        L.pa_profile_enable.restype = ctypes.c_int
        L.pa_profile_read.argtypes = [pd, pd, pd, ctypes.POINTER(ctypes.c_int64)]
        L.pa_profile_read.restype = ctypes.c_int
        L.pa_launch_count.argtypes = []
        L.pa_launch_count.restype = ctypes.c_int64
        _lib = L
    return _lib


def _check(rc: int, where: str):
    if rc != PA_OK:
        raise PagedKVError(rc, where)


def _ptr(t: Optional[torch.Tensor]):
    return None if t is None else ctypes.c_void_p(t.data_ptr())


def _stream(stream) -> ctypes.c_void_p:
    if stream is None:
        stream = torch.cuda.current_stream()
    return ctypes.c_void_p(stream.cuda_stream)


def shape_of(k_cache: torch.Tensor, num_q_heads: int) -> PaShape:
    """pa_shape of a cache tensor viewed as [num_blocks, num_kv_heads, block_size, head_dim]
    (any strides over the first three axes; the last axis must be contiguous)."""
    assert k_cache.dtype == torch.bfloat16 and k_cache.dim() == 4 and k_cache.stride(3) == 1
    nb, hkv, bs, d = k_cache.shape
    return PaShape(num_q_heads, hkv, d, bs, nb, PA_BF16, k_cache.stride(0), k_cache.stride(1),
                   k_cache.stride(2))


def pa_workspace_bytes(shape: PaShape, max_batch: int, max_total_tokens: int,
                       partition_tokens: int = 0) -> int:
    out = ctypes.c_size_t(0)
    _check(lib().pa_workspace_bytes(ctypes.byref(shape), max_batch, max_total_tokens,
                                    partition_tokens, ctypes.byref(out)), "pa_workspace_bytes")
    return int(out.value)


def pa_decode(q, k_cache, v_cache, block_tables, seq_lens, scale, out, workspace, *,
              partition_tokens: int = 0, flags: int = 0, dev_status=None, stream=None,
              shape: Optional[PaShape] = None):
    """Forward to pa_decode.  q/out [B,H,D] bf16; caches [NB,Hkv,bs,D] bf16 views of one
    layer; block_tables int32 [B,max_blocks]; seq_lens int32 [B]; workspace uint8."""
    if shape is None:
        shape = shape_of(k_cache, q.shape[1])
        assert v_cache.stride() == k_cache.stride() and v_cache.shape == k_cache.shape
    assert block_tables.dtype == torch.int32 and seq_lens.dtype == torch.int32
    assert block_tables.is_contiguous()
    max_blocks = block_tables.shape[1] if block_tables.dim() == 2 else 0
    if q.is_contiguous() and out.is_contiguous():
        rc = lib().pa_decode(ctypes.byref(shape), _ptr(q), _ptr(k_cache), _ptr(v_cache),
                             _ptr(block_tables), max_blocks, _ptr(seq_lens), q.shape[0],
                             float(scale), _ptr(out), _ptr(workspace),
                             workspace.numel() * workspace.element_size(), partition_tokens, flags,
                             _ptr(dev_status), _stream(stream))
        _check(rc, "pa_decode")
        return out
    # views into wider tensors (a rank's heads of a batch-wide q, the q part of a fused QKV
    # projection): each sequence's [H, D] rows must be contiguous, sequences may be further apart
    for t in (q, out):
        assert t.dim() == 3 and t.stride(2) == 1 and t.stride(1) == t.shape[2]
    rc = lib().pa_decode_strided(ctypes.byref(shape), _ptr(q), q.stride(0), _ptr(k_cache),
                                 _ptr(v_cache), _ptr(block_tables), max_blocks, _ptr(seq_lens),
                                 q.shape[0], float(scale), _ptr(out), out.stride(0),
                                 _ptr(workspace), workspace.numel() * workspace.element_size(),
                                 partition_tokens, flags, _ptr(dev_status), _stream(stream))
    _check(rc, "pa_decode_strided")
    return out


def pa_partial_floats(shape: PaShape, batch: int) -> int:
    out = ctypes.c_size_t(0)
    _check(lib().pa_partial_floats(ctypes.byref(shape), batch, ctypes.byref(out)),
           "pa_partial_floats")
    return int(out.value)


def pa_decode_partial(q, k_cache, v_cache, block_tables, seq_lens, scale, part, workspace, *,
                      partition_tokens: int = 0, dev_status=None, stream=None,
                      shape: Optional[PaShape] = None):
    """Forward to pa_decode_partial: attention over this rank's slice of every sequence,
    written to `part` (float32, B*H*(D+2) elements) as one partial record."""
    if shape is None:
        shape = shape_of(k_cache, q.shape[1])
        assert v_cache.stride() == k_cache.stride() and v_cache.shape == k_cache.shape
    assert block_tables.dtype == torch.int32 and seq_lens.dtype == torch.int32
    assert q.is_contiguous() and block_tables.is_contiguous()
    assert part.dtype == torch.float32 and part.is_contiguous()
    assert part.numel() >= q.shape[0] * q.shape[1] * (q.shape[2] + 2)
    rc = lib().pa_decode_partial(ctypes.byref(shape), _ptr(q), _ptr(k_cache), _ptr(v_cache),
                                 _ptr(block_tables),
                                 block_tables.shape[1] if block_tables.dim() == 2 else 0,
                                 _ptr(seq_lens), q.shape[0], float(scale), _ptr(part),
                                 _ptr(workspace), workspace.numel() * workspace.element_size(),
                                 partition_tokens, _ptr(dev_status), _stream(stream))
    _check(rc, "pa_decode_partial")
    return part


def pa_merge_partials(parts, rows: int, head_dim: int, out, stream=None):
    """Forward to pa_merge_partials.  `parts`: a list of float32 tensors (one record each), or
    one [R, rows*(D+2)] tensor as an all-gather leaves it; out bf16 [rows, D] (any shape with
    that many contiguous elements)."""
    if isinstance(parts, torch.Tensor):
        assert parts.dim() == 2 and parts.is_contiguous()
        parts = [parts[i] for i in range(parts.shape[0])]
    for t in parts:
        assert t.dtype == torch.float32 and t.is_contiguous()
        assert t.numel() >= rows * (head_dim + 2)
    assert out.dtype == torch.bfloat16 and out.is_contiguous() and out.numel() == rows * head_dim
    arr = (ctypes.c_void_p * max(1, len(parts)))(*[t.data_ptr() for t in parts])
    rc = lib().pa_merge_partials(arr, len(parts), rows, head_dim, _ptr(out), _stream(stream))
    _check(rc, "pa_merge_partials")
    return out


def pa_host_io_bytes(shape: PaShape, max_batch: int, max_blocks_per_seq: int) -> int:
    out = ctypes.c_size_t(0)
    _check(lib().pa_host_io_bytes(ctypes.byref(shape), max_batch, max_blocks_per_seq,
                                  ctypes.byref(out)), "pa_host_io_bytes")
    return int(out.value)


def pa_decode_host(q_host, k_cache, v_cache, block_tables_host, seq_lens_host, scale, out_host,
                   io_buf, workspace, *, partition_tokens: int = 0, dev_status=None, stream=None):
    """Forward to pa_decode_host: q / tables / lengths / out are pinned host tensors."""
    shape = shape_of(k_cache, q_host.shape[1])
    for t in (q_host, block_tables_host, seq_lens_host, out_host):
        assert not t.is_cuda and t.is_contiguous()
    rc = lib().pa_decode_host(ctypes.byref(shape), _ptr(q_host), _ptr(k_cache), _ptr(v_cache),
                              _ptr(block_tables_host), block_tables_host.shape[1],
                              _ptr(seq_lens_host), q_host.shape[0], float(scale), _ptr(out_host),
                              _ptr(io_buf), io_buf.numel() * io_buf.element_size(),
                              _ptr(workspace), workspace.numel() * workspace.element_size(),
                              partition_tokens, _ptr(dev_status), _stream(stream))
    _check(rc, "pa_decode_host")
    return out_host


def pool_desc(k_pool: torch.Tensor, v_pool: torch.Tensor, num_q_heads: int = 0):
    """(kv_pool_desc, pa_shape) of pools shaped [layers, NB, Hkv, bs, D]."""
    assert k_pool.dim() == 5 and k_pool.dtype == torch.bfloat16 and k_pool.stride(4) == 1
    assert v_pool.shape == k_pool.shape and v_pool.stride()[1:] == k_pool.stride()[1:]
    shape = shape_of(k_pool[0], num_q_heads or k_pool.shape[2])
    return KvPoolDesc(k_pool.shape[0], 0, k_pool.stride(0), v_pool.stride(0)), shape


def kv_block_bytes(k_pool, v_pool) -> int:
    pool, shape = pool_desc(k_pool, v_pool)
    out = ctypes.c_size_t(0)
    _check(lib().kv_block_bytes(ctypes.byref(pool), ctypes.byref(shape), ctypes.byref(out)),
           "kv_block_bytes")
    return int(out.value)


def _ids(block_ids):
    import numpy as np

    a = np.ascontiguousarray(block_ids, dtype=np.int32)
    return a, a.ctypes.data_as(ctypes.c_void_p)


def kv_swap_out(k_pool, v_pool, block_ids, pinned_host_buf, staging=None, stream=None):
    """Forward to kv_swap_out.  block_ids: host int32 sequence; pinned_host_buf: pinned
    uint8 tensor; staging: optional device uint8 tensor."""
    pool, shape = pool_desc(k_pool, v_pool)
    ids, pids = _ids(block_ids)
    rc = lib().kv_swap_out(ctypes.byref(pool), ctypes.byref(shape), _ptr(k_pool), _ptr(v_pool),
                           pids, len(ids), _ptr(pinned_host_buf),
                           pinned_host_buf.numel() * pinned_host_buf.element_size(),
                           _ptr(staging), 0 if staging is None else staging.numel() * staging.element_size(),
                           _stream(stream))
    _check(rc, "kv_swap_out")


def kv_swap_in(k_pool, v_pool, pinned_host_buf, block_ids, staging=None, stream=None):
    """Forward to kv_swap_in (arguments as kv_swap_out)."""
    pool, shape = pool_desc(k_pool, v_pool)
    ids, pids = _ids(block_ids)
    rc = lib().kv_swap_in(ctypes.byref(pool), ctypes.byref(shape), _ptr(k_pool), _ptr(v_pool),
                          _ptr(pinned_host_buf),
                          pinned_host_buf.numel() * pinned_host_buf.element_size(), pids, len(ids),
                          _ptr(staging), 0 if staging is None else staging.numel() * staging.element_size(),
                          _stream(stream))
    _check(rc, "kv_swap_in")


def pa_launch_count() -> int:
    return int(lib().pa_launch_count())


def pa_profile_enable(on: bool):
    _check(lib().pa_profile_enable(1 if on else 0), "pa_profile_enable")


def pa_profile_read():
    """(plan_ms, attention_ms, combine_ms, calls) summed over the calls recorded so far."""
    t = [ctypes.c_double(0) for _ in range(3)]
    n = ctypes.c_int64(0)
    _check(lib().pa_profile_read(ctypes.byref(t[0]), ctypes.byref(t[1]), ctypes.byref(t[2]),
                                 ctypes.byref(n)), "pa_profile_read")
    return t[0].value, t[1].value, t[2].value, int(n.value)


def pa_decode_static(q, k_cache, v_cache, block_tables, seq_lens, scale, out, max_total_tokens, *,
                     partition_tokens: int = 0, dev_status=None, stream=None):
    """Forward to pa_decode_static: pa_decode without a caller workspace.  The scratch is a
    fixed array inside the library (PA_STATIC_WORKSPACE_BYTES per GPU), shared by all calls,
    so calls must not overlap on the GPU; `max_total_tokens` bounds the sum of seq_lens."""
    shape = shape_of(k_cache, q.shape[1])
    assert v_cache.stride() == k_cache.stride() and v_cache.shape == k_cache.shape
    assert block_tables.dtype == torch.int32 and seq_lens.dtype == torch.int32
    assert q.is_contiguous() and out.is_contiguous() and block_tables.is_contiguous()
    rc = lib().pa_decode_static(ctypes.byref(shape), _ptr(q), _ptr(k_cache), _ptr(v_cache),
                                _ptr(block_tables), block_tables.shape[1], _ptr(seq_lens),
                                q.shape[0], int(max_total_tokens), float(scale), _ptr(out),
                                partition_tokens, _ptr(dev_status), _stream(stream))
    _check(rc, "pa_decode_static")
    return out


def kv_append(k_cache, v_cache, k_new, v_new, slot_mapping, *, dev_status=None, stream=None):
    """Forward to kv_append: write k_new/v_new [B,Hkv,D] into flat slots slot_mapping (int64
    [B], negative = skip) of one layer's caches [NB,Hkv,bs,D]."""
    shape = shape_of(k_cache, k_cache.shape[1])
    assert v_cache.stride() == k_cache.stride() and v_cache.shape == k_cache.shape
    assert slot_mapping.dtype == torch.int64 and k_new.is_contiguous() and v_new.is_contiguous()
    assert k_new.dtype == torch.bfloat16 and k_new.shape == v_new.shape
    rc = lib().kv_append(ctypes.byref(shape), _ptr(k_cache), _ptr(v_cache), _ptr(k_new),
                         _ptr(v_new), _ptr(slot_mapping), k_new.shape[0], _ptr(dev_status),
                         _stream(stream))
    _check(rc, "kv_append")


def pa_prefill_workspace_bytes(max_batch: int) -> int:
    out = ctypes.c_size_t(0)
    _check(lib().pa_prefill_workspace_bytes(max_batch, ctypes.byref(out)),
           "pa_prefill_workspace_bytes")
    return int(out.value)


def pa_prefill_split_workspace_bytes(shape: PaShape, max_batch: int, max_total_q: int,
                                     max_splits: int) -> int:
    out = ctypes.c_size_t(0)
    _check(lib().pa_prefill_split_workspace_bytes(ctypes.byref(shape), max_batch, max_total_q,
                                                  max_splits, ctypes.byref(out)),
           "pa_prefill_split_workspace_bytes")
    return int(out.value)


def pa_prefill_last_launch():
    """Forward to pa_prefill_last_launch: (tiles per CTA, split tokens, partial rows per row)."""
    a, b, c = ctypes.c_int32(0), ctypes.c_int32(0), ctypes.c_int32(0)
    _check(lib().pa_prefill_last_launch(ctypes.byref(a), ctypes.byref(b), ctypes.byref(c)),
           "pa_prefill_last_launch")
    return a.value, b.value, c.value


def pa_prefill_select_launch(shape: PaShape, batch: int, total_q: int, max_blocks_per_seq: int,
                             workspace_bytes: int, kv_split_tokens: int = 0, sm_count: int = 148):
    """Forward to pa_prefill_select_launch (host only): (tiles per CTA, split tokens, splits)."""
    a, b, c = ctypes.c_int32(0), ctypes.c_int32(0), ctypes.c_int32(0)
    _check(lib().pa_prefill_select_launch(ctypes.byref(shape), batch, total_q, max_blocks_per_seq,
                                          workspace_bytes, kv_split_tokens, sm_count,
                                          ctypes.byref(a), ctypes.byref(b), ctypes.byref(c)),
           "pa_prefill_select_launch")
    return a.value, b.value, c.value


def _prefill_args(q, k_cache, v_cache, block_tables, ctx_lens, cu_q_lens, out):
    shape = shape_of(k_cache, q.shape[1])
    assert v_cache.stride() == k_cache.stride() and v_cache.shape == k_cache.shape
    assert block_tables.dtype == torch.int32 and ctx_lens.dtype == torch.int32
    assert cu_q_lens.dtype == torch.int32 and cu_q_lens.numel() == ctx_lens.numel() + 1
    assert q.is_contiguous() and out.is_contiguous() and block_tables.is_contiguous()
    return shape


def pa_prefill(q, k_cache, v_cache, block_tables, ctx_lens, cu_q_lens, scale, out, workspace, *,
               dev_status=None, stream=None):
    """Forward to pa_prefill.  q/out [total_q,H,D] bf16 (packed tokens); ctx_lens int32 [B];
    cu_q_lens int32 [B+1]; caches and block_tables as for pa_decode."""
    shape = _prefill_args(q, k_cache, v_cache, block_tables, ctx_lens, cu_q_lens, out)
    rc = lib().pa_prefill(ctypes.byref(shape), _ptr(q), _ptr(k_cache), _ptr(v_cache),
                          _ptr(block_tables), block_tables.shape[1], _ptr(ctx_lens),
                          _ptr(cu_q_lens), ctx_lens.numel(), q.shape[0], float(scale), _ptr(out),
                          _ptr(workspace), workspace.numel() * workspace.element_size(),
                          _ptr(dev_status), _stream(stream))
    _check(rc, "pa_prefill")
    return out


def pa_prefill_split(q, k_cache, v_cache, block_tables, ctx_lens, cu_q_lens, scale, out,
                     workspace, *, kv_split_tokens=0, dev_status=None, stream=None):
    """Forward to pa_prefill_split: pa_prefill with the KV range split over CTAs
    (kv_split_tokens: 0 = chosen by the library, > 0 = forced, < 0 = never)."""
    shape = _prefill_args(q, k_cache, v_cache, block_tables, ctx_lens, cu_q_lens, out)
    rc = lib().pa_prefill_split(ctypes.byref(shape), _ptr(q), _ptr(k_cache), _ptr(v_cache),
                                _ptr(block_tables), block_tables.shape[1], _ptr(ctx_lens),
                                _ptr(cu_q_lens), ctx_lens.numel(), q.shape[0], float(scale),
                                _ptr(out), _ptr(workspace),
                                workspace.numel() * workspace.element_size(),
                                int(kv_split_tokens), _ptr(dev_status), _stream(stream))
    _check(rc, "pa_prefill_split")
    return out


def pa_selftest_wait_expiry(limit_us: int, dev_status, stream=None):
    """Forward to pa_selftest_wait_expiry: a bounded wait that must run out and report it."""
    _check(lib().pa_selftest_wait_expiry(int(limit_us), _ptr(dev_status), _stream(stream)),
           "pa_selftest_wait_expiry")


def pa_probe_tma_issue(buf, warps: int, boxes: int, reps: int, dev_status, stream=None) -> int:
    """Forward to pa_probe_tma_issue; returns the number of 2 KB boxes the launch issues."""
    n = ctypes.c_int64(0)
    _check(lib().pa_probe_tma_issue(_ptr(buf), buf.numel() * buf.element_size(), warps, boxes, reps,
                                    ctypes.byref(n), _ptr(dev_status), _stream(stream)),
           "pa_probe_tma_issue")
    return int(n.value)


def pa_probe_read(buf, scattered: bool, dev_status, seed: int = 1, stream=None):
    """Forward to pa_probe_read: read every 4 KiB granule of `buf` once, in order or scattered."""
    _check(lib().pa_probe_read(_ptr(buf), buf.numel() * buf.element_size(), 1 if scattered else 0,
                               seed, None, _ptr(dev_status), _stream(stream)), "pa_probe_read")
