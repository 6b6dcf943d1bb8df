"""ctypes front end of the fp64 CPU oracle (`pa_oracle.cpp`).  TEST INFRASTRUCTURE ONLY.

Only the tests, the smoke check and the benchmark's CPU-baseline leg may import this
package.  It takes and returns numpy arrays; bf16 tensors travel as uint16 bit patterns.
It imports nothing from the CUDA package.
"""
from __future__ import annotations

import ctypes
import os
import subprocess

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "pa_oracle.cpp")
_LIB = os.path.join(_HERE, "liboracle.so")
_lib = None


def build(force: bool = False) -> str:
    """Compile pa_oracle.cpp into liboracle.so next to it (g++, OpenMP, no fast-math)."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        cmd = ["g++", "-O2", "-std=c++17", "-fopenmp", "-shared", "-fPIC", _SRC, "-o", _LIB]
        subprocess.run(cmd, check=True)
    return _LIB


def _load():
    global _lib
    if _lib is None:
        lib = ctypes.CDLL(build())
        i32, i64, dbl, vp = ctypes.c_int32, ctypes.c_int64, ctypes.c_double, ctypes.c_void_p
        lib.oracle_threads.argtypes = [ctypes.c_int]
        lib.oracle_threads.restype = ctypes.c_int
        lib.oracle_pa_decode.argtypes = [vp, vp, vp, vp, i32, vp, i32, i32, i32, i32, i32, i32,
                                         i64, i64, i64, dbl, vp, i32]
        lib.oracle_pa_decode.restype = ctypes.c_int
        swap = [vp, vp, i32, i64, i64, i32, i32, i32, i32, i64, i64, i64, vp, i32, vp]
        lib.oracle_swap_out.argtypes = swap
        lib.oracle_swap_out.restype = ctypes.c_int
        lib.oracle_swap_in.argtypes = swap
        lib.oracle_swap_in.restype = ctypes.c_int
        lib.oracle_pa_prefill.argtypes = [vp, vp, vp, vp, i32, vp, vp, i32, i32, i32, i32, i32, i32,
                                          i64, i64, i64, dbl, vp, i32]
        lib.oracle_pa_prefill.restype = ctypes.c_int
        lib.oracle_kv_append.argtypes = [vp, vp, vp, vp, vp, i32, i32, i32, i32, i32, i64, i64, i64]
        lib.oracle_kv_append.restype = ctypes.c_int
        _lib = lib
    return _lib


def _ptr(a: np.ndarray):
    return a.ctypes.data_as(ctypes.c_void_p)


def threads(requested: int = 0) -> int:
    return int(_load().oracle_threads(requested))


def _elem_strides(a: np.ndarray):
    assert a.dtype == np.uint16 and a.ndim == 4 and a.strides[3] == 2
    return tuple(s // 2 for s in a.strides[:3])


def _sigma(scale) -> float:
    """The scale is an fp32 argument of the method: whatever the caller passes is rounded to
    fp32 first and that value, widened exactly, is what the fp64 arithmetic uses."""
    return float(np.float32(scale))


def pa_decode(q, k_cache, v_cache, block_tables, seq_lens, scale, num_threads: int = 0):
    """fp64 attention output [B, H, D] for bf16-bit inputs.

    q uint16[B,H,D]; k_cache / v_cache uint16[NB,Hkv,bs,D] (any strides over the first
    three axes, identical for both); block_tables int32[B,max_blocks]; seq_lens int32[B].
    """
    q = np.ascontiguousarray(q, dtype=np.uint16)
    block_tables = np.ascontiguousarray(block_tables, dtype=np.int32)
    seq_lens = np.ascontiguousarray(seq_lens, dtype=np.int32)
    B, H, D = q.shape
    NB, Hkv, bs, D2 = k_cache.shape
    assert D2 == D and v_cache.shape == k_cache.shape
    sb, sh, st = _elem_strides(k_cache)
    assert _elem_strides(v_cache) == (sb, sh, st)
    if block_tables.ndim != 2 or block_tables.shape[0] != B:
        raise ValueError("block_tables must be [B, max_blocks]")
    out = np.zeros((B, H, D), dtype=np.float64)
    rc = _load().oracle_pa_decode(_ptr(q), _ptr(k_cache), _ptr(v_cache), _ptr(block_tables),
                                  block_tables.shape[1], _ptr(seq_lens), B, H, Hkv, D, bs, NB,
                                  sb, sh, st, _sigma(scale), _ptr(out), num_threads)
    if rc != 0:
        raise ValueError("oracle_pa_decode: invalid length or block id")
    return out


def _pool_args(k_pool, v_pool):
    # pools: uint16[layers, NB, Hkv, bs, D]
    assert k_pool.dtype == np.uint16 and k_pool.ndim == 5 and k_pool.shape == v_pool.shape
    assert k_pool.strides[4] == 2 and v_pool.strides == k_pool.strides
    Lyr, NB, Hkv, bs, D = k_pool.shape
    ls, sb, sh, st = (s // 2 for s in k_pool.strides[:4])
    return Lyr, NB, Hkv, bs, D, ls, sb, sh, st


def swap_out(k_pool, v_pool, block_ids):
    """Host image uint16[n, layers, 2, Hkv, bs, D] of the listed blocks."""
    Lyr, NB, Hkv, bs, D, ls, sb, sh, st = _pool_args(k_pool, v_pool)
    ids = np.ascontiguousarray(block_ids, dtype=np.int32)
    host = np.zeros((len(ids), Lyr, 2, Hkv, bs, D), dtype=np.uint16)
    rc = _load().oracle_swap_out(_ptr(k_pool), _ptr(v_pool), Lyr, ls, ls, Hkv, D, bs, NB,
                                 sb, sh, st, _ptr(ids), len(ids), _ptr(host))
    if rc != 0:
        raise ValueError("oracle_swap_out: block id out of range")
    return host


def swap_in(k_pool, v_pool, host, block_ids):
    """Write host slot i into block block_ids[i] of the pools (in place)."""
    Lyr, NB, Hkv, bs, D, ls, sb, sh, st = _pool_args(k_pool, v_pool)
    ids = np.ascontiguousarray(block_ids, dtype=np.int32)
    host = np.ascontiguousarray(host, dtype=np.uint16)
    assert host.size == len(ids) * Lyr * 2 * Hkv * bs * D
    rc = _load().oracle_swap_in(_ptr(k_pool), _ptr(v_pool), Lyr, ls, ls, Hkv, D, bs, NB,
                                sb, sh, st, _ptr(ids), len(ids), _ptr(host))
    if rc != 0:
        raise ValueError("oracle_swap_in: block id out of range")


def kv_append(k_cache, v_cache, k_new, v_new, slot_mapping):
    """Write token b's K/V rows (uint16[B,Hkv,D]) into flat slot slot_mapping[b] of one
    layer's caches (uint16[NB,Hkv,bs,D], modified in place); negative slots are skipped."""
    NB, Hkv, bs, D = k_cache.shape
    sb, sh, st = _elem_strides(k_cache)
    assert _elem_strides(v_cache) == (sb, sh, st)
    k_new = np.ascontiguousarray(k_new, dtype=np.uint16)
    v_new = np.ascontiguousarray(v_new, dtype=np.uint16)
    slots = np.ascontiguousarray(slot_mapping, dtype=np.int64)
    assert k_new.shape == (len(slots), Hkv, D) and v_new.shape == k_new.shape
    rc = _load().oracle_kv_append(_ptr(k_cache), _ptr(v_cache), _ptr(k_new), _ptr(v_new),
                                  _ptr(slots), len(slots), Hkv, D, bs, NB, sb, sh, st)
    if rc != 0:
        raise ValueError("oracle_kv_append: slot beyond the pool")


def pa_prefill(q, k_cache, v_cache, block_tables, ctx_lens, cu_q_lens, scale, num_threads: int = 0):
    """fp64 causal attention [total_q, H, D] of packed query tokens over the paged cache.

    q uint16[total_q,H,D]; sequence b owns rows cu_q_lens[b]..cu_q_lens[b+1]-1, which are the
    last tokens of its ctx_lens[b] cached tokens."""
    q = np.ascontiguousarray(q, dtype=np.uint16)
    block_tables = np.ascontiguousarray(block_tables, dtype=np.int32)
    ctx_lens = np.ascontiguousarray(ctx_lens, dtype=np.int32)
    cu = np.ascontiguousarray(cu_q_lens, dtype=np.int32)
    T, H, D = q.shape
    NB, Hkv, bs, _ = k_cache.shape
    B = len(ctx_lens)
    assert len(cu) == B + 1 and (B == 0 or cu[-1] == T)
    sb, sh, st = _elem_strides(k_cache)
    assert _elem_strides(v_cache) == (sb, sh, st)
    out = np.zeros((T, H, D), dtype=np.float64)
    rc = _load().oracle_pa_prefill(_ptr(q), _ptr(k_cache), _ptr(v_cache), _ptr(block_tables),
                                   block_tables.shape[1], _ptr(ctx_lens), _ptr(cu), B, H, Hkv, D,
                                   bs, NB, sb, sh, st, _sigma(scale), _ptr(out), num_threads)
    if rc != 0:
        raise ValueError("oracle_pa_prefill: inconsistent lengths or bad block id")
    return out
