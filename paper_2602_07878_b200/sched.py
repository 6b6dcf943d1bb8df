"""ctypes binding of the host-side scheduler / block manager (include/pagedkv_sched.h).

Argument marshalling only: the queues, the free-block list and the preemption policy live in
the C++ library.  `Scheduler.step()` returns numpy views that can be handed to the GPU entry
points (pa_decode, kv_append, pa_prefill, kv_swap_out, kv_swap_in).
"""
from __future__ import annotations

import ctypes
from dataclasses import dataclass

import numpy as np

from . import api

SWAP, RECOMPUTE = 0, 1
VICTIM_LIFO, VICTIM_LARGEST = 0, 1


class SchedConfig(ctypes.Structure):
    _fields_ = [(n, ctypes.c_int32) for n in
                ("num_blocks", "block_size", "max_num_seqs", "max_batched_tokens", "preempt_mode",
                 "max_blocks_per_seq", "host_blocks")]


class SchedStats(ctypes.Structure):
    _fields_ = [(n, ctypes.c_int64) for n in
                ("steps", "preemptions", "swapped_out_blocks", "swapped_in_blocks",
                 "recomputed_tokens", "finished", "hol_blocked_steps", "decode_tokens",
                 "prefill_tokens")] + \
               [(n, ctypes.c_int32) for n in ("free_blocks", "running", "waiting", "reserved")]


class SchedPolicy(ctypes.Structure):
    _fields_ = [(n, ctypes.c_int32) for n in
                ("victim_policy", "demote_victims", "admit_lookahead", "max_output_tokens",
                 "max_seq_blocks")]


class SchedRequestStats(ctypes.Structure):
    _fields_ = [(n, ctypes.c_int64) for n in ("queued_step", "first_token_step", "finished_step")] + \
               [(n, ctypes.c_int32) for n in ("preemptions", "generated")]


_p64, _p32 = ctypes.POINTER(ctypes.c_int64), ctypes.POINTER(ctypes.c_int32)


class SchedStepOut(ctypes.Structure):
    _fields_ = [("n_decode", ctypes.c_int32), ("decode_ids", _p64), ("decode_lens", _p32),
                ("decode_slots", _p64), ("decode_tables", _p32),
                ("n_prefill", ctypes.c_int32), ("prefill_tokens", ctypes.c_int32),
                ("prefill_ids", _p64), ("prefill_q_lens", _p32), ("prefill_ctx_lens", _p32),
                ("prefill_tables", _p32), ("prefill_slots", _p64),
                ("n_swap_out", ctypes.c_int32), ("swap_out_blocks", _p32),
                ("swap_out_host_slots", _p32),
                ("n_swap_in", ctypes.c_int32), ("swap_in_host_slots", _p32),
                ("swap_in_blocks", _p32),
                ("n_finished", ctypes.c_int32), ("finished_ids", _p64)]


@dataclass
class Step:
    decode_ids: np.ndarray
    decode_lens: np.ndarray
    decode_slots: np.ndarray
    decode_tables: np.ndarray
    prefill_ids: np.ndarray
    prefill_q_lens: np.ndarray
    prefill_ctx_lens: np.ndarray
    prefill_tables: np.ndarray
    prefill_slots: np.ndarray
    swap_out_blocks: np.ndarray
    swap_out_host_slots: np.ndarray
    swap_in_host_slots: np.ndarray
    swap_in_blocks: np.ndarray
    finished_ids: np.ndarray
    idle: bool


def _arr(ptr, n, dtype, shape=None):
    if n == 0:
        a = np.zeros(0, dtype=dtype)
    else:
        a = np.ctypeslib.as_array(ptr, shape=(n,)).astype(dtype, copy=True)
    return a if shape is None else a.reshape(shape)


class Scheduler:
    def __init__(self, num_blocks, block_size=16, max_num_seqs=256, max_batched_tokens=512,
                 preempt_mode=SWAP, max_blocks_per_seq=2048, host_blocks=0):
        L = api.lib()
        L.sched_create.argtypes = [ctypes.POINTER(SchedConfig)]
        L.sched_create.restype = ctypes.c_void_p
        L.sched_destroy.argtypes = [ctypes.c_void_p]
        L.sched_destroy.restype = None
        L.sched_add_request.argtypes = [ctypes.c_void_p, ctypes.c_int64, ctypes.c_int32, ctypes.c_int32]
        L.sched_add_request.restype = ctypes.c_int
        L.sched_step.argtypes = [ctypes.c_void_p, ctypes.POINTER(SchedStepOut)]
        L.sched_step.restype = ctypes.c_int
        L.sched_get_stats.argtypes = [ctypes.c_void_p, ctypes.POINTER(SchedStats)]
        L.sched_get_stats.restype = None
        L.sched_set_policy.argtypes = [ctypes.c_void_p, ctypes.POINTER(SchedPolicy)]
        L.sched_set_policy.restype = ctypes.c_int
        L.sched_get_request_stats.argtypes = [ctypes.c_void_p, ctypes.c_int64,
                                              ctypes.POINTER(SchedRequestStats)]
        L.sched_get_request_stats.restype = ctypes.c_int
        self._L = L
        self.cfg = SchedConfig(num_blocks, block_size, max_num_seqs, max_batched_tokens,
                               preempt_mode, max_blocks_per_seq, host_blocks)
        self._h = L.sched_create(ctypes.byref(self.cfg))
        if not self._h:
            raise ValueError("invalid scheduler configuration")

    def close(self):
        if self._h:
            self._L.sched_destroy(self._h)
            self._h = None

    __del__ = close

    def add_request(self, req_id: int, prompt_len: int, max_new_tokens: int) -> bool:
        return self._L.sched_add_request(self._h, req_id, prompt_len, max_new_tokens) == 0

    def set_policy(self, victim_policy=VICTIM_LIFO, demote_victims=False, admit_lookahead=0,
                   max_output_tokens=0, max_seq_blocks=0) -> None:
        pol = SchedPolicy(victim_policy, int(demote_victims), admit_lookahead, max_output_tokens,
                          max_seq_blocks)
        if self._L.sched_set_policy(self._h, ctypes.byref(pol)) != 0:
            raise ValueError("invalid scheduler policy")

    def request_stats(self, req_id: int) -> SchedRequestStats:
        r = SchedRequestStats()
        if self._L.sched_get_request_stats(self._h, req_id, ctypes.byref(r)) != 0:
            raise KeyError(req_id)
        return r

    def stats(self) -> SchedStats:
        s = SchedStats()
        self._L.sched_get_stats(self._h, ctypes.byref(s))
        return s

    def step(self) -> Step:
        o = SchedStepOut()
        idle = self._L.sched_step(self._h, ctypes.byref(o)) == 1
        mb = self.cfg.max_blocks_per_seq
        return Step(
            _arr(o.decode_ids, o.n_decode, np.int64), _arr(o.decode_lens, o.n_decode, np.int32),
            _arr(o.decode_slots, o.n_decode, np.int64),
            _arr(o.decode_tables, o.n_decode * mb, np.int32, (o.n_decode, mb)),
            _arr(o.prefill_ids, o.n_prefill, np.int64), _arr(o.prefill_q_lens, o.n_prefill, np.int32),
            _arr(o.prefill_ctx_lens, o.n_prefill, np.int32),
            _arr(o.prefill_tables, o.n_prefill * mb, np.int32, (o.n_prefill, mb)),
            _arr(o.prefill_slots, o.prefill_tokens, np.int64),
            _arr(o.swap_out_blocks, o.n_swap_out, np.int32),
            _arr(o.swap_out_host_slots, o.n_swap_out, np.int32),
            _arr(o.swap_in_host_slots, o.n_swap_in, np.int32),
            _arr(o.swap_in_blocks, o.n_swap_in, np.int32),
            _arr(o.finished_ids, o.n_finished, np.int64), idle)
