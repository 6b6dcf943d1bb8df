"""Host-only checks of the C-ABI: the library loads without a GPU, exports every symbol
the header declares, and refuses bad arguments before touching the device."""
import ctypes
import os
import re

import pytest

from paper_2602_07878_b200 import api, build

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def L():
    build.build()
    return api.lib()


def declared_functions():
    names = []
    for header in ("pagedkv.h", "pagedkv_sched.h"):
        text = open(os.path.join(ROOT, "include", header)).read()
        text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
        names += re.findall(r"^\s*(?:const\s+char\s*\*|void\s*\*|int64_t|int|void)\s+(\w+)\s*\(",
                            text, flags=re.M)
    return names


def test_header_symbols_are_exported(L):
    names = declared_functions()
    assert {"pa_decode", "kv_swap_out", "kv_swap_in", "pa_workspace_bytes", "pa_prefill",
            "kv_append", "sched_create", "sched_step", "sched_destroy"} <= set(names)
    for n in names:
        assert hasattr(L, n), f"{n} declared in pagedkv.h but not exported"
    assert set(api.EXPORTS) <= set(names)


def test_status_strings(L):
    assert L.pa_status_string(0) == b"ok"
    for code in api.ERR.values():
        s = L.pa_status_string(code)
        assert s and s != b"unknown status"
    assert L.pa_status_string(-99) == b"unknown status"


def good_shape():
    return api.PaShape(32, 8, 128, 16, 1000, api.PA_BF16, 8 * 16 * 128, 16 * 128, 128)


def test_workspace_bytes_grows_and_validates(L):
    s = good_shape()
    a = api.pa_workspace_bytes(s, 16, 10000)
    b = api.pa_workspace_bytes(s, 256, 400000)
    c = api.pa_workspace_bytes(s, 256, 400000, 64)
    assert 0 < a < b < c
    out = ctypes.c_size_t()
    assert L.pa_workspace_bytes(None, 1, 1, 0, ctypes.byref(out)) == api.ERR["NULL"]
    for p in (8, 24, 528, -16):
        assert L.pa_workspace_bytes(ctypes.byref(s), 1, 1, p, ctypes.byref(out)) == api.ERR["ARG"]


def test_workspace_bytes_holds_two_plan_regions_and_the_partial_records(L):
    # per work item: a 16-byte record in each of the two plan regions, H (max, sum) pairs and H
    # fp32 rows of D; per sequence: 8 + 4 bytes in each region; a few 256-byte roundings on top
    s = good_shape()
    H, D = s.num_q_heads, s.head_dim
    for batch, tokens, P in [(1, 16, 0), (256, 400000, 0), (256, 400000, 64), (3000, 90000, 512)]:
        items = tokens // (P or 256) + batch + 1
        need = items * (2 * 16 + H * 8 + H * D * 4) + 2 * batch * 12
        got = api.pa_workspace_bytes(s, batch, tokens, P)
        assert need <= got <= need + 16 * 256, (batch, tokens, P, need, got)


@pytest.mark.parametrize("field,value", [("head_dim", 96), ("block_size", 32), ("num_q_heads", 30),
                                         ("num_q_heads", 8 * 17), ("dtype", 0),
                                         ("stride_tok", 132), ("num_blocks", 0),
                                         ("stride_tok", 64)])
def test_bad_shapes_are_refused(L, field, value):
    s = good_shape()
    setattr(s, field, value)
    out = ctypes.c_size_t()
    assert L.pa_workspace_bytes(ctypes.byref(s), 1, 16, 0, ctypes.byref(out)) == api.ERR["SHAPE"]


def test_pa_decode_argument_errors_return_before_any_launch(L):
    s = good_shape()
    n0 = L.pa_launch_count()
    sp = ctypes.byref(s)
    A = ctypes.c_void_p(0x10000)          # aligned fake addresses: never dereferenced on host
    U = ctypes.c_void_p(0x10008)
    args = lambda **kw: [kw.get("shape", sp), kw.get("q", A), A, A, kw.get("tables", A), 8, A,
                         kw.get("batch", 4), 0.1, kw.get("out", A), kw.get("ws", A),
                         kw.get("ws_bytes", 1 << 24), kw.get("part", 0), kw.get("flags", 0),
                         None, None]
    assert L.pa_decode(*args(shape=None)) == api.ERR["NULL"]
    assert L.pa_decode(*args(q=None)) == api.ERR["NULL"]
    assert L.pa_decode(*args(tables=None)) == api.ERR["NULL"]
    assert L.pa_decode(*args(q=U)) == api.ERR["ALIGN"]
    assert L.pa_decode(*args(out=U)) == api.ERR["ALIGN"]
    assert L.pa_decode(*args(ws=ctypes.c_void_p(0x10010))) == api.ERR["ALIGN"]
    assert L.pa_decode(*args(ws_bytes=1024)) == api.ERR["WORKSPACE"]
    assert L.pa_decode(*args(batch=-1)) == api.ERR["ARG"]
    assert L.pa_decode(*args(part=20)) == api.ERR["ARG"]
    assert L.pa_decode(*args(flags=6)) == api.ERR["ARG"]
    assert L.pa_decode(*args(batch=0)) == api.PA_OK          # empty batch: nothing to do
    assert L.pa_launch_count() == n0


def test_swap_argument_errors_return_before_any_launch(L):
    s = good_shape()
    pool = api.KvPoolDesc(4, 0, 1000 * 8 * 16 * 128, 1000 * 8 * 16 * 128)
    bb = ctypes.c_size_t()
    assert L.kv_block_bytes(ctypes.byref(pool), ctypes.byref(s), ctypes.byref(bb)) == 0
    assert bb.value == 4 * 2 * 8 * 16 * 128 * 2
    A = ctypes.c_void_p(0x10000)
    ids = (ctypes.c_int32 * 3)(5, 7, 5)
    n0 = L.pa_launch_count()
    call = lambda ids_, n, hb, host=A: L.kv_swap_out(ctypes.byref(pool), ctypes.byref(s), A, A,
                                                     ids_, n, host, hb, None, 0, None)
    assert call(ids, 3, 3 * bb.value) == api.ERR["BLOCK_ID"]          # duplicate id
    ids2 = (ctypes.c_int32 * 2)(5, 1000)
    assert call(ids2, 2, 2 * bb.value) == api.ERR["BLOCK_ID"]         # out of range
    ids3 = (ctypes.c_int32 * 2)(5, 6)
    assert call(ids3, 2, 2 * bb.value - 1) == api.ERR["HOSTBUF"]
    assert call(ids3, -1, 0) == api.ERR["ARG"]
    assert call(ids3, 0, 0) == api.PA_OK
    assert call(ids3, 2, 2 * bb.value, ctypes.c_void_p(0x10004)) == api.ERR["ALIGN"]
    assert call(None, 2, 2 * bb.value) == api.ERR["NULL"]
    assert L.kv_swap_in(ctypes.byref(pool), ctypes.byref(s), A, A, A, 3 * bb.value, ids, 3,
                        None, 0, None) == api.ERR["BLOCK_ID"]
    assert L.pa_launch_count() == n0


def test_tma_issue_probe_refuses_bad_shapes_before_any_launch():
    import ctypes
    L = api.lib()
    n = ctypes.c_int64(0)
    buf, st = ctypes.c_void_p(1 << 20), ctypes.c_void_p(256)      # never dereferenced on the host
    call = lambda warps, boxes, reps=1, nbytes=1 << 20: L.pa_probe_tma_issue(
        buf, nbytes, warps, boxes, reps, ctypes.byref(n), st, None)
    assert call(0, 2) == api.ERR["ARG"] and call(9, 2) == api.ERR["ARG"]
    assert call(1, 3) == api.ERR["ARG"] and call(1, 18) == api.ERR["ARG"]
    assert call(8, 4) == api.ERR["ARG"]            # 32 boxes per slot round do not fit the rings
    assert call(1, 2, 0) == api.ERR["ARG"] and call(1, 2, 1, 1 << 10) == api.ERR["ARG"]
    assert L.pa_probe_tma_issue(None, 1 << 20, 1, 2, 1, None, st, None) == api.ERR["NULL"]
