"""pa_decode_static: decode attention for callers that cannot allocate device memory.

A serving engine that gave the whole GPU to its KV pool, or a plug-in that only ever sees
the current step's tensors, has no way to cudaMalloc the workspace pa_decode asks for.
pa_decode_static keeps its scratch in a fixed array inside the library instead.  This file
checks, through the C-ABI, that it gives the same result as pa_decode with a caller-owned
workspace and as the fp64 oracle -- several times in a row with different shapes, because every
call reuses the same array and finds the previous call's leftovers in it -- that the device's
free memory does not move across a call, and that a request beyond the array's size is refused
before anything is launched.  It is collected last on purpose.
"""
import ctypes

import numpy as np
import pytest
import torch

from paper_2602_07878_b200 import api
from paper_2602_07878_b200 import workloads as wl
from helpers import GpuDecode, assert_parity, oracle_for, torch_to_f64

pytestmark = pytest.mark.gpu


def _both_ways(spec):
    q = wl.q_np(spec)
    k, v = wl.pools_np(spec)
    g = GpuDecode(spec, q, k, v)
    ref = g.run().clone()                      # existing entry point, caller workspace
    out = torch.full_like(g.q, float("nan"))
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    run = lambda: api.pa_decode_static(g.q, g.k, g.v, g.tables, g.lens, spec.scale, out,
                                       spec.total_tokens, dev_status=status)
    run()                                      # the first call on a device looks the array up
    torch.cuda.synchronize()
    out.fill_(float("nan"))
    allocations = lambda: torch.cuda.memory_stats().get("allocation.all.allocated", 0)
    before = allocations()                     # count of requests to torch's allocator so far
    free_before = torch.cuda.mem_get_info()[0]  # the driver's own count of free bytes
    run()
    torch.cuda.synchronize()
    assert allocations() == before             # torch's allocator was not asked for anything
    assert torch.cuda.mem_get_info()[0] == free_before   # nor the driver, by the library itself
    assert int(status.item()) == 0
    # the definition itself, under the plain decode tolerance
    assert_parity(torch_to_f64(out), oracle_for(spec, q, k, v), f"{spec.name} against the oracle")
    return torch_to_f64(out), torch_to_f64(ref)


def test_static_scratch_matches_caller_workspace_on_two_calls_in_a_row():
    # call 1: mixed long/short GQA batch that is split into many partitions
    got, ref = _both_ways(wl.config_spec(3, scale_down=8))
    assert_parity(got, ref, "first call")
    # call 2: different geometry, finds call 1's plan and partials in the array
    spec = wl.make_spec("t", seq_lens=[0, 5, 700, 16, 1300], num_q_heads=8, num_kv_heads=8,
                        head_dim=64, occupancy=0.9, seed=77)
    got, ref = _both_ways(spec)
    assert_parity(got, ref, "second call")
    assert (got[0] == 0).all()
    # and once more with the first shape
    got, ref = _both_ways(wl.config_spec(1))
    assert_parity(got, ref, "third call")


def test_request_beyond_the_static_array_is_refused():
    spec = wl.config_spec(1)
    q = wl.q_np(spec)
    k, v = wl.pools_np(spec)
    g = GpuDecode(spec, q, k, v)
    shape = api.shape_of(g.k, 8)
    too_many = 1 << 34                          # tokens whose partials cannot fit in 64 MiB
    assert api.pa_workspace_bytes(shape, 4, too_many) > api.PA_STATIC_WORKSPACE_BYTES
    n0 = api.pa_launch_count()
    with pytest.raises(api.PagedKVError) as e:
        api.pa_decode_static(g.q, g.k, g.v, g.tables, g.lens, spec.scale, g.out, too_many)
    assert e.value.code == api.ERR["STATIC_LIMIT"]
    assert "static workspace" in str(e.value)
    assert api.pa_launch_count() == n0
