"""End to end: the host scheduler drives kv_append, pa_prefill, pa_decode and the swaps through
a pool that is too small for its traffic, so sequences are preempted, swapped out and in (or
recomputed) while others decode.  Every attention output of every iteration is compared with
the fp64 oracle working from dense per-sequence copies that never touch the GPU."""
import numpy as np
import pytest
import torch

import oracle
from paper_2602_07878_b200 import api
from paper_2602_07878_b200 import workloads as wl
from paper_2602_07878_b200.sched import RECOMPUTE, SWAP, Scheduler
from helpers import assert_parity, bits_to_torch, prefill_ref, torch_to_f64

pytestmark = pytest.mark.gpu

H, HKV, D, NB = 8, 2, 128, 24


def tok_bits(kind, seq_id, t):
    """bf16 bits of token t of sequence seq_id: 'k'/'v' rows [HKV, D] or a 'q' row [H, D]."""
    n = (H if kind == "q" else HKV) * D
    seed = {"q": 0x71, "k": 0x72, "v": 0x73}[kind]
    return wl.normal_bf16_np((seq_id * 8192 + t) * n, n, seed).reshape(-1, D)


def dense_inputs(ids, lens):
    """Compact pool + tables holding tokens 0..len-1 of every listed sequence."""
    nblk = [(int(L) + 15) // 16 for L in lens]
    k = np.full((sum(nblk), HKV, 16, D), wl.BF16_NAN_BITS, np.uint16)
    v = k.copy()
    tables = np.zeros((len(ids), max(nblk)), np.int32)
    o = 0
    for i, (sid, L) in enumerate(zip(ids, lens)):
        for t in range(int(L)):
            k[o + t // 16, :, t % 16] = tok_bits("k", int(sid), t)
            v[o + t // 16, :, t % 16] = tok_bits("v", int(sid), t)
        tables[i, :nblk[i]] = np.arange(o, o + nblk[i])
        o += nblk[i]
    return k, v, tables


def runs(host_slots):
    """Split indices into runs of consecutive host slots (one victim = one contiguous run)."""
    out, start = [], 0
    for i in range(1, len(host_slots) + 1):
        if i == len(host_slots) or host_slots[i] != host_slots[i - 1] + 1:
            out.append((start, i))
            start = i
    return out


FAIR = dict(victim_policy=1, demote_victims=True, admit_lookahead=3)


@pytest.mark.parametrize("mode,policy", [(SWAP, {}), (RECOMPUTE, {}), (SWAP, FAIR), (RECOMPUTE, FAIR),
                                         (SWAP, dict(max_output_tokens=20, max_seq_blocks=6))])
def test_scheduler_driven_engine_loop_matches_oracle(mode, policy):
    rng = np.random.default_rng(5)
    sched = Scheduler(num_blocks=NB, max_num_seqs=8, max_batched_tokens=96, preempt_mode=mode,
                      max_blocks_per_seq=16, host_blocks=64)
    sched.set_policy(**policy)
    for i in range(10):
        assert sched.add_request(i, int(rng.integers(5, 120)), int(rng.integers(8, 70)))
    dev = "cuda"
    k_pool = torch.full((1, NB, HKV, 16, D), float("nan"), dtype=torch.bfloat16, device=dev)
    v_pool = k_pool.clone()
    kc, vc = k_pool[0], v_pool[0]
    bb = api.kv_block_bytes(k_pool, v_pool)
    host = torch.zeros(64 * bb, dtype=torch.uint8, pin_memory=True)
    shape = api.shape_of(kc, H)
    ws = torch.empty(api.pa_workspace_bytes(shape, 8, 8 * 16 * 16), dtype=torch.uint8, device=dev)
    pws = torch.empty(api.pa_prefill_workspace_bytes(8), dtype=torch.uint8, device=dev)
    status = torch.zeros(1, dtype=torch.int32, device=dev)
    scale = np.float32(1.0 / np.sqrt(D))
    pos_of = {}          # sequence id -> tokens in the cache (as the test tracks them)
    checked_decode = checked_prefill = 0
    for _ in range(5000):
        st = sched.step()
        if st.idle:
            break
        # ---- swaps decided by the scheduler ----
        for a, b in runs(list(st.swap_out_host_slots)):
            api.kv_swap_out(k_pool, v_pool, st.swap_out_blocks[a:b],
                            host[int(st.swap_out_host_slots[a]) * bb:])
        if len(st.swap_out_blocks):
            torch.cuda.synchronize()
            idx = torch.from_numpy(st.swap_out_blocks.astype(np.int64)).to(dev)
            kc[idx] = float("nan")                 # the freed blocks may be reused by anyone
            vc[idx] = float("nan")
        for a, b in runs(list(st.swap_in_host_slots)):
            api.kv_swap_in(k_pool, v_pool, host[int(st.swap_in_host_slots[a]) * bb:],
                           st.swap_in_blocks[a:b])
        # ---- prefill chunks ----
        if len(st.prefill_ids):
            cu = np.concatenate([[0], np.cumsum(st.prefill_q_lens)]).astype(np.int32)
            q_rows, k_rows, v_rows = [], [], []
            for sid, ql, ctx in zip(st.prefill_ids, st.prefill_q_lens, st.prefill_ctx_lens):
                for t in range(int(ctx - ql), int(ctx)):
                    q_rows.append(tok_bits("q", int(sid), t))
                    k_rows.append(tok_bits("k", int(sid), t))
                    v_rows.append(tok_bits("v", int(sid), t))
                pos_of[int(sid)] = int(ctx)
            qb = np.stack(q_rows)
            api.kv_append(kc, vc, bits_to_torch(np.stack(k_rows)), bits_to_torch(np.stack(v_rows)),
                          torch.from_numpy(st.prefill_slots).to(dev), dev_status=status)
            q = bits_to_torch(qb)
            out = torch.full_like(q, float("nan"))
            api.pa_prefill(q, kc, vc, torch.from_numpy(st.prefill_tables).to(dev),
                           torch.from_numpy(st.prefill_ctx_lens).to(dev), torch.from_numpy(cu).to(dev),
                           scale, out, pws, dev_status=status)
            torch.cuda.synchronize()
            dk, dv, dt = dense_inputs(st.prefill_ids, st.prefill_ctx_lens)
            ref, abs_ref = prefill_ref(qb, dk, dv, dt, st.prefill_ctx_lens, cu, scale)
            assert_parity(torch_to_f64(out), ref, "prefill", amended=abs_ref)
            checked_prefill += 1
        # ---- decode: append the new token, attend ----
        if len(st.decode_ids):
            new_pos = st.decode_lens - 1
            for sid, t in zip(st.decode_ids, new_pos):
                assert pos_of[int(sid)] == int(t)   # swaps / recompute restored the whole context
                pos_of[int(sid)] = int(t) + 1
            kn = np.stack([tok_bits("k", int(s), int(t)) for s, t in zip(st.decode_ids, new_pos)])
            vn = np.stack([tok_bits("v", int(s), int(t)) for s, t in zip(st.decode_ids, new_pos)])
            qb = np.stack([tok_bits("q", int(s), int(t)) for s, t in zip(st.decode_ids, new_pos)])
            api.kv_append(kc, vc, bits_to_torch(kn), bits_to_torch(vn),
                          torch.from_numpy(st.decode_slots).to(dev), dev_status=status)
            q = bits_to_torch(qb)
            out = torch.full_like(q, float("nan"))
            api.pa_decode(q, kc, vc, torch.from_numpy(st.decode_tables).to(dev),
                          torch.from_numpy(st.decode_lens).to(dev), scale, out, ws,
                          partition_tokens=64, dev_status=status)
            torch.cuda.synchronize()
            dk, dv, dt = dense_inputs(st.decode_ids, st.decode_lens)
            ref = oracle.pa_decode(qb, dk, dv, dt, st.decode_lens, scale)
            assert_parity(torch_to_f64(out), ref, "decode")
            checked_decode += 1
    stats = sched.stats()
    assert int(status.item()) == 0
    assert stats.finished == 10 and stats.free_blocks == NB
    if not policy.get("max_output_tokens"):          # under quotas the pool may never run dry
        assert stats.preemptions > 0
        assert (stats.swapped_out_blocks > 0) == (mode == SWAP)
        assert checked_decode > 50
    assert checked_decode > 15 and checked_prefill > 5
