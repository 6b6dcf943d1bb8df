"""Host-side scheduler / block manager: the behaviours Section 5.1 of the paper describes,
checked on small hand-traceable scenarios, plus conservation invariants on a random run."""
import numpy as np
import pytest

from paper_2602_07878_b200 import build
from paper_2602_07878_b200.sched import RECOMPUTE, SWAP, Scheduler


@pytest.fixture(scope="module", autouse=True)
def _lib():
    build.build()


def run_until_idle(s, limit=100000):
    steps = []
    for _ in range(limit):
        st = s.step()
        if st.idle:
            return steps
        steps.append(st)
    raise AssertionError("scheduler did not drain")


def test_prefill_is_chunked_under_the_token_budget_then_decodes():
    s = Scheduler(num_blocks=64, max_batched_tokens=32, max_blocks_per_seq=16)
    assert s.add_request(7, prompt_len=70, max_new_tokens=3)
    steps = run_until_idle(s)
    q = [int(st.prefill_q_lens[0]) for st in steps if len(st.prefill_ids)]
    ctx = [int(st.prefill_ctx_lens[0]) for st in steps if len(st.prefill_ids)]
    assert q == [32, 32, 6] and ctx == [32, 64, 70]
    dec = [st for st in steps if len(st.decode_ids)]
    assert [int(st.decode_lens[0]) for st in dec] == [71, 72, 73]
    assert list(dec[-1].finished_ids) == [7]
    # slots follow the block table: token t lives in block table[t // 16], offset t % 16
    first = steps[0]
    tab = first.prefill_tables[0]
    assert [int(x) for x in first.prefill_slots] == [int(tab[t // 16]) * 16 + t % 16 for t in range(32)]
    assert int(dec[0].decode_slots[0]) == int(dec[0].decode_tables[0][70 // 16]) * 16 + 70 % 16
    st = s.stats()
    assert st.free_blocks == 64 and st.finished == 1 and st.prefill_tokens == 70 and st.decode_tokens == 3


def test_fcfs_head_of_line_blocking_on_memory():
    # 10 blocks.  A (6 blocks of prompt) runs; B needs 6 and does not fit; C needs 1 and would
    # fit, but stands behind B: nobody behind a blocked head is admitted.
    s = Scheduler(num_blocks=10, max_batched_tokens=512, max_blocks_per_seq=8)
    s.add_request(1, 96, 8)
    s.add_request(2, 96, 8)
    s.add_request(3, 10, 2)
    st = s.step()
    assert list(st.prefill_ids) == [1]
    assert s.stats().waiting == 2 and s.stats().hol_blocked_steps == 1
    for _ in range(3):
        st = s.step()
        assert 3 not in list(st.prefill_ids) and 3 not in list(st.decode_ids)
    first_seen = {}
    for n, st in enumerate(run_until_idle(s)):
        for i in st.prefill_ids:
            first_seen.setdefault(int(i), n)
    assert first_seen[2] <= first_seen[3]         # 3 is admitted no earlier than the head, 2
    assert s.stats().finished == 3


def test_lifo_preemption_swaps_the_newest_and_requeues_it_first():
    # pool of 6 blocks, three 2-block prompts fill it; at 32 tokens every sequence needs a
    # third block: the newest (3) is evicted first, then 2; they return in that order
    s = Scheduler(num_blocks=6, max_batched_tokens=512, max_blocks_per_seq=8, host_blocks=16,
                  preempt_mode=SWAP)
    for i in (1, 2, 3):
        s.add_request(i, 31, 40)
    s.step()                                       # prefill of all three
    st = s.step()                                  # len 31 -> 32: still inside block 2
    assert len(st.decode_ids) == 3 and len(st.swap_out_blocks) == 0
    st = s.step()                                  # everyone needs a 3rd block, none is free
    # evicting the newest (3) frees two blocks: exactly what 1 and 2 need
    assert s.stats().preemptions == 1
    assert list(st.decode_ids) == [1, 2]
    assert len(st.swap_out_blocks) == 2 and len(set(st.swap_out_host_slots)) == 2
    assert s.stats().waiting == 1 and s.stats().hol_blocked_steps >= 1   # 3 cannot come back yet
    # at 48 tokens both need a 4th block: now 2 is the newest and goes, in FRONT of 3
    back = []
    for st in run_until_idle(s):
        if len(st.swap_in_blocks):
            back.append([int(i) for i in st.decode_ids])
    assert s.stats().preemptions >= 2
    assert back and back[0][-1] == 2              # the later victim returns first
    stt = s.stats()
    assert stt.swapped_in_blocks == stt.swapped_out_blocks and stt.finished == 3
    assert stt.free_blocks == 6


def test_recompute_mode_drops_kv_and_prefills_prompt_plus_generated():
    s = Scheduler(num_blocks=4, max_batched_tokens=512, max_blocks_per_seq=8,
                  preempt_mode=RECOMPUTE)
    s.add_request(1, 31, 30)
    s.add_request(2, 31, 30)
    s.step()
    s.step()                                       # both at 32 tokens
    st = s.step()                                  # 2 is evicted, nothing is swapped
    assert s.stats().preemptions == 1 and len(st.swap_out_blocks) == 0
    assert s.stats().recomputed_tokens == 32
    seen = None
    for st in run_until_idle(s):
        if 2 in list(st.prefill_ids):
            seen = (int(st.prefill_q_lens[0]), int(st.prefill_ctx_lens[0]))
            break
    assert seen == (32, 32)                        # prompt 31 + 1 generated token again


def test_random_traffic_conserves_blocks_and_never_shares_one():
    rng = np.random.default_rng(0)
    for mode in (SWAP, RECOMPUTE):
        s = Scheduler(num_blocks=200, max_num_seqs=32, max_batched_tokens=256,
                      max_blocks_per_seq=64, host_blocks=400, preempt_mode=mode)
        for i in range(120):
            assert s.add_request(i, int(rng.integers(1, 400)), int(rng.integers(1, 300)))
        assert not s.add_request(999, 900, 200)    # can never fit 64 blocks per sequence
        owner = {}
        total_decode = 0
        for st in run_until_idle(s):
            used = set()
            for row, L in zip(st.decode_tables, st.decode_lens):
                blk = [int(b) for b in row[: (int(L) + 15) // 16]]
                assert all(0 <= b < 200 for b in blk) and not (used & set(blk))
                used |= set(blk)
            for row, L in zip(st.prefill_tables, st.prefill_ctx_lens):
                blk = [int(b) for b in row[: (int(L) + 15) // 16]]
                assert all(0 <= b < 200 for b in blk) and not (used & set(blk))
                used |= set(blk)
            assert int(st.prefill_q_lens.sum()) + len(st.decode_ids) <= 256
            total_decode += len(st.decode_ids)
        stt = s.stats()
        assert stt.finished == 120 and stt.free_blocks == 200 and stt.running == 0
        assert stt.preemptions > 0 and stt.decode_tokens == total_decode
        assert stt.swapped_in_blocks == stt.swapped_out_blocks
        assert (stt.swapped_out_blocks > 0) == (mode == SWAP)
