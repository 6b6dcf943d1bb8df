"""Countermeasure switches of the host scheduler (Section 7 of the paper names output-length
quotas and fairness-aware scheduling without defining them; the readings are in the header).
Hand-traceable cases per switch, then a synthetic squeeze (a few long-running requests keep a
small pool full while short requests arrive) on which the switches are compared."""
import numpy as np
import pytest

from paper_2602_07878_b200 import build
from paper_2602_07878_b200.sched import SWAP, VICTIM_LARGEST, VICTIM_LIFO, Scheduler


@pytest.fixture(scope="module", autouse=True)
def _lib():
    build.build()


def drain(s, limit=200000):
    for _ in range(limit):
        if s.step().idle:
            return
    raise AssertionError("scheduler did not drain")


def test_default_policy_is_the_engine_of_section_5_1():
    # identical step-by-step output with no policy call and with an all-zero policy
    def trace(set_zero):
        s = Scheduler(num_blocks=12, max_batched_tokens=64, max_blocks_per_seq=12, host_blocks=32)
        if set_zero:
            s.set_policy()
        for i, (p, n) in enumerate([(40, 60), (30, 70), (20, 50), (10, 5)]):
            s.add_request(i, p, n)
        out = []
        for _ in range(2000):
            st = s.step()
            if st.idle:
                break
            out.append((tuple(st.decode_ids), tuple(st.prefill_ids), tuple(st.swap_out_blocks),
                        tuple(st.swap_in_blocks), tuple(st.finished_ids)))
        return out
    assert trace(False) == trace(True)


def test_lookahead_lets_a_short_request_pass_a_blocked_head():
    # the head-of-line case of Section 5.1.1: B (6 blocks) does not fit behind A; C (1 block) does
    s = Scheduler(num_blocks=10, max_batched_tokens=512, max_blocks_per_seq=8)
    s.set_policy(admit_lookahead=1)
    s.add_request(1, 96, 8)
    s.add_request(2, 96, 8)
    s.add_request(3, 10, 2)
    st = s.step()
    assert list(st.prefill_ids) == [1, 3]           # C admitted in the same iteration as A
    assert s.stats().hol_blocked_steps == 1         # the head was still found blocked
    drain(s)
    r2, r3 = s.request_stats(2), s.request_stats(3)
    assert r3.finished_step < r2.first_token_step   # C is done before B even starts


def test_output_quota_truncates_generation():
    s = Scheduler(num_blocks=64, max_batched_tokens=512, max_blocks_per_seq=32)
    s.set_policy(max_output_tokens=5)
    s.add_request(1, 20, 300)
    s.add_request(2, 20, 3)
    drain(s)
    assert s.request_stats(1).generated == 5 and s.request_stats(2).generated == 3
    assert s.stats().free_blocks == 64


def test_block_quota_cuts_a_sequence_off_at_its_cap():
    s = Scheduler(num_blocks=64, max_batched_tokens=512, max_blocks_per_seq=32)
    s.set_policy(max_seq_blocks=3)
    s.add_request(1, 20, 300)                        # 2 blocks of prompt, grows to 3 and stops
    drain(s)
    r = s.request_stats(1)
    assert r.generated == 3 * 16 - 20 and r.finished_step > 0
    assert s.stats().free_blocks == 64


def test_largest_victim_and_demotion():
    # 8 blocks: A holds 5 (prompt 70), B holds 2 (prompt 20), one block free.  A reaches token
    # 80 first and takes the last block; B reaches 32 and the pool is empty.  LIFO evicts B
    # (admitted last); the fairness choice evicts A, which holds the most.
    def run(victim, demote):
        s = Scheduler(num_blocks=8, max_batched_tokens=512, max_blocks_per_seq=8, host_blocks=16)
        s.set_policy(victim_policy=victim, demote_victims=demote)
        s.add_request(1, 70, 40)
        s.add_request(2, 20, 40)
        first = None
        for _ in range(500):
            st = s.step()
            if st.idle:
                break
            if first is None and len(st.swap_out_blocks):
                first = len(st.swap_out_blocks)
        return first, s.request_stats(1), s.request_stats(2)
    n_lifo, a, b = run(VICTIM_LIFO, False)
    assert n_lifo == 2 and b.preemptions >= 1 and a.preemptions == 0
    n_fair, a, b = run(VICTIM_LARGEST, True)
    assert n_fair == 6 and a.preemptions >= 1 and b.preemptions == 0
    assert b.finished_step < a.finished_step


def squeeze(policy, seed=5):
    """A pool of 96 blocks; four long-running requests (prompt 200, 900 new tokens) arrive
    first and between them outgrow the pool; 60 short requests (prompt 16..64, 8..32 new
    tokens) arrive three per iteration from step 20 on.  Returns the short requests' mean
    queueing delay to the first token, the total preemptions and the steps to drain."""
    rng = np.random.default_rng(seed)
    s = Scheduler(num_blocks=96, max_num_seqs=32, max_batched_tokens=256, preempt_mode=SWAP,
                  max_blocks_per_seq=96, host_blocks=512)
    s.set_policy(**policy)
    for i in range(4):
        assert s.add_request(i, 200, 900)
    shorts = [(100 + i, int(rng.integers(16, 65)), int(rng.integers(8, 33))) for i in range(60)]
    step = 0
    while True:
        if step >= 20:
            for rid, p, n in shorts[(step - 20) * 3:(step - 20) * 3 + 3]:
                assert s.add_request(rid, p, n)
        st = s.step()
        step += 1
        if st.idle and step > 45:
            break
        assert step < 200000
    ttft = [s.request_stats(rid).first_token_step - s.request_stats(rid).queued_step
            for rid, _, _ in shorts]
    done = all(s.request_stats(i).finished_step > 0 for i in list(range(4)) + [r for r, _, _ in shorts])
    assert done and s.stats().free_blocks == 96
    return float(np.mean(ttft)), int(s.stats().preemptions), int(s.stats().steps)


def test_fairness_switches_shorten_the_short_requests_wait_under_a_squeeze():
    base_ttft, base_pre, base_steps = squeeze({})
    fair_ttft, fair_pre, fair_steps = squeeze(dict(victim_policy=VICTIM_LARGEST, demote_victims=True,
                                                   admit_lookahead=8))
    quota_ttft, quota_pre, quota_steps = squeeze(dict(max_output_tokens=128))
    # the engine as described lets the long requests hold the pool: short ones queue behind them
    assert base_ttft > 4 * fair_ttft, (base_ttft, fair_ttft)
    # an output quota removes the squeeze altogether, at the price of truncating the long jobs
    assert quota_ttft < base_ttft and quota_steps < base_steps
    # every request still finishes under the fairness switches (no starvation in this mix)
    assert fair_steps < 4 * base_steps


@pytest.mark.parametrize("seed", range(6))
def test_random_traffic_under_random_policies_keeps_the_invariants(seed):
    """Whatever the switches: no physical block is ever in two tables of one iteration, the
    token budget holds, swapped blocks come back, everything drains and every block returns to
    the free list; quotas bound what a request generates and holds."""
    rng = np.random.default_rng(1000 + seed)
    policy = dict(victim_policy=int(rng.integers(0, 2)), demote_victims=bool(rng.integers(0, 2)),
                  admit_lookahead=int(rng.integers(0, 6)),
                  max_output_tokens=int(rng.choice([0, 40, 150])),
                  max_seq_blocks=int(rng.choice([0, 12, 30])))
    mode = int(rng.integers(0, 2))
    s = Scheduler(num_blocks=160, max_num_seqs=24, max_batched_tokens=192, max_blocks_per_seq=48,
                  host_blocks=int(rng.choice([0, 40, 400])), preempt_mode=mode)
    s.set_policy(**policy)
    n_req, added = 90, 0
    for step in range(200000):
        while added < n_req and added <= step // 2:           # arrivals spread over time
            assert s.add_request(added, int(rng.integers(1, 300)), int(rng.integers(1, 260)))
            added += 1
        st = s.step()
        if st.idle and added == n_req:
            break
        used = set()
        for tab, lens in ((st.decode_tables, st.decode_lens), (st.prefill_tables, st.prefill_ctx_lens)):
            for row, L in zip(tab, lens):
                blk = [int(b) for b in row[: (int(L) + 15) // 16]]
                assert all(0 <= b < 160 for b in blk) and not (used & set(blk)), policy
                if policy["max_seq_blocks"]:
                    assert len(blk) <= max(policy["max_seq_blocks"], 1 + 299 // 16), policy
                used |= set(blk)
        assert int(st.prefill_q_lens.sum()) + len(st.decode_ids) <= 192
        assert not (set(int(b) for b in st.swap_in_blocks) - used)   # restored blocks are in use
    else:
        raise AssertionError(f"did not drain under {policy}")
    stt = s.stats()
    assert stt.finished == n_req and stt.free_blocks == 160 and stt.running == 0 and stt.waiting == 0
    assert stt.swapped_in_blocks == stt.swapped_out_blocks
    for i in range(n_req):
        r = s.request_stats(i)
        assert r.finished_step >= r.first_token_step >= r.queued_step >= 0 or r.generated == 0
        if policy["max_output_tokens"]:
            assert r.generated <= policy["max_output_tokens"]
