// Host-side block manager and iteration-level scheduler, modelled on the serving engine the
// paper analyses (Section 5.1 "Revisiting vLLM Scheduler"):
//   * a global free-block queue that running sequences consume as they decode (5.1.1);
//   * FCFS admission from WAITING through can_allocate(); a head request that does not fit
//     stops admission for everyone behind it (memory-based head-of-line blocking, 5.1.1);
//   * when running sequences outgrow the pool, the most recently admitted one is preempted
//     (LIFO) and put back at the FRONT of WAITING (5.1.2);
//   * recovery by swapping (the victim's blocks go to host memory and come back into newly
//     allocated blocks) or by recomputation (its KV is dropped and prompt + generated tokens
//     are prefilled again), prefill running in chunks under a per-iteration token budget
//     (Appendix B.1);
//   * optionally the countermeasures Section 7 names (output-length and memory quotas, a
//     fairness-aware choice of victim and of the next request to admit), as switches on the
//     same engine so that their effect on queueing and preemption can be measured.
// It produces, per iteration, exactly what the GPU entry points take: block tables and
// lengths for pa_decode, slot mappings for kv_append, (query, context) lengths for
// pa_prefill, and block-id lists for kv_swap_out / kv_swap_in.  No prompt or probe tooling.
#include <algorithm>
#include <cstdint>
#include <deque>
#include <unordered_map>
#include <vector>

#include "../../include/pagedkv_sched.h"

namespace {

enum State { WAITING_NEW, WAITING_SWAPPED, WAITING_RECOMPUTE, PREFILL, DECODE, FINISHED };

struct Seq {
    int64_t id;
    int32_t prompt_len, max_new, generated;
    int32_t len;        // tokens whose KV is in the cache
    int32_t target;     // tokens that must be prefilled before decoding (prompt [+ generated])
    State state;
    std::vector<int32_t> blocks;  // logical -> physical
    int32_t host_start, host_slots;  // range of host slots holding its blocks while swapped out
    int64_t admitted_at;          // order of admission, for LIFO victim choice
    int64_t queued_step, first_token_step, finished_step;
    int32_t preemptions;
};

struct Sched {
    sched_config cfg;
    sched_policy policy{};
    std::unordered_map<int64_t, int> by_id;
    std::deque<int32_t> free_blocks;
    std::vector<Seq> seqs;
    std::deque<int> waiting;  // indices into seqs, front = head of line
    std::vector<int> running;  // admission order
    int64_t clock = 0, admit_counter = 0;
    sched_stats stats{};
    // buffers behind the pointers of the last sched_step
    std::vector<int64_t> o_decode_ids, o_prefill_ids, o_slots, o_prefill_slots, o_finished;
    std::vector<int32_t> o_lens, o_tables, o_pf_q, o_pf_ctx, o_pf_tables, o_swap_out, o_swap_in_src,
        o_swap_in_dst, o_swap_out_host;

    std::vector<std::pair<int32_t, int32_t>> host_free;  // (start, length) ranges, sorted

    int host_alloc(int n) {  // first fit; -1 if the swap space is full
        for (size_t i = 0; i < host_free.size(); ++i)
            if (host_free[i].second >= n) {
                const int start = host_free[i].first;
                host_free[i].first += n;
                host_free[i].second -= n;
                if (host_free[i].second == 0) host_free.erase(host_free.begin() + i);
                return start;
            }
        return -1;
    }
    void host_release(int start, int n) {
        auto it = std::lower_bound(host_free.begin(), host_free.end(), std::make_pair(start, 0));
        it = host_free.insert(it, {start, n});
        if (it + 1 != host_free.end() && it->first + it->second == (it + 1)->first) {
            it->second += (it + 1)->second;
            host_free.erase(it + 1);
        }
        if (it != host_free.begin() && (it - 1)->first + (it - 1)->second == it->first) {
            (it - 1)->second += it->second;
            host_free.erase(it);
        }
    }
    int blocks_for(int tokens) const { return (tokens + cfg.block_size - 1) / cfg.block_size; }
    bool take(Seq& s, int n) {
        if ((int)free_blocks.size() < n) return false;
        for (int i = 0; i < n; ++i) {
            s.blocks.push_back(free_blocks.front());
            free_blocks.pop_front();
        }
        return true;
    }
    void release(Seq& s) {
        for (int32_t b : s.blocks) free_blocks.push_back(b);
        s.blocks.clear();
    }
};

// Preempt a running sequence (Section 5.1.2): its blocks are reclaimed and it goes back to the
// FRONT of the waiting queue.  Swap mode keeps its KV in host slots; recompute mode (and any
// victim still in prefill, or a full swap space) drops the KV and re-prefills later.
void preempt(Sched& S, int idx) {
    Seq& s = S.seqs[idx];
    ++S.stats.preemptions;
    ++s.preemptions;
    int host = -1;
    if (S.cfg.preempt_mode == SCHED_PREEMPT_SWAP && s.state == DECODE)
        host = S.host_alloc((int)s.blocks.size());
    if (host >= 0) {
        for (size_t i = 0; i < s.blocks.size(); ++i) {
            S.o_swap_out.push_back(s.blocks[i]);
            S.o_swap_out_host.push_back(host + (int)i);
        }
        S.stats.swapped_out_blocks += (int64_t)s.blocks.size();
        s.host_start = host;
        s.host_slots = (int)s.blocks.size();
        s.state = WAITING_SWAPPED;
    } else {
        S.stats.recomputed_tokens += s.len;
        s.target = s.prompt_len + s.generated;
        s.len = 0;
        s.state = WAITING_RECOMPUTE;
    }
    S.release(s);
    S.running.erase(std::find(S.running.begin(), S.running.end(), idx));
    if (S.policy.demote_victims) S.waiting.push_back(idx); else S.waiting.push_front(idx);
}

// Which running sequence gives up its blocks: the last admitted one (Section 5.1.2), or, as a
// fairness measure, the one that holds the most blocks (ties: the later admitted).
int pick_victim(const Sched& S) {
    if (S.policy.victim_policy == SCHED_VICTIM_LIFO) return S.running.back();
    int best = S.running.back();
    for (int idx : S.running)
        if (S.seqs[idx].blocks.size() > S.seqs[best].blocks.size() ||
            (S.seqs[idx].blocks.size() == S.seqs[best].blocks.size() &&
             S.seqs[idx].admitted_at > S.seqs[best].admitted_at))
            best = idx;
    return best;
}

void finish(Sched& S, int idx) {
    Seq& s = S.seqs[idx];
    S.o_finished.push_back(s.id);
    S.release(s);
    s.state = FINISHED;
    s.finished_step = S.stats.steps;
    S.running.erase(std::find(S.running.begin(), S.running.end(), idx));
    ++S.stats.finished;
}

void write_table(const Sched& S, const Seq& s, std::vector<int32_t>& dst) {
    const size_t base = dst.size();
    dst.resize(base + S.cfg.max_blocks_per_seq, -1);
    std::copy(s.blocks.begin(), s.blocks.end(), dst.begin() + base);
}

int64_t slot_of(const Sched& S, const Seq& s, int token) {
    return (int64_t)s.blocks[token / S.cfg.block_size] * S.cfg.block_size + token % S.cfg.block_size;
}

}  // namespace

extern "C" void* sched_create(const sched_config* cfg) {
    if (!cfg || cfg->num_blocks <= 0 || cfg->block_size <= 0 || cfg->max_num_seqs <= 0 ||
        cfg->max_batched_tokens <= 0 || cfg->max_blocks_per_seq <= 0 || cfg->host_blocks < 0 ||
        (cfg->preempt_mode != SCHED_PREEMPT_SWAP && cfg->preempt_mode != SCHED_PREEMPT_RECOMPUTE))
        return nullptr;
    Sched* S = new Sched();
    S->cfg = *cfg;
    for (int i = 0; i < cfg->num_blocks; ++i) S->free_blocks.push_back(i);
    if (cfg->host_blocks > 0) S->host_free.push_back({0, cfg->host_blocks});
    return S;
}

extern "C" void sched_destroy(void* sched) { delete static_cast<Sched*>(sched); }

extern "C" int sched_add_request(void* sched, int64_t id, int32_t prompt_len,
                                 int32_t max_new_tokens) {
    Sched& S = *static_cast<Sched*>(sched);
    if (prompt_len <= 0 || max_new_tokens <= 0) return -1;
    const int need = S.blocks_for(prompt_len + max_new_tokens);
    if (need > S.cfg.max_blocks_per_seq || need > S.cfg.num_blocks) return -1;
    Seq s{};
    s.id = id;
    s.prompt_len = prompt_len;
    s.max_new = max_new_tokens;
    s.target = prompt_len;
    s.state = WAITING_NEW;
    s.queued_step = S.stats.steps;
    s.first_token_step = s.finished_step = -1;
    if (S.by_id.count(id)) return -1;
    S.by_id[id] = (int)S.seqs.size();
    S.seqs.push_back(s);
    S.waiting.push_back((int)S.seqs.size() - 1);
    return 0;
}

extern "C" void sched_get_stats(const void* sched, sched_stats* stats) {
    const Sched& S = *static_cast<const Sched*>(sched);
    *stats = S.stats;
    stats->free_blocks = (int32_t)S.free_blocks.size();
    stats->running = (int32_t)S.running.size();
    stats->waiting = (int32_t)S.waiting.size();
}

extern "C" int sched_set_policy(void* sched, const sched_policy* p) {
    if (!sched || !p) return -1;
    if ((p->victim_policy != SCHED_VICTIM_LIFO && p->victim_policy != SCHED_VICTIM_LARGEST) ||
        p->admit_lookahead < 0 || p->max_output_tokens < 0 || p->max_seq_blocks < 0 ||
        (p->demote_victims != 0 && p->demote_victims != 1))
        return -1;
    static_cast<Sched*>(sched)->policy = *p;
    return 0;
}

extern "C" int sched_get_request_stats(const void* sched, int64_t id, sched_request_stats* out) {
    const Sched& S = *static_cast<const Sched*>(sched);
    auto it = S.by_id.find(id);
    if (it == S.by_id.end() || !out) return -1;
    const Seq& s = S.seqs[it->second];
    *out = {s.queued_step, s.first_token_step, s.finished_step, s.preemptions, s.generated};
    return 0;
}

extern "C" int sched_step(void* sched, sched_step_out* out) {
    Sched& S = *static_cast<Sched*>(sched);
    const int bs = S.cfg.block_size;
    for (auto* v : {&S.o_decode_ids, &S.o_prefill_ids, &S.o_slots, &S.o_prefill_slots, &S.o_finished})
        v->clear();
    for (auto* v : {&S.o_lens, &S.o_tables, &S.o_pf_q, &S.o_pf_ctx, &S.o_pf_tables, &S.o_swap_out,
                    &S.o_swap_in_src, &S.o_swap_in_dst, &S.o_swap_out_host})
        v->clear();
    if (S.running.empty() && S.waiting.empty()) {
        *out = sched_step_out{};
        return 1;
    }
    ++S.stats.steps;

    // ---- 1. every decoding sequence needs room for its next token (5.1.1); when the pool
    //         runs dry the most recently admitted sequence is evicted (5.1.2, LIFO) ----------
    for (size_t i = 0; i < S.running.size();) {
        const int idx = S.running[i];
        Seq& s = S.seqs[idx];
        if (s.state != DECODE || s.len % bs != 0 || (int)s.blocks.size() > s.len / bs) {
            ++i;
            continue;
        }
        // memory quota: a sequence at its cap is cut off instead of growing
        if (S.policy.max_seq_blocks > 0 && (int)s.blocks.size() >= S.policy.max_seq_blocks) {
            finish(S, idx);
            continue;
        }
        bool self_evicted = false;
        while (S.free_blocks.empty()) {
            const int victim = pick_victim(S);
            const size_t vpos = std::find(S.running.begin(), S.running.end(), victim) - S.running.begin();
            preempt(S, victim);
            if (victim == idx) {
                self_evicted = true;
                break;
            }
            if (vpos < i) --i;  // a victim ahead of this sequence left the list: positions shift
        }
        if (self_evicted) continue;  // running shrank; position i now holds the next sequence
        S.take(s, 1);
        ++i;
    }

    // ---- 2. FCFS admission: the head of WAITING must fit, or nobody behind it is looked at ---
    int budget = S.cfg.max_batched_tokens;
    for (int idx : S.running)
        if (S.seqs[idx].state == DECODE) --budget;
    bool blocked = false;
    size_t pos = 0;  // position in WAITING being tried; > 0 only behind a head that does not fit
    int skipped = 0;
    while (pos < S.waiting.size() && (int)S.running.size() < S.cfg.max_num_seqs) {
        const int idx = S.waiting[pos];
        Seq& s = S.seqs[idx];
        const bool swapped = s.state == WAITING_SWAPPED;
        // a swapped sequence comes back whole and also needs the block of its next token
        const int need = swapped ? std::max(s.host_slots, S.blocks_for(s.len + 1))
                                 : S.blocks_for(s.target);
        if (!swapped && budget <= 0) break;  // no prefill tokens left this iteration
        if ((int)S.free_blocks.size() < need) {  // can_allocate() fails: head-of-line blocking,
            blocked = true;                      // unless the policy lets a few requests pass
            if (skipped >= S.policy.admit_lookahead) break;
            ++skipped;
            ++pos;
            continue;
        }
        S.waiting.erase(S.waiting.begin() + pos);
        S.take(s, need);
        if (swapped) {
            for (int i = 0; i < s.host_slots; ++i) {
                S.o_swap_in_src.push_back(s.host_start + i);
                S.o_swap_in_dst.push_back(s.blocks[i]);
            }
            S.stats.swapped_in_blocks += s.host_slots;
            S.host_release(s.host_start, s.host_slots);
            s.host_slots = 0;
            s.state = DECODE;
            --budget;  // it decodes in this very iteration
        } else {
            s.state = PREFILL;
            s.len = 0;
        }
        s.admitted_at = S.admit_counter++;
        S.running.push_back(idx);
    }
    if (blocked) ++S.stats.hol_blocked_steps;

    // ---- 3. this iteration's batch: one token per decoding sequence, then prefill chunks
    //         under what is left of the token budget (Appendix B.1) ---------------------------
    std::vector<int> done;
    for (int idx : S.running) {
        Seq& s = S.seqs[idx];
        if (s.state != DECODE) continue;
        S.o_decode_ids.push_back(s.id);
        S.o_slots.push_back(slot_of(S, s, s.len));
        S.o_lens.push_back(s.len + 1);
        write_table(S, s, S.o_tables);
        ++s.len;
        ++s.generated;
        ++S.stats.decode_tokens;
        if (s.first_token_step < 0) s.first_token_step = S.stats.steps;
        const int cap = S.policy.max_output_tokens > 0 ? std::min(s.max_new, S.policy.max_output_tokens)
                                                       : s.max_new;
        if (s.generated >= cap) done.push_back(idx);
    }
    int prefill_tokens = 0;
    for (int idx : S.running) {
        Seq& s = S.seqs[idx];
        if (s.state != PREFILL || budget <= 0) continue;
        const int q = std::min(s.target - s.len, budget);
        for (int t = s.len; t < s.len + q; ++t) S.o_prefill_slots.push_back(slot_of(S, s, t));
        S.o_prefill_ids.push_back(s.id);
        S.o_pf_q.push_back(q);
        S.o_pf_ctx.push_back(s.len + q);
        write_table(S, s, S.o_pf_tables);
        s.len += q;
        budget -= q;
        prefill_tokens += q;
        if (s.len == s.target) s.state = DECODE;  // decodes from the next iteration on
    }
    S.stats.prefill_tokens += prefill_tokens;
    for (int idx : done) finish(S, idx);

    out->n_decode = (int32_t)S.o_decode_ids.size();
    out->decode_ids = S.o_decode_ids.data();
    out->decode_lens = S.o_lens.data();
    out->decode_slots = S.o_slots.data();
    out->decode_tables = S.o_tables.data();
    out->n_prefill = (int32_t)S.o_prefill_ids.size();
    out->prefill_tokens = prefill_tokens;
    out->prefill_ids = S.o_prefill_ids.data();
    out->prefill_q_lens = S.o_pf_q.data();
    out->prefill_ctx_lens = S.o_pf_ctx.data();
    out->prefill_tables = S.o_pf_tables.data();
    out->prefill_slots = S.o_prefill_slots.data();
    out->n_swap_out = (int32_t)S.o_swap_out.size();
    out->swap_out_blocks = S.o_swap_out.data();
    out->swap_out_host_slots = S.o_swap_out_host.data();
    out->n_swap_in = (int32_t)S.o_swap_in_src.size();
    out->swap_in_host_slots = S.o_swap_in_src.data();
    out->swap_in_blocks = S.o_swap_in_dst.data();
    out->n_finished = (int32_t)S.o_finished.size();
    out->finished_ids = S.o_finished.data();
    return 0;
}
