/*
 * pagedkv_sched.h -- host-side block manager and iteration-level scheduler (plain C ABI).
 *
 * A model of the engine the paper analyses (Section 5.1): a global free-block queue, FCFS
 * admission with can_allocate() and memory-based head-of-line blocking (5.1.1), LIFO
 * preemption with the victim put back at the front of WAITING, recovery by swapping or by
 * recomputation (5.1.2), and chunked prefill under a per-iteration token budget (Appendix
 * B.1).  Every iteration it emits the arguments of the GPU entry points of pagedkv.h.  All
 * pointers in sched_step_out point into the scheduler object and stay valid until the next
 * sched_step / sched_destroy.  Nothing here touches a GPU.
 */
#ifndef PAGEDKV_SCHED_H_
#define PAGEDKV_SCHED_H_

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define SCHED_PREEMPT_SWAP 0
#define SCHED_PREEMPT_RECOMPUTE 1

typedef struct sched_config {
    int32_t num_blocks;          /* physical KV blocks in the pool                          */
    int32_t block_size;          /* tokens per block                                        */
    int32_t max_num_seqs;        /* cap on RUNNING sequences                                */
    int32_t max_batched_tokens;  /* token budget per iteration (decode tokens + prefill)    */
    int32_t preempt_mode;        /* SCHED_PREEMPT_SWAP or SCHED_PREEMPT_RECOMPUTE           */
    int32_t max_blocks_per_seq;  /* row width of the emitted block tables                   */
    int32_t host_blocks;         /* capacity of the host swap space, in blocks              */
} sched_config;

typedef struct sched_stats {
    int64_t steps, preemptions, swapped_out_blocks, swapped_in_blocks, recomputed_tokens;
    int64_t finished, hol_blocked_steps, decode_tokens, prefill_tokens;
    int32_t free_blocks, running, waiting, reserved;
} sched_stats;

typedef struct sched_step_out {
    /* decode set: one new token per sequence; lens include it; slots = where its K/V go */
    int32_t n_decode;
    const int64_t* decode_ids;
    const int32_t* decode_lens;
    const int64_t* decode_slots;
    const int32_t* decode_tables;       /* [n_decode][max_blocks_per_seq], unused entries -1 */
    /* prefill chunks: sequence i contributes prefill_q_lens[i] query tokens ending at
       context length prefill_ctx_lens[i]; prefill_slots lists the slots of all of them */
    int32_t n_prefill;
    int32_t prefill_tokens;
    const int64_t* prefill_ids;
    const int32_t* prefill_q_lens;
    const int32_t* prefill_ctx_lens;
    const int32_t* prefill_tables;      /* [n_prefill][max_blocks_per_seq] */
    const int64_t* prefill_slots;       /* [prefill_tokens] */
    /* swaps decided this iteration: device block <-> host slot pairs, in order */
    int32_t n_swap_out;
    const int32_t* swap_out_blocks;
    const int32_t* swap_out_host_slots;
    int32_t n_swap_in;
    const int32_t* swap_in_host_slots;
    const int32_t* swap_in_blocks;
    int32_t n_finished;
    const int64_t* finished_ids;
} sched_step_out;

/*
 * Countermeasures (Section 7 "Countermeasures" names them without defining them; the readings
 * taken here are stated per field).  All zero = the engine of Section 5.1 unchanged.
 */
#define SCHED_VICTIM_LIFO 0     /* Section 5.1.2: the most recently admitted sequence            */
#define SCHED_VICTIM_LARGEST 1  /* fairness: the running sequence that holds the most blocks     */
typedef struct sched_policy {
    int32_t victim_policy;     /* SCHED_VICTIM_*                                                 */
    int32_t demote_victims;    /* 1: a preempted sequence re-queues at the BACK of WAITING (it is
                                  "de-escalated"), not at the front                              */
    int32_t admit_lookahead;   /* fairness: when the head of WAITING does not fit, up to this many
                                  requests behind it are tried (0 = strict FCFS, head-of-line
                                  blocking as in Section 5.1.1)                                  */
    int32_t max_output_tokens; /* quota: a request finishes after this many generated tokens even
                                  if it asked for more (0 = no cap)                              */
    int32_t max_seq_blocks;    /* quota: a request that would need more KV blocks than this is
                                  finished (truncated) instead of growing (0 = no cap)           */
} sched_policy;

/* Per-request outcome in iterations (the scheduler's clock): the step it was queued at, the
 * step that produced its first generated token (-1 if none yet), the step it finished at (-1
 * if not yet), how often it was preempted, how many tokens it generated. */
typedef struct sched_request_stats {
    int64_t queued_step, first_token_step, finished_step;
    int32_t preemptions, generated;
} sched_request_stats;

/* Returns NULL on an invalid configuration. */
void* sched_create(const sched_config* cfg);
void sched_destroy(void* sched);
/* Queue a request (FCFS).  Returns 0, or -1 if it can never fit (prompt + max_new_tokens
 * needs more than max_blocks_per_seq or num_blocks blocks). */
int sched_add_request(void* sched, int64_t id, int32_t prompt_len, int32_t max_new_tokens);
/* Run one iteration.  Returns 0, or 1 when nothing is running or waiting any more. */
int sched_step(void* sched, sched_step_out* out);
void sched_get_stats(const void* sched, sched_stats* stats);
/* Set the countermeasures; takes effect from the next sched_step.  Returns 0, or -1 on an
 * unknown policy or a negative field. */
int sched_set_policy(void* sched, const sched_policy* policy);
/* Outcome of request `id` so far.  Returns 0, or -1 if the id is unknown. */
int sched_get_request_stats(const void* sched, int64_t id, sched_request_stats* out);

#ifdef __cplusplus
}
#endif
#endif /* PAGEDKV_SCHED_H_ */
