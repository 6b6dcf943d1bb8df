/*
 * pagedkv.h -- C ABI of the B200 (sm_100a) paged-attention decode and KV-block swap library.
 *
 * The calls follow the serving model of the paper (arXiv 2602.07878): a decode step reads
 * the KV cache of every running sequence through a logical-to-physical block map
 * (Section 2.1 "Decoding", Section 2.2 "KV-Cache", Section 4.2 / Eq. 3), and preemption by
 * swapping moves a victim's KV blocks to host memory and later back into newly allocated
 * blocks (Section 5.1.2 "Swapping").
 *
 * Conventions for every call
 *   - Plain C types only.  "dev" pointers are CUDA device addresses, "host" pointers are
 *     host addresses; "pinned" means page-locked host memory that the GPU can address.
 *   - The caller owns every buffer (inputs, outputs, workspace, staging, host images).
 *     Unless a call's comment says otherwise the library allocates no device memory and
 *     keeps no state besides cached device properties.
 *   - Work is enqueued on `cuda_stream` (a cudaStream_t passed as void*, NULL = default
 *     stream) and the call returns without waiting for the GPU.
 *   - The return value is PA_OK or a negative PA_ERR_* code for an error found on the
 *     host; in that case nothing was launched.  Errors in device-resident data (a bad
 *     length or block id) cannot be seen by the host without a sync; they are reported
 *     through the optional `dev_status` word and never make the GPU read outside the pool.
 *   - bf16 is the only element type; accumulation is fp32.
 *   - Environment variables, each read once per process, for measurements and tests:
 *     PAGEDKV_PREFILL=mma selects the warp-level-MMA prefill kernel instead of the tcgen05 one;
 *     PAGEDKV_PREFILL_TILES=1|2 fixes the row tiles per CTA of the tcgen05 prefill kernel;
 *     PAGEDKV_VARIANT=warps,slots picks another compiled shape of the decode kernel (warps per
 *     CTA, TMA ring slots per warp; default 8,3).
 */
#ifndef PAGEDKV_H_
#define PAGEDKV_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

/* ---- host-side return codes ---------------------------------------------------------- */
#define PA_OK 0
#define PA_ERR_NULL (-1)      /* a required pointer is NULL                                */
#define PA_ERR_SHAPE (-2)     /* unsupported head_dim / block_size / head counts / strides */
#define PA_ERR_ALIGN (-3)     /* a buffer is not 16-byte aligned                           */
#define PA_ERR_WORKSPACE (-4) /* workspace / staging buffer too small                      */
#define PA_ERR_HOSTBUF (-5)   /* host image buffer too small                               */
#define PA_ERR_BLOCK_ID (-6)  /* swap block id out of range or listed twice                */
#define PA_ERR_CUDA (-7)      /* a CUDA runtime/driver call failed; see pa_last_cuda_error */
#define PA_ERR_ARG (-8)       /* negative count, bad partition size or similar             */
#define PA_ERR_STATIC_LIMIT (-9) /* pa_decode_static: needs more than PA_STATIC_WORKSPACE_BYTES */

/* ---- bits OR-ed into *dev_status by the kernels -------------------------------------- */
#define PA_STATUS_BAD_SEQ_LEN 1   /* seq_lens[b] < 0 or > max_blocks_per_seq * block_size  */
#define PA_STATUS_BAD_BLOCK_ID 2  /* a used block-table entry is outside [0, num_blocks)   */
#define PA_STATUS_TIMEOUT 4       /* a bounded wait inside a kernel gave up                */
#define PA_STATUS_WORKSPACE 8     /* the partition plan does not fit the workspace         */

#define PA_BF16 1

/* pa_decode flags */
#define PA_FLAG_REUSE_PLAN 1 /* skip planning: workspace still holds the plan of an earlier
                                call with the same seq_lens, batch and partition_tokens  */

/*
 * Geometry of one layer's K (and identically V) cache.  Element (block p, kv head h,
 * slot t, dim d) lives at  base + p*stride_block + h*stride_head + t*stride_tok + d
 * (strides in bf16 elements, dim is contiguous).  The recommended layout is
 * [num_blocks][num_kv_heads][block_size][head_dim]; any strides that are multiples of
 * 8 elements are accepted.
 */
typedef struct pa_shape {
    int32_t num_q_heads;  /* H; a multiple of num_kv_heads, H / Hkv <= 16                  */
    int32_t num_kv_heads; /* Hkv                                                           */
    int32_t head_dim;     /* D: 64, 128 or 256                                             */
    int32_t block_size;   /* tokens per block: 16                                          */
    int32_t num_blocks;   /* physical pool size, at least 1                                */
    int32_t dtype;        /* PA_BF16                                                       */
    int64_t stride_block;
    int64_t stride_head;
    int64_t stride_tok;
} pa_shape;

/* All layers of a pool: layer l of K starts layer_stride_k elements after layer l-1. */
typedef struct kv_pool_desc {
    int32_t num_layers;
    int32_t reserved;
    int64_t layer_stride_k;
    int64_t layer_stride_v;
} kv_pool_desc;

/*
 * Bytes of device workspace pa_decode needs for batches of at most `max_batch` sequences
 * holding at most `max_total_tokens` cached tokens in total.  `partition_tokens` is the
 * value that will be passed to pa_decode (0 = automatic).  The workspace holds the
 * partition plan and the fp32 partial results of sequences that are split (it serves the three
 * stages of a call: plan, partition attention, combine).
 */
int pa_workspace_bytes(const pa_shape* shape, int32_t max_batch, int64_t max_total_tokens,
                       int32_t partition_tokens, size_t* bytes);

/*
 * One decode-attention step over a paged KV cache (Section 2.1 / 2.2; Section 4.2, Eq. 3
 * for the traffic it causes).  For every sequence b < batch and query head h:
 *     out[b,h,:] = softmax_t( scale * <q[b,h,:], K[b,t,h/G,:]> ) . V[b,t,h/G,:],  t < seq_lens[b]
 * where token t of sequence b is slot t % block_size of physical block
 * block_tables[b][t / block_size] and G = num_q_heads / num_kv_heads.
 *
 *   q            dev bf16 [batch, H, D], contiguous, 16-byte aligned
 *   k_cache      dev bf16, one layer, laid out per `shape`; v_cache likewise
 *   block_tables dev int32 [batch, max_blocks_per_seq] row-major; entries at or beyond
 *                ceil(seq_lens[b] / block_size) are never read
 *   seq_lens     dev int32 [batch]; 0 gives a row of zeros.  The plan kernel reads them while
 *                the kernel before it in the stream may still run, if that kernel releases
 *                its dependents early (programmatic dependent launch; the combine kernel of
 *                the previous pa_decode call does, no kernel of this library writes
 *                seq_lens).  Copies, memsets and kernels that do not release their dependents
 *                early are complete before it reads, as stream order says.
 *   scale        softmax scale (e.g. 1/sqrt(D))
 *   out          dev bf16 [batch, H, D], contiguous, 16-byte aligned
 *   workspace    dev, >= pa_workspace_bytes(...), 256-byte aligned; contents are scratch.
 *                One call at a time per workspace: calls that may overlap on the GPU (different
 *                streams) need a workspace each.  Do not hand the same buffer to pa_prefill /
 *                pa_prefill_split as their workspace: consecutive calls of the library on
 *                one stream overlap at their edges, and only pa_decode calls among themselves
 *                keep out of each other's way inside a shared workspace
 *   partition_tokens  0 = choose per call from the batch's total length; otherwise a
 *                multiple of 16 in [16, 512]: sequences longer than this are split into
 *                partitions of this many tokens that run in parallel and are merged by
 *                log-sum-exp.  For a fixed value the result for a sequence depends on
 *                nothing but its own tokens (bit-identical across batches and block ids).
 *   flags        0 or PA_FLAG_REUSE_PLAN
 *   dev_status   dev int32 or NULL.  PA_STATUS_* bits are OR-ed in (never cleared).  A
 *                sequence with a bad length or a bad used block id gets an all-zero row;
 *                the GPU never reads outside the pool.
 * Slots of the last block beyond seq_lens[b] may hold anything (NaN included).
 * Three kernels are enqueued (plan, partition attention, combine); nothing is synced.
 * The workspace holds two plan regions used in turn, so the plan kernel of a call runs beside
 * the combine kernel of the call before it on the same stream and workspace.
 */
int pa_decode(const pa_shape* shape, const void* q, const void* k_cache, const void* v_cache,
              const int32_t* block_tables, int32_t max_blocks_per_seq, const int32_t* seq_lens,
              int32_t batch, float scale, void* out, void* workspace, size_t workspace_bytes,
              int32_t partition_tokens, int32_t flags, int32_t* dev_status, void* cuda_stream);

/*
 * pa_decode whose q and out are views into wider tensors (the same step of Section 2.1 / 2.2).
 * Tensor-parallel serving (Section 6.4: TP 2/4/8) gives each GPU a slice of the KV heads and the
 * query heads of their groups; an engine that keeps a batch-wide [batch, H_all, D] tensor, or
 * takes q straight out of a fused QKV projection, then holds this rank's heads as a strided view.
 * Row (b, h) of q starts at q + b * q_stride_seq + h * D elements, row (b, h) of out at
 * out + b * out_stride_seq + h * D: the H heads of one sequence stay contiguous, consecutive
 * sequences are q_stride_seq / out_stride_seq elements apart (each >= H * D and a multiple of
 * 8, else PA_ERR_ARG / PA_ERR_ALIGN).  Everything else, errors included, is pa_decode's; with
 * both strides equal to H * D the two calls are the same.  The cache slice of a rank is described
 * by `shape` as always (its strides may be those of a wider pool).
 */
int pa_decode_strided(const pa_shape* shape, const void* q, int64_t q_stride_seq,
                      const void* k_cache, const void* v_cache, const int32_t* block_tables,
                      int32_t max_blocks_per_seq, const int32_t* seq_lens, int32_t batch,
                      float scale, void* out, int64_t out_stride_seq, void* workspace,
                      size_t workspace_bytes, int32_t partition_tokens, int32_t flags,
                      int32_t* dev_status, void* cuda_stream);

/*
 * pa_decode for callers that cannot allocate device memory.  (The paper has no counterpart;
 * this is a convenience of the library.)
 *
 * Some users of this library are never in a position to call cudaMalloc for the workspace
 * pa_decode wants: an attention backend loaded into a serving engine that handed the whole
 * GPU to its KV pool at start-up and forbids later allocation, a plug-in that is only given
 * the tensors of the current step, or a latency-critical loop that must not hit the implicit
 * device synchronisation of the allocator.  For them the library carries its own scratch: a
 * fixed array of PA_STATIC_WORKSPACE_BYTES in device memory that belongs to the loaded
 * module.  Every GPU on which the library is loaded gives up that much memory until the
 * process exits, whether or not this entry point is ever called.
 *
 * Arguments are those of pa_decode without workspace / workspace_bytes / flags, plus
 *   max_total_tokens   an upper bound on the sum of seq_lens (the host cannot read them).
 * The call computes pa_workspace_bytes(shape, batch, max_total_tokens, partition_tokens)
 * and returns PA_ERR_STATIC_LIMIT, launching nothing, if that exceeds
 * PA_STATIC_WORKSPACE_BYTES.  (If the bound was understated the plan may not fit; that is
 * reported through PA_STATUS_WORKSPACE like in pa_decode and the output rows are zero.)
 * It calls no cudaMalloc / cudaFree and no allocating library routine; inputs and outputs
 * are still the caller's.
 *
 * First call on each device: the array's device address is looked up once per device (with
 * that device current) and cached.  Make that first call outside any stream capture.  On every
 * call the device that owns `cuda_stream` must be the current device (the cached address is
 * chosen by the current device's ordinal), and the cache does not survive cudaDeviceReset: a
 * process that resets a device must not call this entry point on it afterwards.
 * Sharing: all calls on a device use the same array, and it keeps what the last call left
 * there.  The call clears the plan header before use; everything else is overwritten
 * before it is read.  Two calls whose GPU work overlaps (different streams, or different
 * host threads feeding different streams) race on the array and corrupt each other's
 * results: serialise them on one stream or with events.  Plan reuse is not offered here for
 * the same reason.
 */
#define PA_STATIC_WORKSPACE_BYTES (64u << 20)
int pa_decode_static(const pa_shape* shape, const void* q, const void* k_cache,
                     const void* v_cache, const int32_t* block_tables,
                     int32_t max_blocks_per_seq, const int32_t* seq_lens, int32_t batch,
                     int64_t max_total_tokens, float scale, void* out, int32_t partition_tokens,
                     int32_t* dev_status, void* cuda_stream);

/* ---- sequence-split decode: one context sharded over several GPUs -------------------------
 * Tensor-parallel serving (Section 6.4, TP 2/4/8) shards KV heads, which needs no exchange
 * inside this path.  A context can also be split by tokens: each rank keeps a slice of every
 * sequence's blocks, attends over its slice, and the ranks exchange one small record per
 * rank before a final merge.  The merge is the same log-sum-exp combine that joins the
 * partitions of one call.
 *
 * A partial record for `rows` = batch * num_q_heads output rows of width D is
 * rows * (D + 2) floats: first the un-normalised accumulators o[rows][D]
 * (o = sum_t 2^(s_t - m) V_t over the rank's tokens, s_t = scale * log2(e) * <q, K_t>), then
 * (m, l)[rows] pairs with m the maximum of s_t and l = sum_t 2^(s_t - m).  A row whose
 * slice is empty has o = 0, m = -inf, l = 0; a row that met a bad block id has m = NaN.
 *
 * pa_partial_floats: floats to set aside for one record: rows * (D + 2) rounded up to a
 *   multiple of 4, so that records packed back to back stay 16-byte aligned.
 * pa_decode_partial: pa_decode over the rank's slice (its own block table rows and local
 *   lengths), result written as one record to `part` (device, 16-byte aligned).  All other
 *   arguments, the workspace and the errors are those of pa_decode.
 * pa_merge_partials: out[row] = sum_i 2^(m_i - M) o_i[row] / sum_i 2^(m_i - M) l_i, M = max m_i,
 *   rounded to bf16; a row with l = 0 in every record, or NaN in any, is zeros.  `parts` is a
 *   HOST array of num_parts (<= PA_MAX_PARTS) DEVICE pointers, each to one record; they are
 *   copied before return.  The kernel reads them with plain loads only, so a pointer may
 *   be a peer GPU's memory mapped into this process; the caller orders the merge after the
 *   records are complete (an all-gather on the same stream, or an event / barrier across
 *   ranks for peer pointers).  out: device bf16 [rows][head_dim]. */
#define PA_MAX_PARTS 32
int pa_partial_floats(const pa_shape* shape, int32_t batch, size_t* floats);
int pa_decode_partial(const pa_shape* shape, const void* q, const void* k_cache,
                      const void* v_cache, const int32_t* block_tables,
                      int32_t max_blocks_per_seq, const int32_t* seq_lens, int32_t batch,
                      float scale, float* part, void* workspace, size_t workspace_bytes,
                      int32_t partition_tokens, int32_t* dev_status, void* cuda_stream);
int pa_merge_partials(const float* const* parts, int32_t num_parts, int32_t rows,
                      int32_t head_dim, void* out, void* cuda_stream);

/* Bytes of device buffer pa_decode_host needs for its device copies of q, block tables,
 * lengths and out. */
int pa_host_io_bytes(const pa_shape* shape, int32_t max_batch, int32_t max_blocks_per_seq,
                     size_t* bytes);

/*
 * pa_decode for a caller whose per-step tensors live in pinned host memory.  seq_lens_host is
 * copied to `io_buf` (dev, >= pa_host_io_bytes).  q_host (groups of at most 8 query heads per KV
 * head, head_dim 64 or 128), block_tables_host (if 256 KiB or larger) and out_host are used in
 * place when they are pinned memory the GPU can address (the kernels then fetch query rows and
 * table entries ahead of use and post output rows over the host link while they run);
 * otherwise they go through `io_buf` as well.  Everything is enqueued on
 * `cuda_stream`; the KV cache itself stays on the device.  out_host is valid once the stream
 * has reached the end of this call, and the three host inputs must stay unchanged until then.
 */
int pa_decode_host(const pa_shape* shape, const void* q_host, const void* k_cache,
                   const void* v_cache, const int32_t* block_tables_host,
                   int32_t max_blocks_per_seq, const int32_t* seq_lens_host, int32_t batch,
                   float scale, void* out_host, void* io_buf, size_t io_bytes, void* workspace,
                   size_t workspace_bytes, int32_t partition_tokens, int32_t* dev_status,
                   void* cuda_stream);

/* Bytes of device workspace pa_prefill needs for at most `max_batch` sequences. */
int pa_prefill_workspace_bytes(int32_t max_batch, size_t* bytes);

/*
 * Prefill / recomputation attention over the paged cache (Section 2.1 "Prefill"; Section
 * 5.1.2 "Recomputation": a preempted request's prompt and generated tokens are re-processed;
 * Appendix B.1: prefill runs in chunks under a token budget).  Sequence b contributes
 * q_len_b = cu_q_lens[b+1] - cu_q_lens[b] query tokens: the last q_len_b of its ctx_lens[b]
 * cached tokens, whose K/V must already be in the cache (kv_append).  Query i of sequence b
 * sits at position pos = ctx_lens[b] - q_len_b + i and attends causally to tokens t <= pos:
 *     out[cu_q_lens[b] + i, h, :] = softmax_{t <= pos}(scale * <q, K_t>) . V_t
 *
 *   q             dev bf16 [total_q, H, D] (tokens of all sequences packed), 16-byte aligned
 *   k_cache, v_cache, block_tables, max_blocks_per_seq   as for pa_decode
 *   ctx_lens      dev int32 [batch]: cached tokens visible to the last query of the chunk
 *   cu_q_lens     dev int32 [batch + 1]: prefix sums of the query counts, cu_q_lens[0] = 0,
 *                 cu_q_lens[batch] = total_q
 *   out           dev bf16 [total_q, H, D]
 *   workspace     dev, >= pa_prefill_workspace_bytes(batch), 256-byte aligned
 *   dev_status    as for pa_decode: inconsistent lengths set PA_STATUS_BAD_SEQ_LEN (that
 *                 sequence's rows are left unwritten), a bad used block id sets
 *                 PA_STATUS_BAD_BLOCK_ID (affected rows are zero)
 * One or two kernels are enqueued (the attention kernel; before it a one-CTA plan when the
 * batch has more than 32 sequences or the warp-level kernel runs).
 */
int pa_prefill(const pa_shape* shape, const void* q, const void* k_cache, const void* v_cache,
               const int32_t* block_tables, int32_t max_blocks_per_seq, const int32_t* ctx_lens,
               const int32_t* cu_q_lens, int32_t batch, int32_t total_q, float scale, void* out,
               void* workspace, size_t workspace_bytes, int32_t* dev_status, void* cuda_stream);

/*
 * pa_prefill with the KV range of a tile split over several CTAs (flash-decoding applied to
 * the recomputation chunk of Section 5.1.2 / Appendix B.1: a 512-token chunk of one long
 * victim yields fewer 128-row tiles than the GPU has SMs, while each tile walks tens of
 * thousands of cached tokens).  The result is the same function of the inputs as pa_prefill;
 * only the order of the fp32 sums differs.  The units of a sequence whose context spans more
 * than one split leave per-split partial rows in the workspace and count themselves in; the
 * unit of a row group that arrives last merges them into the output rows, in the same kernel.
 * The counters carry the number of the call on that workspace (kept by the library, per
 * workspace address), so nothing in the workspace needs to be cleared by the caller; the first
 * call the library sees on a workspace enqueues one memset of its counters.
 *
 *   kv_split_tokens   0: the library chooses tile shape and split length from the chunk
 *                     size, max_blocks_per_seq (taken as the bound of every context: pass
 *                     a table no wider than the contexts need) and what the workspace holds;
 *                     > 0: split length in tokens (rounded up to a multiple of 64);
 *                     PA_ERR_WORKSPACE if ceil(max_blocks_per_seq * 16 / split) partial
 *                     rows per query row do not fit; < 0: never split.
 *   workspace         dev, 256-byte aligned, >= pa_prefill_workspace_bytes(batch); splits are
 *                     used up to what pa_prefill_split_workspace_bytes(shape, batch, total_q,
 *                     splits) says fits.
 * pa_prefill is this call with kv_split_tokens = 0.
 * One or two kernels are enqueued (plan, attention).  Errors as for pa_prefill; a split that met
 * a bad block id zeroes the rows that depend on it.
 */
int pa_prefill_split_workspace_bytes(const pa_shape* shape, int32_t max_batch,
                                     int32_t max_total_q, int32_t max_splits, size_t* bytes);
int pa_prefill_split(const pa_shape* shape, const void* q, const void* k_cache,
                     const void* v_cache, const int32_t* block_tables,
                     int32_t max_blocks_per_seq, const int32_t* ctx_lens,
                     const int32_t* cu_q_lens, int32_t batch, int32_t total_q, float scale,
                     void* out, void* workspace, size_t workspace_bytes, int32_t kv_split_tokens,
                     int32_t* dev_status, void* cuda_stream);
/* What pa_prefill_split would launch for these arguments on a GPU with `sm_count` SMs: row
 * tiles per CTA (0 = the warp-level kernel), split length in tokens (0 = unsplit) and
 * partial rows per query row.  Host arithmetic only (no GPU is touched): the cost model
 * behind kv_split_tokens = 0 can be examined, and a caller can size its workspace by trying
 * sizes.  Returns PA_ERR_WORKSPACE where pa_prefill_split would.  No counterpart in the paper. */
int pa_prefill_select_launch(const pa_shape* shape, int32_t batch, int32_t total_q,
                             int32_t max_blocks_per_seq, size_t workspace_bytes,
                             int32_t kv_split_tokens, int32_t sm_count, int32_t* tiles_per_cta,
                             int32_t* split_tokens, int32_t* kv_splits);
/* What the calling thread's last pa_prefill / pa_prefill_split launched: row tiles per CTA (0 =
 * the warp-level kernel), split length in tokens (0 = unsplit) and partial rows per query row.
 * A measurement and test aid; no counterpart in the paper. */
int pa_prefill_last_launch(int32_t* tiles_per_cta, int32_t* kv_split_tokens, int32_t* kv_splits);

/*
 * KV append (Section 2.2 "KV-Cache": with every decoding step the KV vectors of the newly
 * generated token are appended to the cache).  For every b < batch with slot_mapping[b] >= 0
 * the rows k_new[b,:,:] and v_new[b,:,:] are written to slot (slot_mapping[b] % block_size)
 * of physical block (slot_mapping[b] / block_size) of one layer's caches.
 *
 *   k_cache, v_cache  dev bf16, one layer, laid out per `shape` (written in place)
 *   k_new, v_new      dev bf16 [batch, Hkv, D], contiguous, 16-byte aligned
 *   slot_mapping      dev int64 [batch]; negative = padding entry, nothing is written;
 *                     a slot at or beyond num_blocks * block_size writes nothing and sets
 *                     PA_STATUS_BAD_BLOCK_ID in *dev_status (dev int32 or NULL)
 * Two tokens mapped to the same slot in one call leave either one there.  One kernel is
 * enqueued on `cuda_stream`.
 */
int kv_append(const pa_shape* shape, void* k_cache, void* v_cache, const void* k_new,
              const void* v_new, const int64_t* slot_mapping, int32_t batch,
              int32_t* dev_status, void* cuda_stream);

/* Bytes of one block's host image: num_layers * 2 * Hkv * block_size * D * 2. */
int kv_block_bytes(const kv_pool_desc* pool, const pa_shape* shape, size_t* bytes);

/*
 * Swap-out (Section 5.1.2 "Swapping": the victim's KV blocks are offloaded from GPU
 * memory to host memory).  Packs whole blocks -- every layer, K then V, unused slots
 * included, bit for bit -- into a contiguous host image laid out
 *     [i < n][layer][K|V][kv head][slot][dim]
 * so that slot i of the image holds physical block block_ids[i].
 *
 *   k_pool, v_pool   dev bf16 pools holding all layers (see kv_pool_desc / pa_shape)
 *   block_ids        HOST int32 [n]; copied before the call returns; each in
 *                    [0, num_blocks) and listed once
 *   pinned_host_buf  pinned host memory, 16-byte aligned, >= n * kv_block_bytes
 *   staging          dev scratch or NULL.  With a staging buffer (any size >= one block
 *                    image, 256-byte aligned) blocks are gathered into it by a kernel and
 *                    moved by the copy engine; with NULL the gather kernel stores straight
 *                    into the pinned buffer.  A swap larger than the staging buffer is moved
 *                    in pieces that alternate between the buffer's two halves (each at least
 *                    one block image), the copy of one piece running beside the gather of
 *                    the next: for the length of such a call the library creates a side
 *                    stream and four events, tied to `cuda_stream` by event waits and
 *                    destroyed before the call returns.
 * The image is complete when `cuda_stream` reaches the end of the call.
 */
int kv_swap_out(const kv_pool_desc* pool, const pa_shape* shape, const void* k_pool,
                const void* v_pool, const int32_t* block_ids, int32_t n, void* pinned_host_buf,
                size_t host_bytes, void* staging, size_t staging_bytes, void* cuda_stream);

/*
 * Swap-in (Section 5.1.2: the blocks migrate back over the host link when the victim is
 * re-admitted, into whatever blocks the allocator hands out).  Inverse of kv_swap_out:
 * image slot i is written to physical block block_ids[i]; no other byte of the pools
 * changes.  Arguments as for kv_swap_out.
 */
int kv_swap_in(const kv_pool_desc* pool, const pa_shape* shape, void* k_pool, void* v_pool,
               const void* pinned_host_buf, size_t host_bytes, const int32_t* block_ids,
               int32_t n, void* staging, size_t staging_bytes, void* cuda_stream);

/*
 * Per-kernel timing of pa_decode (no counterpart in the paper; a measurement aid).  While
 * enabled, every pa_decode call records CUDA events on its stream before the plan kernel,
 * before and after the partition-attention kernel and after the combine kernel.
 * pa_profile_read waits for the recorded calls to finish, returns the summed device time of
 * each kernel in milliseconds and the number of calls, and forgets them.  Any output
 * pointer may be NULL.  Events are host objects; no device memory is allocated.
 */
int pa_profile_enable(int on);
int pa_profile_read(double* plan_ms, double* attention_ms, double* combine_ms, int64_t* calls);

/*
 * Read-bandwidth probe (no counterpart in the paper; a measurement aid).  One kernel reads
 * `bytes` (rounded down to 4 KiB granules) of `dev_buf` and nothing else: granule by granule
 * in order (scattered = 0) or in a pseudo-random order that visits every granule once
 * (scattered != 0), each granule with one bulk asynchronous copy into shared memory -- the
 * mechanism and granule size of the attention kernel's K/V tiles.  bytes / elapsed time is the
 * practical ceiling for a read-only stream, respectively for 4 KiB gathers out of a fragmented
 * pool.  dev_sink (dev, 8 bytes, may be NULL) is never written in practice; dev_status gets
 * PA_STATUS_TIMEOUT if a bounded wait gives up.
 */
int pa_probe_read(const void* dev_buf, size_t bytes, int32_t scattered, uint32_t seed,
                  void* dev_sink, int32_t* dev_status, void* cuda_stream);

/*
 * Issue-rate probe for tiled TMA loads (no counterpart in the paper; a measurement aid behind
 * the choice of four producer warps in the prefill kernel).  `dev_buf` (256-byte aligned, 64 KiB
 * to 2 GiB, whole multiples of 32 KiB are used) is viewed as [blocks][8][16][128] bf16; on every
 * SM `warps` warps (1..8) each keep six ring slots in flight and issue, per slot, `boxes` boxes
 * of 2 KB (64 dims x 16 tokens: the K/V box of the attention kernels) from as many lanes of one
 * instruction (`boxes` even, 2..16, warps * boxes <= 16), walking the buffer `reps` times.  With
 * a buffer that fits L2 the elapsed time measures how fast boxes can be issued and delivered.
 * *boxes_issued (host, may be NULL) receives the number of boxes the launch issues in total.
 * dev_status gets PA_STATUS_TIMEOUT if a bounded wait gives up.
 */
int pa_probe_tma_issue(const void* dev_buf, size_t bytes, int32_t warps, int32_t boxes,
                       int32_t reps, int64_t* boxes_issued, int32_t* dev_status,
                       void* cuda_stream);

/*
 * Self-test of the bounded waits (no counterpart in the paper).  Every wait inside the
 * kernels (on TMA data, on tensor-core completion, on another warp) gives up after a wall-
 * clock limit, reports PA_STATUS_TIMEOUT and lets the kernel return, so that a lost signal
 * costs an error code and not a hung GPU.  This call launches one warp that performs such a
 * wait on a barrier nobody completes, with a limit of `limit_us` microseconds (1..100000),
 * and ORs PA_STATUS_TIMEOUT into *dev_status (dev int32) when the limit has passed.
 */
int pa_selftest_wait_expiry(int32_t limit_us, int32_t* dev_status, void* cuda_stream);

/* Text for a PA_* return code. */
const char* pa_status_string(int code);

/* The cudaError_t / CUresult value behind the calling thread's last PA_ERR_CUDA (0 if none). */
int pa_last_cuda_error(void);

/* Number of kernels the library has launched since it was loaded (all threads). */
int64_t pa_launch_count(void);

#ifdef __cplusplus
}
#endif
#endif /* PAGEDKV_H_ */
