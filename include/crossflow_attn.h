/*
 * crossflow_attn — mixed decode + chunked-prefill paged grouped-query attention for one B200.
 *
 * The workload is the one a Crossflow decode node produces (arxiv 2609.27085): the worker keeps
 * a local prefill queue, reuses any resident prefix and "construct[s] a mixed prefill/decode
 * batch" (Section 5); prefill is issued in bounded units that are revalidated between units
 * (Section 4.4), so one call here is one unit of one layer: many one-token decode sequences
 * plus a few prefill chunks, each chunk attending causally to its own new tokens and to an
 * already-cached prefix.  The paper adds no model kernels (Section 5) and gives no formula;
 * the arithmetic is textbook softmax attention over a paged KV cache:
 *
 *   sequence s, new-token row i in [0, query_len[s]), query head h:
 *     p = context_len[s] - query_len[s] + i,  g = h / (num_q_heads / num_kv_heads)
 *     x_j = softmax_scale * <q, k_j>  for j in [0, p],  k_j/v_j at page block_table[s][j / B], slot j % B, head g
 *     out = sum_j softmax(x)_j * v_j ,  lse = ln sum_j exp(x_j)
 *
 * Conventions
 *   - bf16 storage, fp32 accumulation, one fp32 -> bf16 rounding (nearest even) of the output.
 *   - context_len[s] counts the visible KV tokens INCLUDING this call's query_len[s] new tokens.
 *   - Rows of q / k_new / v_new / out are packed in sequence order: sequence s owns rows
 *     [sum_{t<s} query_len[t], ... + query_len[s]).  Decode (query_len 1) and prefill
 *     (query_len > 1) sequences may appear in any order; query_len 0 is legal (no rows).
 *   - Block-table entries past ceil(context_len/B), cache slots past context_len and unassigned
 *     pages are never read into the result (they may hold NaN).  An entry in use that lies outside
 *     [0, num_blocks) is never dereferenced: a new row aimed at it is not written, attention reads page 0
 *     in its place (the rows of that sequence are then meaningless) and cf_get_async_status reports
 *     CF_ERR_OUT_OF_RANGE.
 *   - Pointers marked DEVICE must be device memory of the context's GPU and stay alive until the
 *     stream has finished the enqueued work.  Pointers marked HOST are read before the call returns.
 *   - All calls on one context must be issued on one stream (or be ordered by the caller): they
 *     share the context's plan buffers and split-K workspace.
 *   - Every entry point returns a cf_status; nothing throws.  Argument errors are detected on the
 *     host BEFORE anything is enqueued.  There is no CPU fallback and no other backend: on a
 *     device that is not compute capability 10.x cf_create returns CF_ERR_ARCH.
 */
#ifndef CROSSFLOW_ATTN_H
#define CROSSFLOW_ATTN_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct cf_ctx cf_ctx; /* opaque; one per device; owns plan staging and split-K workspace */
typedef struct cf_plan cf_plan; /* opaque; a device-resident plan for one set of sequence lengths */

typedef enum {
    CF_OK = 0,
    CF_ERR_INVALID_ARG = 1,  /* null pointer, negative size, query_len > context_len, ... */
    CF_ERR_UNSUPPORTED = 2,  /* head_dim / block_size / group size / stride outside the supported set */
    CF_ERR_OUT_OF_RANGE = 3, /* context_len exceeds max_blocks_per_seq * block_size */
    CF_ERR_WORKSPACE = 4,    /* fixed-size workspace too small for this batch */
    CF_ERR_CUDA = 5,         /* a CUDA runtime call or launch failed */
    CF_ERR_TIMEOUT = 6,      /* a bounded device-side wait expired (reported by cf_get_async_status) */
    CF_ERR_ARCH = 7,         /* device is not sm_100 */
    CF_ERR_BUSY = 8          /* cf_destroy while plans of the context are still alive */
} cf_status;

/* Geometry of the paged cache.  Strides are in ELEMENTS (bf16); head_dim is contiguous.
 * The recommended layout is [num_blocks, num_kv_heads, block_size, head_dim]
 * (stride_block = Hkv*B*D, stride_head = B*D, stride_token = D); [num_blocks, block_size,
 * num_kv_heads, head_dim] is accepted too.  Strides must be multiples of 8 elements (16 bytes).
 * Supported: head_dim 64 or 128; block_size 16; group size (Hq/Hkv) 1, 2, 4 or 8. */
typedef struct {
    int32_t num_q_heads, num_kv_heads, head_dim, block_size, num_blocks;
    int64_t k_stride_block, k_stride_head, k_stride_token;
    int64_t v_stride_block, v_stride_head, v_stride_token;
    float softmax_scale; /* 0 -> 1/sqrt(head_dim) */
    /* Model-specific attention variant (Section 6.1 evaluates GPT-OSS-120B, whose layers alternate full and
     * sliding-window attention and carry a learned sink logit per head; the paper itself does not describe it).
     *   window_size W > 0: the query at position p sees keys j in [max(0, p - W + 1), p]; 0: every key up to p.
     *     Block-table entries of pages that lie entirely left of every query's window are never read, so an
     *     engine may have released those pages.
     *   sink_logits: DEVICE fp32 [num_q_heads] or NULL.  The logit of head h (natural-log units, NOT multiplied
     *     by softmax_scale) joins the softmax denominator and carries no value:
     *       out = sum_j exp(x_j) v_j / (exp(sink_h) + sum_j exp(x_j)),  lse = ln(exp(sink_h) + sum_j exp(x_j)). */
    int32_t window_size;
    const float* sink_logits;
    /* Precision of the cache (the paper does not state the KV precision of its runs, Section 6.1).
     *   kv_dtype = CF_KV_BF16 (0): the pools hold bf16.
     *   kv_dtype = CF_KV_FP8_E4M3 (1): the pools hold e4m3 codes (one byte per element; strides in elements are then
     *     strides in bytes and must be multiples of 16; head_dim must be 128) with one fp32 scale per KV head:
     *     a cached value reads as e4m3(code) * k_scale[g] (v_scale[g]).  cf_kv_append stores
     *     e4m3_rne_sat((float)x / scale[g]) (IEEE fp32 division, nearest-even, saturating at +-448).  Halves the bytes
     *     decode has to stream.  k_scale, v_scale: DEVICE fp32 [num_kv_heads].  Attention reads the codes exactly
     *     (e4m3 -> fp16 / bf16 is exact) and applies the scales in fp32; prefill chunks first expand the pages they
     *     need into a bf16 staging area inside the workspace.  Not available through cf_decode_attention_static. */
    int32_t kv_dtype;
    const float* k_scale;
    const float* v_scale;
} cf_cache_desc;
enum { CF_KV_BF16 = 0, CF_KV_FP8_E4M3 = 1 };

/* Create a context on `device`.  workspace_bytes = 0: the split-K workspace starts at a default
 * size and grows when a batch needs more (growth allocates and synchronises the device);
 * workspace_bytes > 0: fixed size, a batch that needs more gets CF_ERR_WORKSPACE. */
cf_status cf_create(cf_ctx** out, int device, size_t workspace_bytes);
/* Synchronises the device and frees everything the context owns.  A context that still has live plans
 * (cf_plan_create without cf_plan_destroy) is not destroyed: CF_ERR_BUSY, nothing freed. */
cf_status cf_destroy(cf_ctx* ctx);

/* Section 2.1: prefill "materializes" the KV cache; decode appends one token per step.
 * Copies row r of k_new / v_new (sequence s, new token i) to position P+i of sequence s:
 * page block_table[s][(P+i)/B], slot (P+i)%B, P = context_len[s]-query_len[s].  Bit-exact byte move.
 *   k_cache, v_cache : DEVICE, bf16 pools described by desc (written)
 *   k_new, v_new     : DEVICE, bf16 [T, Hkv, D] contiguous, T = sum(query_len)
 *   block_table      : DEVICE, int32 [num_seqs, max_blocks_per_seq]
 *   context_len, query_len : HOST, int32 [num_seqs]
 *   cuda_stream      : a cudaStream_t (NULL = default stream).  Asynchronous. */
cf_status cf_kv_append(cf_ctx* ctx, const cf_cache_desc* desc, void* k_cache, void* v_cache,
                       const void* k_new, const void* v_new,
                       const int32_t* block_table, int32_t max_blocks_per_seq,
                       const int32_t* context_len, const int32_t* query_len,
                       int32_t num_seqs, void* cuda_stream);

/* Section 5 (mixed prefill/decode batch) + Section 4.4 (one bounded unit): attention of every new
 * token over its sequence's cached prefix and the new tokens up to itself.  Call after
 * cf_kv_append with the same length arrays.  Launch sequence on the one stream: plan upload ->
 * split-K decode -> combine -> chunked prefill (decode first, as decode latency is the protected
 * quantity).  Decode and prefill write disjoint rows of `out`.
 *   q    : DEVICE, bf16 [T, Hq, D] contiguous
 *   out  : DEVICE, bf16 [T, Hq, D] contiguous (written)
 *   lse  : DEVICE, fp32 [T, Hq] natural-log sum-exp of the scaled scores, or NULL
 *   other arguments as in cf_kv_append (caches are read-only here).  Asynchronous. */
cf_status cf_mixed_attention(cf_ctx* ctx, const cf_cache_desc* desc, const void* q,
                             const void* k_cache, const void* v_cache,
                             const int32_t* block_table, int32_t max_blocks_per_seq,
                             const int32_t* context_len, const int32_t* query_len, int32_t num_seqs,
                             void* out, float* lse, void* cuda_stream);

/* The same with a description of shared prefixes (Section 4.4: a radix-cache lookup tells how much of a prompt
 * is already resident; Section 2.1: agent turns and sub-agents share long prefixes).  Sequences with the same
 * share_group[s] >= 0 promise that their block-table rows are identical for the first shared_len[s] tokens (the
 * same physical pages); share_group[s] < 0: shares nothing.  The result is what cf_mixed_attention gives for the
 * same arguments - aliased block tables define it - but the decode sequences of a group (two or more, full
 * attention, at least 256 common tokens) read the common pages once per KV chunk for a whole set of members
 * instead of once each; each member's own suffix is read as usual and merged with it.  Prefill chunks and
 * sliding-window layers are served as by cf_mixed_attention.  share_group, shared_len: HOST int32 [num_seqs],
 * both or neither (neither: exactly cf_mixed_attention).  If the promise does not hold the affected rows are
 * meaningless, but nothing is read outside the pages the tables name. */
cf_status cf_mixed_attention_shared(cf_ctx* ctx, const cf_cache_desc* desc, const void* q,
                                    const void* k_cache, const void* v_cache,
                                    const int32_t* block_table, int32_t max_blocks_per_seq,
                                    const int32_t* context_len, const int32_t* query_len,
                                    const int32_t* share_group, const int32_t* shared_len, int32_t num_seqs,
                                    void* out, float* lse, void* cuda_stream);

/* Plan once, launch many times.  The lengths of a scheduler iteration are the same for every layer
 * of the model (Section 5: one mixed batch per iteration), so the host planning and the plan upload can
 * be done once: cf_plan_create validates, plans and uploads (it allocates the plan's own device buffers
 * and split-K partials, and enqueues one copy on cuda_stream); cf_kv_append_planned and
 * cf_mixed_attention_planned then only enqueue kernels - no allocation, no host synchronisation, no
 * host-side copy - with the same results as cf_kv_append / cf_mixed_attention.  That also makes the
 * two planned calls legal inside a CUDA stream capture (the pointers passed are baked into the graph;
 * the overlap variant and per-kernel timing do not apply to them when captured).  A plan must outlive
 * every launch and every graph that uses it; cf_plan_destroy synchronises the device.  Planned calls
 * on one context share its error word and must be ordered like all other calls. */
cf_status cf_plan_create(cf_ctx* ctx, const cf_cache_desc* desc, const int32_t* context_len, const int32_t* query_len,
                         int32_t num_seqs, int32_t max_blocks_per_seq, void* cuda_stream, cf_plan** out);
cf_status cf_plan_destroy(cf_plan* plan);
cf_status cf_kv_append_planned(cf_plan* plan, void* k_cache, void* v_cache, const void* k_new, const void* v_new,
                               const int32_t* block_table, void* cuda_stream);
cf_status cf_mixed_attention_planned(cf_plan* plan, const void* q, const void* k_cache, const void* v_cache,
                                     const int32_t* block_table, void* out, float* lse, void* cuda_stream);

/* One whole unit from HOST buffers (how a serving loop that keeps activations on the host would
 * drive the library): copies q, k_new, v_new (HOST, pinned memory recommended) to context-owned
 * device staging, runs cf_kv_append + cf_mixed_attention on cuda_stream, and copies `out` back to
 * out_host.  The caches and the block table stay DEVICE pointers (they are the node's resident
 * state).  The input copy and the read-back run on two context-owned copy streams, ordered against
 * the kernels by events and triple-buffered, so that consecutive calls overlap step i+1's input copy
 * and step i-1's read-back with step i's kernels.  Asynchronous.  out_host of every call issued so far
 * is valid once cf_host_steps_flush(ctx, stream) has been called and `stream` synchronised; the host
 * input buffers of a call must stay unchanged until then as well. */
cf_status cf_mixed_step_host(cf_ctx* ctx, const cf_cache_desc* desc,
                             const void* q_host, const void* k_new_host, const void* v_new_host,
                             void* k_cache, void* v_cache,
                             const int32_t* block_table, int32_t max_blocks_per_seq,
                             const int32_t* context_len, const int32_t* query_len, int32_t num_seqs,
                             void* out_host, void* cuda_stream);
/* Makes cuda_stream wait for the read-backs of all cf_mixed_step_host calls issued so far. */
cf_status cf_host_steps_flush(cf_ctx* ctx, void* cuda_stream);

/* After the caller has synchronised the stream: CF_OK, or what the kernels found since the last query
 * (CF_ERR_TIMEOUT: a bounded wait inside a kernel gave up and the kernel returned normally;
 * CF_ERR_OUT_OF_RANGE: a block-table entry in use was outside the pool and was not dereferenced;
 * a timeout is reported first when both happened).  Reading clears the record. */
cf_status cf_get_async_status(cf_ctx* ctx);

/* Section 5 names two executor backends: the chunked mixed-batch path (time-multiplexed) and a spatial
 * partition of the node between prefill and decode.  Both are launch sequences of cf_mixed_attention; a
 * batch that holds both kinds of work runs the spatial one unless it is switched off.  The same plan gives the
 * same bits in either sequence (planned calls); an unplanned call plans for the sequence it will run (the
 * spatial one balances the prefill items over its first grid's SMs and may cut other items into KV ranges), so
 * across sequences unplanned results agree to rounding.
 *   cf_set_overlap(ctx, 0): serial sequence, decode -> (combine) -> prefill -> (prefill combine) on the
 *     caller's stream alone.
 *   cf_set_overlap(ctx, n), n > 0 (the initial state is n = 1): n persistent prefill CTAs, one per SM (n = 1:
 *     the library's default share of the SMs, cf_spatial_share), are enqueued first, on the caller's stream; a context-owned
 *     side stream, forked from the caller's, runs decode on the SMs left over as soon as those CTAs hold their
 *     SMs (it waits for their count with a stream memory operation), and behind it a second prefill
 *     grid that draws from the same work queue, so the SMs decode frees join the prefill.  The side stream is
 *     joined back into the caller's stream inside the call, so the caller still sees one stream.
 * Environment at cf_create: CF_OVERLAP=0 (serial), CF_SPATIAL_SMS=n (the share that n = 1 stands for).
 * cf_set_timing and cf_mixed_step_host use the serial sequence. */
cf_status cf_set_overlap(cf_ctx* ctx, int n);

/* The library's default share (host only, no GPU needed): how many of num_sms SMs (0 = 148) the first prefill grid
 * of the spatial sequence takes for these lengths; 0 when the batch has no decode or no prefill part.  Decode is
 * left the SMs it needs to be done by the time the prefill is - it saturates HBM from about 65 SMs (about 100 with
 * eight query heads per KV head) and needs that many times (its own time / the call's time) - and the share is kept
 * within [3/5, 7/8] of the SMs.  A scheduler that lends a decode node's capacity (Section 4.2) can read off it how
 * much of the node a chunk will occupy beside the running decode batch. */
int32_t cf_spatial_share(const cf_cache_desc* desc, const int32_t* context_len, const int32_t* query_len,
                         int32_t num_seqs, int32_t num_sms);

/* Debug aid (synchronous): checks every block-table entry that cf_kv_append / cf_mixed_attention would
 * dereference for these lengths (entries [0, ceil(context_len/B)) of each row) against [0, num_blocks).
 * The kernels themselves trust the table - an entry outside the pool is an out-of-bounds access on the
 * device - so a serving engine runs this in its debug builds or after a scheduler change.  Reads the
 * table only.  Returns CF_OK, or CF_ERR_OUT_OF_RANGE with the number of bad entries in *num_bad. */
cf_status cf_validate_block_table(cf_ctx* ctx, const cf_cache_desc* desc, const int32_t* block_table,
                                  int32_t max_blocks_per_seq, const int32_t* context_len, const int32_t* query_len,
                                  int32_t num_seqs, void* cuda_stream, int32_t* num_bad);

/* TEST ONLY: planner and launch-sequence switches that the test-suite uses to force paths the cost model
 * would not pick on small inputs.  Not part of the supported surface; values <= 0 restore the default.
 *   CF_DEBUG_PREFILL_SPLIT          k >= 2: cut every prefill item into k KV ranges; 1: never split
 *   CF_DEBUG_SEPARATE_COMBINE       1: merge split-K decode partials in the separate combine kernel
 *   CF_DEBUG_DECODE_WAVES           target number of decode CTA waves
 *   CF_DEBUG_DECODE_MIN_CHUNK_PAGES shortest decode chunk, in pages
 *   CF_DEBUG_SPATIAL_NO_WAIT        1: in the spatial sequence decode does not wait (through a stream memory
 *                                   operation) until the first prefill grid's CTAs hold their SMs, but relies on
 *                                   the order of the launches
 *   CF_DEBUG_PREFILL_PAIRS          1: chunked prefill on pairs of SMs (tcgen05.mma.cta_group::2: two CTAs work on four
 *                                   heads of a group and share every K/V tile) where head_dim is 128 and the group
 *                                   size 4 or 8; correct and tested, but measured ~20 % slower than the default
 *                                   one-CTA-per-item kernel */
typedef enum {
    CF_DEBUG_PREFILL_SPLIT = 0,
    CF_DEBUG_SEPARATE_COMBINE = 1,
    CF_DEBUG_DECODE_WAVES = 2,
    CF_DEBUG_DECODE_MIN_CHUNK_PAGES = 3,
    CF_DEBUG_SPATIAL_NO_WAIT = 4,
    CF_DEBUG_PREFILL_PAIRS = 5
} cf_debug_option;
cf_status cf_set_debug_option(cf_ctx* ctx, cf_debug_option option, int value);

/* Self-test of the bounded-wait machinery (no counterpart in the paper): enqueues one tiny kernel whose
 * wait on a barrier that nothing signals expires after a few milliseconds; the kernel then sets the
 * context's error word and returns normally.  After synchronising, cf_get_async_status must report
 * CF_ERR_TIMEOUT once and CF_OK afterwards; the context stays usable. */
cf_status cf_selftest_bounded_wait(cf_ctx* ctx, void* cuda_stream);

/* Per-kernel timing for benchmarks.  After cf_set_timing(ctx, 1) every cf_mixed_attention records
 * CUDA events around its kernels on the caller's stream (no host synchronisation).
 * cf_get_timing_sums waits for the last timed call, returns the summed milliseconds of each
 * kernel over all calls timed since the previous cf_get_timing_sums / cf_set_timing (0 for a
 * kernel that never ran) and the number of calls, and resets the sums. */
cf_status cf_set_timing(cf_ctx* ctx, int enabled);
cf_status cf_get_timing_sums(cf_ctx* ctx, float* ms_decode, float* ms_combine, float* ms_prefill,
                             int32_t* num_calls);
/* Host time (microseconds, wall clock) spent inside cf_kv_append and cf_mixed_attention since the previous
 * query, summed over the calls, the part of it spent in the planner, and the number of cf_mixed_attention
 * calls; resets the sums.  What the caller's thread pays per unit: validation, planning, plan upload,
 * tensor-map lookup and the launches themselves (the GPU work is asynchronous). */
cf_status cf_get_host_time_sums(cf_ctx* ctx, double* us_append, double* us_attention, double* us_planner,
                                int32_t* num_steps);
/* Item counts of the plan the last cf_mixed_attention(_shared) built, for tests and reports: counts[8] =
 * {decode items, split decode sequences, prefill CTAs, decode partial slots, KV-split prefill items,
 *  shared-prefix items, members of shared-prefix sets, 1 if the prefill items are pair items (two CTAs each)}. */
cf_status cf_get_last_plan_counts(cf_ctx* ctx, int32_t* counts);
/* Number of kernels the last cf_mixed_attention launched. */
cf_status cf_get_last_launch_count(cf_ctx* ctx, int32_t* num_launches);

/* Decode attention that allocates nothing (the paper has no counterpart; this serves callers that
 * must not allocate).  Some integrators cannot call cudaMalloc where they need attention: a plugin
 * that is handed only its input and output buffers, a process whose whole GPU is owned by another
 * framework's caching allocator, a latency-critical loop that must stay off the driver's allocator
 * lock.  This entry point needs no cf_ctx: the split-K scratch (work items and fp32 partials) is a
 * fixed 16 MiB array inside the library's device image, resident on every GPU that loads the library
 * until the process exits.  It calls no cudaMalloc / cudaFree / cudaMallocHost and no allocating
 * library routine; the host plan lives on the caller's stack (about 124 KB: mind small thread stacks).
 *   Every sequence decodes exactly one token: q / out are bf16 [num_seqs, Hq, D], lse fp32
 *   [num_seqs, Hq] or NULL, context_len HOST int32 [num_seqs] (>= 1, includes the new token);
 *   caches, block_table and desc as in cf_mixed_attention.  Runs on the CURRENT device.
 *   Limits: num_seqs <= 1024, <= 3584 KV chunks, and partials (chunks of split sequences x Hq x
 *   (D+2) x 4 bytes) + 128 KiB <= 16 MiB; anything larger returns CF_ERR_WORKSPACE and enqueues nothing.
 *   The first call on a device resolves the array's address (host threads may race to it: it is
 *   serialised inside).  The call must NOT be made while cuda_stream is being captured into a graph -
 *   its plan is copied from the caller's stack, which a replay would read after it is gone - and
 *   returns CF_ERR_UNSUPPORTED then.  All calls share the one array and it keeps the previous call's
 *   contents (nothing in it has to start at zero: every partial that is read is written first by the
 *   same call), so two calls whose GPU work overlaps - different streams, or different host threads -
 *   race; keep them on one stream or order them yourself.  The sequences are cut into KV chunks by the
 *   routine cf_mixed_attention uses and merged in the same order, so on an all-decode batch the two
 *   give identical bits (for a context with default planner settings). */
cf_status cf_decode_attention_static(const cf_cache_desc* desc, const void* q,
                                     const void* k_cache, const void* v_cache,
                                     const int32_t* block_table, int32_t max_blocks_per_seq,
                                     const int32_t* context_len, int32_t num_seqs,
                                     void* out, float* lse, void* cuda_stream);

/* Section 4.2: a decode node publishes a lease whose compute credit is counted in token chunks, derived
 * from its latency headroom.  cf_estimate_us predicts, on the host and without a GPU, the device time
 * (microseconds) of the decode, combine and prefill kernels that cf_mixed_attention would launch for
 * these lengths on a B200 with num_sms SMs (0 = 148), from a model fitted to this library's measured
 * times: a scheduler can size the next prefill chunk so that the iteration stays inside its ITL budget.
 * Accuracy on the five workload configurations: within about 15 %.  Any output pointer may be NULL. */
cf_status cf_estimate_us(const cf_cache_desc* desc, const int32_t* context_len, const int32_t* query_len,
                         int32_t num_seqs, int32_t max_blocks_per_seq, int32_t num_sms,
                         float* us_decode, float* us_combine, float* us_prefill);

/* Host planner, exposed for inspection and tests (no GPU needed).  Builds the plan that
 * cf_mixed_attention would build and copies out up to `cap` items of each kind.
 *   opts          : planner settings, or NULL for the defaults of a 148-SM device.  Zero fields mean
 *                   "default"; prefill_sms_mixed > 0 plans a mixed batch for the spatial sequence with
 *                   that many SMs in the first prefill grid; prefill_force_split as CF_DEBUG_PREFILL_SPLIT;
 *                   prefill_pairs as CF_DEBUG_PREFILL_PAIRS.
 *   decode_items  : int32 [cap, 6] = {seq, q_row, kv_begin, kv_end, partial_slot (-1 = writes out directly), chunk_index}
 *   combine_items : int32 [cap, 3] = {q_row, first_partial_slot, num_chunks}
 *   prefill_items : int32 [cap, 8] = {seq, q_row_of_tile, first_row_in_chunk, num_rows, query_head, kv_head,
 *                   first_kv_tile, end_kv_tile}, one entry per (q tile, query head, KV range) in launch
 *                   order; KV tiles are 128 tokens, end_kv_tile is clamped to the tile's own extent; an item
 *                   that is not KV-split has one entry covering all of its tiles
 *   counts        : int32 [6]      = {n_decode_items, n_combine_items, n_prefill_entries, n_partial_slots,
 *                                     n_prefill_work_items (KV ranges of split items counted; an item occupies one
 *                                     SM, or a pair of SMs where pairs are used and then carries four heads),
 *                                     n_prefill_combine_items (one per KV-split item and CTA of a pair)}
 * Any output pointer may be NULL. */
typedef struct {
    int32_t num_sms, prefill_sms_mixed, prefill_force_split, decode_waves, decode_min_chunk_pages, prefill_pairs;
} cf_plan_options;
cf_status cf_plan_inspect(const cf_cache_desc* desc, const int32_t* context_len, const int32_t* query_len,
                          int32_t num_seqs, int32_t max_blocks_per_seq, const cf_plan_options* opts,
                          int32_t* decode_items, int32_t* combine_items, int32_t* prefill_items,
                          int32_t cap, int32_t* counts);

const char* cf_status_string(cf_status s);

#ifdef __cplusplus
}
#endif
#endif /* CROSSFLOW_ATTN_H */
