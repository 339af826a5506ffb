/*
 * trimkv.h -- C ABI of the B200 (sm_100a) decode hot path of global retention-based
 * KV-cache eviction ("Make Each Token Count", DBTrimKV).
 *
 * One handle owns a budgeted, paged KV cache for a fixed batch of independent
 * sequences.  Per decode step the caller appends the new token's K/V (with its
 * retention, produced by the library's gate kernel or supplied), runs attention over
 * the ragged per-(layer, KV-head) pools, and calls score_and_evict, which re-scores
 * every cached entry, keeps the budget's worth of best entries across ALL layers and
 * heads of a sequence and compacts the pools.
 *
 * Conventions
 *   - "device" pointers are CUDA device memory on the current device; "host" pointers
 *     are ordinary host memory.  All tensors are row-major and contiguous.
 *   - The caller owns every buffer it passes; the library copies what it keeps and
 *     holds no caller pointer after the stream work of the call has run.
 *   - Calls that take `stream` (a cudaStream_t passed as void*, NULL = default stream)
 *     only enqueue work.  Argument and state errors are returned at once; errors found
 *     by kernels (non-finite retention, page pool exhausted, a bounded wait that gave
 *     up) are latched in a device error word and reported by trimkv_sync_status and
 *     by the trimkv_get_* calls, which synchronise.
 *   - No exceptions, no abort, no device trap.  There is no CPU fallback.
 *   - Every sequence of the batch advances in lock step: each append adds the same
 *     number of tokens to every sequence.
 *   - Positions are 1-based token indices i per sequence, as in the paper (C_t = {1..t}).
 *   - Not thread-safe per handle; handles are independent.
 */
#ifndef TRIMKV_H_
#define TRIMKV_H_

#include <stddef.h>
#include <stdint.h>

#if defined(__GNUC__)
#define TRIMKV_API __attribute__((visibility("default")))
#else
#define TRIMKV_API
#endif

#ifdef __cplusplus
extern "C" {
#endif

typedef struct trimkv trimkv_t; /* opaque; owns all device memory it allocates */

typedef enum trimkv_status {
    TRIMKV_OK = 0,
    TRIMKV_E_ARG = 1,         /* bad argument (NULL, out of range, misaligned)              */
    TRIMKV_E_STATE = 2,       /* call order violated (e.g. layers hold different token counts) */
    TRIMKV_E_NOMEM = 3,       /* device allocation failed or page pool exhausted             */
    TRIMKV_E_CUDA = 4,        /* a CUDA runtime call failed                                   */
    TRIMKV_E_NONFINITE = 5,   /* NaN retention value met by a kernel                          */
    TRIMKV_E_TIMEOUT = 6,     /* a bounded device-side wait gave up                           */
    TRIMKV_E_UNSUPPORTED = 7  /* shape outside what the kernels handle                        */
} trimkv_status;

#define TRIMKV_DTYPE_BF16 0
#define TRIMKV_DTYPE_F32 1

typedef struct trimkv_config {
    int64_t budget_entries; /* M_global per sequence, in entries = tokens' worth x layers x kv_heads
                               (Sec. 5.2 "global budget of M x #layers x #heads")               */
    int32_t layers;         /* L                                                               */
    int32_t kv_heads;       /* H                                                               */
    int32_t q_heads;        /* Hq, a multiple of H (GQA group g = Hq / H)                      */
    int32_t head_dim;       /* d, a multiple of 8                                              */
    int32_t hidden;         /* D, gate input width; 0 = no gate (retention must be supplied)   */
    int32_t max_batch;      /* B, sequences held by the handle; every call covers all of them  */
    int32_t page_size;      /* entries per page; must be 64                                    */
    int32_t gate_hidden;    /* d_g, hidden width of Proj (Sec. 5.1: 512)                       */
    int32_t gate_embed;     /* d_e, output width of Proj, input of the shared readout          */
    int32_t horizon;        /* lookahead T - t (Sec. 5.1: 2); 0 = infinite horizon             */
    int32_t kv_dtype;       /* TRIMKV_DTYPE_BF16 or TRIMKV_DTYPE_F32 (K, V, q and out)         */
    int32_t max_chunk;      /* largest n_new of one append (1 for pure decode)                 */
    int32_t reserved;       /* must be 0                                                       */
    int64_t max_pool_pages; /* cap on pages of one (layer, head) pool; 0 = a pool may take all */
    int32_t retention_bias; /* 0: decode attention is the plain softmax over the retained set (Eq. (1));
                               1: retention-gated weights beta_i^(t-i) e^{z_i} of Sec. 2.2 (t = tokens seen) */
    int32_t per_pool_budget; /* 0: one global budget per sequence (the paper's method).  > 0: the fixed-budget variant it is
                               compared with (TrimKV): every (layer, head) pool keeps its own per_pool_budget best
                               entries; budget_entries (>= per_pool_budget x layers x kv_heads) then only sizes the cache */
    int32_t shard_total_layers; /* 0: the handle holds whole sequences.  > 0: it holds `layers` consecutive layers, starting
                               at shard_layer0, of sequences whose shard_total_layers layers are spread over several
                               handles (ranks) that share ONE global budget (see the trimkv_shard_* calls).
                               budget_entries is then this handle's CAPACITY: the most entries per sequence its layers
                               may keep after an eviction round                                                      */
    int32_t shard_layer0;   /* first layer of the slice (layer arguments of the other calls stay local: 0 .. layers-1) */
} trimkv_config;

/* Fill *cfg with defaults (batch 1, q_heads = kv_heads, bf16, no gate, page 64, d_g 512,
 * d_e 64, horizon 2, max_chunk 512) for the given budget and shape. */
TRIMKV_API void trimkv_default_config(trimkv_config* cfg, int64_t budget_entries, int layers, int kv_heads, int head_dim);

/* Budgeted cache (Sec. 2.1, Eq. (2): at most M retained entries) with default
 * configuration.  Returns NULL on failure (see trimkv_last_error). */
TRIMKV_API trimkv_t* trimkv_create(int64_t budget_entries, int layers, int kv_heads, int head_dim);

/* Same with explicit configuration.  *out receives the handle. */
TRIMKV_API trimkv_status trimkv_create_ex(const trimkv_config* cfg, trimkv_t** out);

/* Frees everything the handle owns.  NULL is allowed. */
TRIMKV_API void trimkv_destroy(trimkv_t* h);

/* Empties the cache (all pools, token counters) but keeps gate weights.  Synchronises. */
TRIMKV_API trimkv_status trimkv_reset(trimkv_t* h);

/* Gate parameters of one layer (Sec. 4.1, Sec. 5.1): Proj_{l,h}(x) = W2[h] act(W1 x + b1) + b2[h],
 * act = SiLU.  Device pointers, fp32: W1 [d_g, D], b1 [d_g], W2 [H, d_e, d_g], b2 [H, d_e].
 * Copied; synchronises. */
TRIMKV_API trimkv_status trimkv_set_gate(trimkv_t* h, int layer, const float* W1, const float* b1, const float* W2,
                              const float* b2);

/* The readout shared by every layer and head (Sec. 4.1: (w_g, b_g) tied): device w_g [d_e], scalar b_g. */
TRIMKV_API trimkv_status trimkv_set_shared_projection(trimkv_t* h, const float* w_g, float b_g);

/* Retention gate alone (Sec. 4.1): for x [B, n_new, D] fp32 (device) compute, per row and KV head,
 *   s = w_g . Proj_{layer,h}(x) + b_g,  beta = sigmoid(s),  lambda = ln beta,
 *   c = ln sum_{k<horizon} beta^k   (the beta-only factor of Eq. (global_score)).
 * Any of beta/lambda/c (device, fp32 [B, n_new, H]) may be NULL.  Changes no cache state. */
TRIMKV_API trimkv_status trimkv_gate(trimkv_t* h, int layer, int n_new, const float* x, float* beta, float* lambda, float* c,
                          void* stream);

/* Append n_new tokens to every pool of `layer` (a token's retention is estimated once, when it
 * enters the cache, Sec. 3.2).  k, v: device [B, n_new, H, d] in kv_dtype.
 * Retention: x != NULL -> gate on x [B, n_new, D] fp32; else lambda [B, n_new, H] fp32 (<= 0) is
 * required and c [B, n_new, H] is optional (NULL -> derived from lambda on the device in fp32).
 * Token j of the call gets position tokens(layer) + j + 1.  n_new <= max_chunk.
 * Capacity rule: the cache has room for the budget plus ONE chunk of max_chunk tokens per layer, so an eviction round
 * (trimkv_score_and_evict) must run before a sequence would hold more than budget_entries + max_chunk * layers *
 * kv_heads entries (per_pool_budget > 0: per_pool_budget * layers * kv_heads in place of budget_entries).  An append
 * that would exceed this is refused with TRIMKV_E_STATE and changes nothing. */
TRIMKV_API trimkv_status trimkv_append(trimkv_t* h, int layer, int n_new, const float* x, const float* lambda, const float* c,
                            const void* k, const void* v, void* stream);

/* One eviction round at time t = tokens appended so far (Sec. 4.2): for every sequence, score
 * every entry, S = (t + 1 - i) * lambda + c in fp32 (log of Eq. (global_score)), keep the
 * budget_entries highest over all layers and heads (ties: older position, then lower layer, then
 * lower head are kept), drop the rest and compact the pools.  No-op while within budget.
 * TRIMKV_E_STATE unless every layer holds the same number of tokens. */
TRIMKV_API trimkv_status trimkv_score_and_evict(trimkv_t* h, void* stream);

/* Decode attention of one layer over the retained entries (Sec. 2.1 / Eq. (1) with r in {0,1}):
 * q, out: device [B, Hq, d] in kv_dtype; query head j reads the pool of KV head j / g; softmax
 * scale 1/sqrt(d); an empty pool gives zeros. */
TRIMKV_API trimkv_status trimkv_decode_attention(trimkv_t* h, int layer, const void* q, void* out, void* stream);

/* Causal attention of a prompt chunk (Sec. 2.1, restricted to the retained set as in Eq. (1)): call it after
 * trimkv_append(layer, n_new, ...) of the chunk and before the eviction round.  q, out: device [B, n_new, Hq, d] in
 * kv_dtype; token j of the chunk attends to every entry kept from before the chunk and to the chunk's tokens 0..j.
 * TRIMKV_E_UNSUPPORTED with retention_bias set. */
TRIMKV_API trimkv_status trimkv_prefill_attention(trimkv_t* h, int layer, int n_new, const void* q, void* out, void* stream);

/* One whole decode step for all layers at once (the benchmark path): gate on x [L, B, D] fp32
 * (or lambda [L, B, H] if x == NULL), append k, v [L, B, H, d], attention of q [L, B, Hq, d] into
 * out [L, B, Hq, d], then score_and_evict. */
TRIMKV_API trimkv_status trimkv_decode_step_all(trimkv_t* h, const float* x, const float* lambda, const void* k, const void* v,
                                     const void* q, void* out, void* stream);

/* The same step for callers whose per-token tensors live in HOST memory (same shapes).  x (or lambda) is copied to a
 * staging buffer of the handle beside the attention kernel, ahead of the gate.  K, V, q and the output are each touched
 * once by one kernel.  A q_host or out_host in pinned memory the device can address (cudaHostAlloc, cudaHostRegister,
 * torch's pin_memory) is read or written in place across the bus by the attention kernel, and no copy is queued for it;
 * so are a pinned k_host and v_host by the append, while they are under 512 KB together (larger ones travel faster by
 * copy engine).  Buffers in any other memory (pageable, or pinned but not 16-byte aligned) go through staging buffers:
 * K, V, q copied ahead of the append, the output copied back at the end of the step; the results are the same either way.  Everything is ordered after earlier work of `stream` and complete, for
 * `stream`, when the call's work is.  The host buffers must stay untouched until then. */
TRIMKV_API trimkv_status trimkv_decode_step_all_host(trimkv_t* h, const float* x_host, const float* lambda_host,
                                          const void* k_host, const void* v_host, const void* q_host, void* out_host,
                                          void* stream);

/* trimkv_decode_step_all runs on two internal streams by default: K/V append, attention and compaction on one, the
 * gate and the selection beside them on the other (attention never reads retention terms, the selection never reads
 * K/V); both are forked from and joined back to the caller's stream.  enable = 0 runs every phase back to back on the
 * caller's stream instead (same results; for per-kernel timing).  Synchronises. */
TRIMKV_API trimkv_status trimkv_set_overlap(trimkv_t* h, int enable);

/* The handle's own highest-priority stream (a cudaStream_t), on which trimkv_decode_step_all runs its K/V append, attention
 * and compaction.  A caller that passes this stream -- or any stream of its own created with the device's highest
 * priority -- as `stream` saves the step the two hand-offs between the caller's stream and that one (a few microseconds
 * each, on the critical path of short steps).  Owned by the handle; do not destroy it. */
TRIMKV_API void* trimkv_step_stream(trimkv_t* h);

/* Changes the horizon h = T - t of the retention score (Sec. 4.2, Eq. (global_score): ln G~ = (t+1-i) ln beta +
 * ln sum_{k<h} beta^k; h = 1 gives the myopic score beta^(t+1-i), h = 0 stands for h -> infinity, the limit
 * beta^(t+1-i) / (1 - beta) stated below the equation) for an existing cache, e.g. between eviction rounds: the
 * beta-only term c of EVERY stored entry is recomputed on the device from its stored lambda = ln beta (fp32, the same
 * routine that appends use), and later appends use the new horizon.  Entries, K/V and lambda are untouched; the next
 * selection ranks by the new score.  horizon in [0, 64], else TRIMKV_E_ARG.  Asynchronous on `stream`, ordered like
 * trimkv_score_and_evict (the caller orders it against decode steps on other streams). */
TRIMKV_API trimkv_status trimkv_set_horizon(trimkv_t* h, int horizon, void* stream);

/* Pool lengths to host memory, int32 [B, L, H].  Synchronises; reports latched device errors. */
TRIMKV_API trimkv_status trimkv_get_lengths(trimkv_t* h, int32_t* out_host);

/* Positions kept in pool (seq, layer, head), ascending, to host pos_out[0..cap); *n = pool length
 * (also when it exceeds cap, in which case TRIMKV_E_ARG is returned).  Synchronises. */
TRIMKV_API trimkv_status trimkv_get_kept(trimkv_t* h, int seq, int layer, int head, int32_t* pos_out_host, int cap, int* n);

/* Entries of pool (seq, layer, head) in storage order to host arrays (each may be NULL):
 * pos int32 [n], lambda/c fp32 [n], k/v [n, d] in kv_dtype.  *n as above.  Synchronises. */
TRIMKV_API trimkv_status trimkv_get_pool(trimkv_t* h, int seq, int layer, int head, int cap, int* n, int32_t* pos_host,
                              float* lambda_host, float* c_host, void* k_host, void* v_host);

/* Checkpoint / resume.  The cache IS the method's whole state (which entries survive, with their retention terms), so a
 * snapshot is every pool read back with trimkv_get_pool plus the token count.  To resume: create a handle with the same
 * shape, set the gate weights, call trimkv_import_pool for every non-empty pool (host arrays as trimkv_get_pool wrote
 * them: pos int32 [n], lambda and c fp32 [n], k and v [n, d] in kv_dtype; the pool must be empty), then
 * trimkv_import_finish(tokens) with the number of tokens the sequences had seen.  Entries keep their order, positions and
 * fp32 retention terms, so every later eviction round and attention call gives what the original cache would have given.
 * Both calls synchronise.  Errors: a pool that is not empty (TRIMKV_E_STATE), too many entries (TRIMKV_E_NOMEM), NaN
 * retention terms (TRIMKV_E_NONFINITE); import_finish requires every sequence to hold the same number of entries. */
TRIMKV_API trimkv_status trimkv_import_pool(trimkv_t* h, int seq, int layer, int head, int n, const int32_t* pos_host,
                                 const float* lambda_host, const float* c_host, const void* k_host, const void* v_host);
TRIMKV_API trimkv_status trimkv_import_finish(trimkv_t* h, int64_t tokens);

/* Per-sequence figures of the last selection, int64 [B, 4] to host:
 * {1 if the exact redo ran (the sampled candidate range missed) else 0, candidates ranked exactly,
 *  entries evicted, keys sampled}.  Synchronises. */
TRIMKV_API trimkv_status trimkv_get_select_stats(trimkv_t* h, int64_t* out_host);

/* Self-check of the cache's bookkeeping, for tests and debugging (the role a memory checker would play): every pool's
 * block table against the page records and back, the free stack against the page records, page accounting (owned + free
 * = all pages of a sequence), positions within 1..tokens and no NaN retention term among the live entries.  Synchronises,
 * allocates a few bytes of scratch, and returns TRIMKV_E_STATE with the violated rules in trimkv_last_error, else the
 * latched device status. */
TRIMKV_API trimkv_status trimkv_check_invariants(trimkv_t* h);

/* Waits for the handle's enqueued work (device synchronise) and returns the latched device error,
 * TRIMKV_OK if none.  The latch is cleared by trimkv_reset. */
TRIMKV_API trimkv_status trimkv_sync_status(trimkv_t* h);

/* Per-phase device timing (CUDA events recorded on the call's stream around each phase of append,
 * decode_attention, decode_step_all and score_and_evict).  trimkv_profile(h, 1) starts recording,
 * trimkv_profile(h, 0) stops; both synchronise and discard earlier records.  trimkv_profile_read
 * synchronises, writes to host ms[8] the summed milliseconds and to count[8] the number of recorded
 * intervals per phase {0 gate, 1 append, 2 host-to-device copies of K, V and q (host-buffer entry point), 3 attention
 * kernel, 4 device-to-host copy of the output (host-buffer entry point), 5 score+select, 6 compact, 7 host-to-device
 * copy of x or lambda (host-buffer entry point)}, and clears the records.  Phases that run on different internal
 * streams overlap in time. */
/* enable = 2 records the attention main kernel alone (two events per call: cheap enough for a timed run). */
TRIMKV_API trimkv_status trimkv_profile(trimkv_t* h, int enable);
TRIMKV_API trimkv_status trimkv_profile_read(trimkv_t* h, double* ms_host, int64_t* count_host);

/* ---- one sequence sharded by layer over several handles (ranks) ------------------------------------
 * The global eviction rule ranks the entries of ALL layers and heads of a sequence under one budget (Sec. 4.2).  When
 * the layers of a sequence live on several GPUs, each rank creates a handle for its slice (shard_total_layers > 0) and
 * uses append / decode_attention as usual; an eviction round is then run in stages, with three small exchanges between
 * them that the caller performs (an all-gather, an all-reduce, an all-gather: NCCL through torch.distributed, or any
 * other transport).  After each exchange every rank computes the same result from the same data, so all reach the same
 * threshold and each flags its own entries.  Per sequence, with W ranks and B sequences:
 *   1. trimkv_shard_sample     local key sample (Bernoulli, rate from the GLOBAL entry count) -> keys [B][cap], counts [B]
 *      exchange: all-gather keys and counts                          (cap = trimkv_shard_sample_cap() keys of 8 bytes)
 *   2. trimkv_shard_bracket    gathered samples [W][B][cap], [W][B] -> the bracket of the k-th smallest key (same on all ranks)
 *   3. trimkv_shard_filter     one pass over the local metadata: keys below the bracket are flagged and counted, keys
 *                              inside it listed -> n_below [B] (int64), cand_count [B] (int32; -1 = the local list overflowed)
 *      exchange: all-reduce (sum) n_below, all-gather cand_count, then all-gather the candidate records
 *   4. trimkv_shard_candidates local candidate records (16 bytes each: key, slot) -> [B][cand_cap_x]
 *   5. trimkv_shard_resolve    gathered records [W][B][cand_cap_x], counts [W][B], global n_below [B] -> exact threshold;
 *                              this rank's candidates up to it are flagged; resolved [B] (int32) = 0 where the bracket
 *                              missed the threshold or a list overflowed (same on every rank)
 *   6. only if some sequence is unresolved (all ranks see the same flags): exact radix select, 6 rounds of
 *      trimkv_shard_hist (local digit histogram [B][2048], uint32) -> exchange: all-reduce (sum) -> trimkv_shard_digit
 *      (prefix [B] uint64 and rank [B] int64 move one digit down; start: prefix 0, rank k_evict, top 64, then
 *      top = 53, 42, 31, 20, 9), then trimkv_shard_mark with tau = prefix
 *   7. trimkv_shard_compact    compaction of the local pools; returns this rank's entries per sequence (synchronises)
 * t, n_total and k_evict are GLOBAL: tokens seen, entries of one sequence over all ranks, entries to evict.  All
 * pointers are device memory unless the name says host; calls are asynchronous on `stream` except the last one. */
TRIMKV_API int32_t trimkv_shard_sample_cap(void);
TRIMKV_API trimkv_status trimkv_shard_sample(trimkv_t* h, int64_t n_total, int64_t k_evict, uint64_t* keys_out, int32_t* counts_out,
                                  void* stream);
TRIMKV_API trimkv_status trimkv_shard_bracket(trimkv_t* h, int world, const uint64_t* gathered_keys, const int32_t* gathered_counts,
                                   int64_t n_total, int64_t k_evict, void* stream);
TRIMKV_API trimkv_status trimkv_shard_filter(trimkv_t* h, int64_t* n_below_out, int32_t* cand_count_out, void* stream);
TRIMKV_API trimkv_status trimkv_shard_candidates(trimkv_t* h, int64_t cap, void* cand_out, void* stream);
TRIMKV_API trimkv_status trimkv_shard_resolve(trimkv_t* h, int world, int rank, int64_t cap, const void* gathered_cand,
                                   const int32_t* gathered_counts, const int64_t* n_below_global, int64_t k_evict,
                                   int32_t* resolved_out, void* stream);
TRIMKV_API trimkv_status trimkv_shard_hist(trimkv_t* h, const uint64_t* prefix, int top, uint32_t* hist_out, void* stream);
TRIMKV_API trimkv_status trimkv_shard_digit(trimkv_t* h, const uint32_t* hist, uint64_t* prefix, int64_t* rank, int top, void* stream);
TRIMKV_API trimkv_status trimkv_shard_mark(trimkv_t* h, const uint64_t* tau, void* stream);
TRIMKV_API trimkv_status trimkv_shard_compact(trimkv_t* h, int64_t* local_entries_out_host, void* stream);

/* ---- testing aids (not part of the method) ------------------------------------------------------
 * Switches that make rarely taken paths run on demand, so that tests can reach them without a fault:
 *   TRIMKV_TEST_DISTRUST_SAMPLE      the selection ignores its key sample; the exact fallback of the selection (cache:
 *                                    the single-CTA redo; flat arrays: the histogram passes) then runs in every call.
 *                                    Results are unchanged.
 *   TRIMKV_TEST_ATTENTION_NO_COPY    the tensor-core decode attention kernel issues none of its asynchronous K/V copies
 *                                    and uses a short limit for its waits: every wait runs out, the kernel latches
 *                                    TRIMKV_E_TIMEOUT and returns with nothing in flight (its output is not written).
 * h != NULL sets the switches of that handle; h == NULL those of the handle-less calls (trimkv_select_topk and
 * trimkv_select_topk_static) for the whole process.  flags = 0 restores normal operation.  Synchronises. */
#define TRIMKV_TEST_DISTRUST_SAMPLE 1
#define TRIMKV_TEST_ATTENTION_NO_COPY 2
TRIMKV_API trimkv_status trimkv_set_test_hooks(trimkv_t* h, int flags);

/* Message of the calling thread's last failed call; never NULL. */
TRIMKV_API const char* trimkv_last_error(void);

/* Number of kernels this library has launched in the calling process so far. */
TRIMKV_API int64_t trimkv_kernel_launches(void);

/* ---- standalone global selection over a flat score array (Sec. 4.2's ranking alone) ---------
 * Keeps the k_keep largest of n fp32 scores (device); ties: lower index kept.  keep_bits: device
 * uint64 [(n + 63) / 64], bit (i % 64) of word i / 64 set iff score i is kept.  workspace: device
 * scratch of at least trimkv_select_workspace_bytes(n) bytes, 256-byte aligned, contents ignored.
 * NaN scores are not allowed (latched as TRIMKV_E_NONFINITE in the status word).
 * status_out: device int32, set to a trimkv_status by the kernels (may be NULL).
 * The scores are read once: a sampled bracket of the threshold, one pass that writes the keep bits and a short list of
 * keys near the threshold, exact ranking of that list.  If the bracket misses (about one call in 10^4) an exact
 * multi-pass fallback runs instead; the result is the same either way.  After the call, int64 workspace[64 .. 69)
 * (byte offset 512) holds counters for tests and tuning: {fallback taken: 0 none, 1 exact over the candidate list,
 * 2 exact over all scores; keys in the sampled bracket; keys ranked exactly; keys sampled; form of the streaming
 * pass's per-score tests: 2 arithmetic (no warp votes: both ends of the bracket finite, and neither its half-width
 * nor the threshold estimate under 2^-100 in magnitude), 1 one subtraction and one compare, 0 two compares (an end
 * of the bracket is open)}. */
TRIMKV_API size_t trimkv_select_workspace_bytes(int64_t n);
TRIMKV_API trimkv_status trimkv_select_topk(const float* scores, int64_t n, int64_t k_keep, uint64_t* keep_bits, void* workspace,
                                 size_t workspace_bytes, int32_t* status_out, void* stream);

/* ---- the same selection for callers that cannot allocate ------------------------------------
 * (No counterpart in the paper: this entry point exists for the sake of the caller's environment.)
 * Some users of this library run where device allocation is off limits at call time: inside a
 * serving loop whose memory was carved up at start-up, under an allocator they do not control, or in
 * a host framework that forbids cudaMalloc after initialisation.  They cannot size and provide the
 * workspace that trimkv_select_topk wants.  This variant does the identical selection (same result,
 * bit for bit) with its scratch memory in an array built into the library image, and itself calls no
 * cudaMalloc, cudaFree or any other allocating routine.  The caller still passes scores, keep_bits
 * and status_out (device memory, as for trimkv_select_topk).
 *   - Limit: n <= TRIMKV_SELECT_STATIC_MAX_N scores; a larger n is refused with
 *     TRIMKV_E_UNSUPPORTED and a message in trimkv_last_error.  The array takes about 2.4 MB of
 *     device memory on every GPU that loads the library, until the process exits.
 *   - The first call on each device looks up the array's device address (with that device current;
 *     the CUDA runtime may load the library's device code at that moment, which is the driver's
 *     business, not an allocation of this call); make that first call outside any stream capture.
 *     The address is cached per device; after a cudaDeviceReset it is looked up again.
 *   - All calls share the one array, which keeps whatever the last call left in it; each call
 *     clears, on `stream`, the part that must start at zero.  Two calls whose GPU work may overlap
 *     (different streams, or different threads or handles on one device) race on it: serialise them. */
#define TRIMKV_SELECT_STATIC_MAX_N (1 << 22)
TRIMKV_API trimkv_status trimkv_select_topk_static(const float* scores, int64_t n, int64_t k_keep, uint64_t* keep_bits,
                                        int32_t* status_out, void* stream);

#ifdef __cplusplus
}
#endif
#endif /* TRIMKV_H_ */
