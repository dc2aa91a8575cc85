/*
 * h2o.h — C ABI of the B200 (sm_100a) implementation of the H2O KV-cache
 * eviction hot path: attention over a budget-limited KV cache whose slots are
 * kept or evicted by accumulated attention score.
 *
 * Vocabulary.  A *unit* is one (sequence, head); units never interact (the
 * paper evicts per head, Appendix A).  Per sequence s the cache holds
 * B_s = k_s + r_s *slots* per head: k_s heavy hitters and the r_s most recent
 * tokens (the even split of the budget of Section 5; the heavy and recent regions
 * of Appendix A).  Slot order carries no meaning; each slot records the token
 * position it holds.
 *
 * Conventions common to every call
 *   - Returns 0 (H2O_OK) or a negative H2O_ERR_* code; nothing is printed, thrown
 *     or aborted.  Argument, size and call-order errors are found before anything is
 *     enqueued.  H2O_ERR_CUDA can come from a launch in the middle of a call that
 *     enqueues several kernels (h2o_prefill_select, h2o_decode_chunk); the cache is
 *     then partly written, every later prefill or decode call on it returns
 *     H2O_ERR_STATE, and h2o_cache_reset makes it usable again.
 *   - "dev" pointers are CUDA device pointers on the cache's device, "host"
 *     pointers are ordinary host memory.  The library never allocates or frees
 *     device memory and keeps no caller pointer after a call returns, except the
 *     workspace given to h2o_cache_create, which the caller must keep alive and
 *     untouched until h2o_cache_destroy.
 *   - Calls taking a stream are asynchronous on that stream (a cudaStream_t
 *     passed as void*; NULL is the legacy default stream).  A cache must be
 *     driven from one stream at a time.
 *   - Tensors are dense, row-major, 16-byte aligned, of the cache's dtype.
 *   - There is no CPU fallback: without a CUDA device of compute capability 10.x
 *     h2o_cache_create fails with H2O_ERR_CUDA / H2O_ERR_UNSUPPORTED.
 */
#ifndef H2O_B200_H_
#define H2O_B200_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define H2O_OK 0
#define H2O_ERR_INVALID_ARG (-1) /* NULL pointer, non-positive size, negative budget, ...      */
#define H2O_ERR_UNSUPPORTED (-2) /* dtype / head_dim / device the kernels are not written for   */
#define H2O_ERR_WORKSPACE (-3)   /* workspace or scratch too small or misaligned                */
#define H2O_ERR_STATE (-4)       /* call order violated (e.g. second prefill on one cache)      */
#define H2O_ERR_CUDA (-5)        /* a CUDA runtime call or kernel launch failed                 */
#define H2O_ERR_TIMEOUT (-6)     /* a bounded device-side wait gave up (seen by h2o_cache_status) */

/*
 * H2O_BF16_KV4: q / k / v / out are bf16 (head_dim 128 only); the stored K/V slots are 4-bit group-quantised
 * (the paper's third question, on quantisation: it names the combination, not a quantiser; this library's
 * own: groups of 32 channels, zero = group minimum, scale = bf16((max - min) / 15), code =
 * clamp(rint((x - zero) / scale), 0, 15), all in fp32; 80 bytes per row instead of 256).  A row is
 * quantised when it enters the cache: kept prompt rows at selection, a new token's row after its own
 * decode step, in which it takes part at full precision.  Prompt attention itself is unquantised.
 * h2o_decode_chunk takes one decode-step kernel per token in this format; units are not split over
 * thread-block clusters.
 */
typedef enum { H2O_F32 = 0, H2O_BF16 = 1, H2O_BF16_KV4 = 2 } h2o_dtype_t;

typedef struct h2o_cache h2o_cache_t; /* opaque, host-side */

/*
 * Problem statement (Section 2.1: Q, K in R^{n x d} and a space budget;
 * Appendix A: parameter K heavy + K recent, chosen per sequence here).
 */
typedef struct {
  int32_t batch;                /* number of sequences, >= 1                                   */
  int32_t n_heads;              /* heads per sequence, >= 1                                    */
  int32_t head_dim;             /* d: 64 or 128                                                */
  int32_t dtype;                /* h2o_dtype_t of q/k/v/out and of the stored K/V slots        */
  const int32_t* heavy_budget;  /* host [batch]: k_s >= 0                                      */
  const int32_t* recent_window; /* host [batch]: r_s >= 0, k_s + r_s >= 1                      */
  float softmax_scale;          /* c in exp(c q.k); <= 0 selects 1/sqrt(head_dim)              */
  int32_t device;               /* CUDA device ordinal                                         */
  int32_t query_group;          /* grouped-query attention: query heads per (K/V) head: 0 or 1 (none), 2, 4 or 8 */
} h2o_config_t;

/*
 * Grouped-query attention (query_group = G > 1; no counterpart in the paper, which evicts per head; its comparison
 * with a method that accumulates scores across heads is the nearest text).  n_heads counts the K/V heads: a unit is
 * one (sequence, K/V head) and its G query heads share its cache.  q and out then have n_heads * G heads, query
 * head = head * G + g ([..., n_heads * G, head_dim]); k, v, k_new, v_new and evicted_pos keep n_heads.  Every query
 * head attends the unit's entries with its own softmax, and a key's accumulated score grows by the SUM of the
 * probabilities the group's heads gave it; selection after the prompt and eviction use that sum.  Each K and V row
 * is read once for the whole group.  Supported: f32 / bf16 slots, budgets with G * (k_s + r_s + 1) * 4 bytes up to
 * about 160 KB; bf16 with head_dim 128 runs on the tensor-core prompt kernels and the streaming step kernel, the
 * rest on the fp32-FMA prompt kernels and the plain grouped step kernel; "Top-K" attention and 4-bit slots are not
 * combined with it, sparse patterns only where the streaming step kernel applies (H2O_ERR_UNSUPPORTED otherwise).
 */

/* Bytes of device workspace h2o_cache_create needs for this configuration
 * (K/V slots, accumulated scores, positions, counters).  Pure host arithmetic.
 * Returns 0 for an invalid or unsupported configuration. */
size_t h2o_cache_workspace_bytes(const h2o_config_t* cfg);

/* Bytes of device scratch one h2o_prefill_select call needs for prompts of
 * `total_tokens` tokens in all (row statistics and column sums, per head).
 * Pure host arithmetic; 0 for invalid arguments. */
size_t h2o_prefill_scratch_bytes(const h2o_config_t* cfg, int64_t total_tokens);

/*
 * Create an empty cache (every unit holds 0 tokens, next position t = 0) inside
 * the caller's device workspace (256-byte aligned, at least
 * h2o_cache_workspace_bytes(cfg) bytes).  The budget arrays are copied.  Small
 * tables are copied to the device synchronously; no kernel state survives a
 * failed create.  *out is set only on success.
 * Pre-allocated storage whose evicted entry is overwritten by the new one, without
 * moving any other row, follows Section 4.2 (implementation details) and Appendix A.
 */
int h2o_cache_create(h2o_cache_t** out, const h2o_config_t* cfg, void* dev_workspace, size_t workspace_bytes);

/*
 * Attach a handle to a workspace that ALREADY holds a cache of the same configuration —
 * a byte copy of another handle's workspace, taken while no work on it was in flight and
 * possibly restored from a file: the whole state of a cache (K/V slots, scores, positions,
 * counters) lives in its workspace, so copying the bytes is the snapshot and this call is
 * the resume.  Nothing in the workspace is modified; its unit table is compared with the
 * one `cfg` produces (H2O_ERR_STATE if they differ).  The handle accepts decode calls;
 * h2o_prefill_select is refused (H2O_ERR_STATE) until h2o_cache_reset.
 * No counterpart in the paper (its cache is transient state of one generation).
 */
int h2o_cache_attach(h2o_cache_t** out, const h2o_config_t* cfg, void* dev_workspace, size_t workspace_bytes);

/*
 * Prefill selection (Appendix A pseudocode, prefill branch: attention over the
 * whole prompt, then the heavy hitters and the most recent tokens are kept, all
 * tokens if the prompt is not longer than the budget).  For every unit:
 *   P[i][j] = softmax_j(c q_i.k_j), j <= i          causal attention, n_s rows
 *   out_i   = sum_j P[i][j] v_j
 *   acc0[j] = sum_{i >= j} P[i][j]                   accumulated score (Algorithm 2, accumulation line)
 *   keep the last r_s positions and the k_s positions of [0, n_s - r_s) with the
 *   largest acc0 (equal scores: the higher position is kept), copy their K/V rows,
 *   acc0 and position into the unit's slots; t = n_s.
 * q, k, v, out : dev [total_tokens, n_heads, head_dim], sequences concatenated
 *                token-major; out may not alias the inputs.
 * cu_seqlens   : host [batch + 1], cu[0] = 0, non-decreasing; n_s = cu[s+1]-cu[s] >= 1.
 * scratch      : dev, 256-byte aligned, >= h2o_prefill_scratch_bytes(cfg, cu[batch]);
 *                used only by the work this call enqueues.
 * Allowed once per cache and only before any decode step (H2O_ERR_STATE otherwise).
 */
int h2o_prefill_select(h2o_cache_t* cache, const void* q, const void* k, const void* v,
                       const int32_t* cu_seqlens, void* out, void* scratch, size_t scratch_bytes, void* stream);

/*
 * One decoding step for every unit, fused in one kernel (Algorithm 2 loop body
 * with the cache layout of Appendix A).  With S the unit's kept set and t its
 * next position:
 *   p      = softmax over S u {t} of c q.k_x           (the new token attends to itself)
 *   out    = sum_x p_x v_x
 *   acc_x += p_x for x in S;  acc_t = p_t
 *   if the unit already holds B_s tokens: evict the candidate (pos <= t - r_s) with
 *   the smallest acc (equal: lowest position) and store the new token in its slot;
 *   otherwise append.  With r_s = 0 the new token itself is a candidate and may be
 *   the one dropped.  t += 1.
 * q, k_new, v_new, out : dev [batch, n_heads, head_dim].
 * evicted_pos          : dev [batch, n_heads] int32 or NULL; position evicted by this
 *                        step, -1 if none.
 * May be called on a cache that was never prefilled (token-by-token mode, the
 * fill phase of Algorithm 2).
 */
int h2o_decode_step(h2o_cache_t* cache, const void* q, const void* k_new, const void* v_new, void* out,
                    int32_t* evicted_pos, void* stream);

/*
 * n_tokens consecutive decoding steps for every unit in one call: Algorithm 1 applied
 * token by token (the paper's sequential generation; with an empty cache and the prompt
 * as input it is the token-by-token eviction of Algorithm 1 over the prompt, the
 * mechanics of the streaming experiment of Section 5.3).  The result — outputs, cache
 * contents, accumulated scores, evicted positions — is that of n_tokens calls of
 * h2o_decode_step on the rows of the inputs in order.
 * q, k, v, out : dev [n_tokens, batch, n_heads, head_dim] (step-major), 16-byte aligned.
 * evicted_pos  : dev [n_tokens, batch, n_heads] int32 or NULL.
 * n_tokens     : >= 1.
 * For bf16, head_dim 128 and budgets with max_s(k_s + r_s) + 32 <= 1024 the steps run 32
 * at a time inside one kernel (scores and outputs on the tensor cores, the sequential
 * part in registers); every other configuration is served by one decode-step kernel per
 * token.  Both are asynchronous on `stream`.
 */
int h2o_decode_chunk(h2o_cache_t* cache, const void* q, const void* k, const void* v, int32_t n_tokens,
                     void* out, int32_t* evicted_pos, void* stream);

/*
 * h2o_prefill_select for callers that cannot allocate device memory (the paper has no
 * counterpart; this is a deployment convenience).  Some hosts of this library may not call
 * cudaMalloc at all: a plugin inside a serving process whose memory pool is owned by someone
 * else, a real-time loop that must not touch the allocator's lock or trigger its implicit
 * synchronisation, a runtime that hands out device memory only at start-up.  They can pass
 * the inputs and outputs they already hold, but have no buffer to offer as scratch.  This entry
 * point takes none: the scratch is a fixed array of h2o_prefill_static_scratch_bytes() bytes
 * (16 MiB) that is part of the library image, so every GPU that loads the library holds that
 * much memory until the process exits.
 *   - Arguments and semantics are those of h2o_prefill_select, minus scratch / scratch_bytes.
 *   - Limit: prompts whose scratch need, h2o_prefill_scratch_bytes(cfg, cu[batch]), exceeds the
 *     array are refused with H2O_ERR_WORKSPACE and nothing is launched (16 MiB covers about one
 *     million (token, head) pairs, e.g. 8 prompts of 2048 tokens with 32 heads).
 *   - It performs no device allocation or free and calls no allocating library routine.
 *   - The first call on a device looks up the array's device address (one runtime query, with
 *     that device made current for the query); make that first call before starting any stream
 *     capture on the device.
 *   - All calls on a device share the one array, and the array keeps whatever the last call
 *     left in it.  Nothing in it needs to start at zero, so no clearing is done; but two calls
 *     whose work overlaps on the GPU (different streams, no ordering between them) race on it
 *     and corrupt each other.  Order such calls, or use h2o_prefill_select with own buffers.
 */
size_t h2o_prefill_static_scratch_bytes(void);
int h2o_prefill_select_static(h2o_cache_t* cache, const void* q, const void* k, const void* v,
                              const int32_t* cu_seqlens, void* out, void* stream);

/*
 * The same two calls for callers whose tensors live in HOST memory (pinned memory
 * makes the copies asynchronous).  Inputs are copied to `staging` (dev, 256-byte
 * aligned) on the stream, the device call above runs on the staged copies, and the
 * results are copied back to the host buffers on the same stream; the host buffers
 * must stay valid until the stream has finished this work.
 *   h2o_prefill_select_host: staging >= 4 tensors of [total_tokens, n_heads, head_dim]
 *                            (each rounded up to 256 bytes); scratch as above.
 *   h2o_decode_step_host   : staging >= 4 tensors of [batch, n_heads, head_dim] plus
 *                            [batch, n_heads] int32 (each rounded up to 256 bytes).
 *   (With query_group = G > 1 the q and out tensors of both calls carry n_heads * G heads.)
 * When every buffer of h2o_decode_step_host is pinned or registered host memory (which the
 * device can address) and 16-byte aligned, the kernel reads and writes it directly and no
 * copy is enqueued; the buffers must then not be touched by the host until the stream has
 * finished the call, and `staging` is unused.
 * h2o_host_staging_bytes(cfg, tokens) gives the size for `tokens` rows per tensor
 * (tokens = total_tokens for prefill, batch for decode); 0 for invalid arguments.
 * No counterpart in the paper; the semantics are those of the device calls.
 */
size_t h2o_host_staging_bytes(const h2o_config_t* cfg, int64_t tokens);
int h2o_prefill_select_host(h2o_cache_t* cache, const void* q_host, const void* k_host, const void* v_host,
                            const int32_t* cu_seqlens, void* out_host, void* staging, size_t staging_bytes,
                            void* scratch, size_t scratch_bytes, void* stream);
int h2o_decode_step_host(h2o_cache_t* cache, const void* q_host, const void* k_new_host, const void* v_new_host,
                         void* out_host, int32_t* evicted_pos_host, void* staging, size_t staging_bytes, void* stream);

/*
 * Return the cache to the empty state of h2o_cache_create (every unit holds 0
 * tokens, t = 0, status cleared) with work enqueued on the stream, so that a
 * workspace can serve a new batch of prompts without a new handle.
 */
int h2o_cache_reset(h2o_cache_t* cache, void* stream);

/* Free the host-side handle.  NULL is accepted.  The workspace stays the caller's. */
int h2o_cache_destroy(h2o_cache_t* cache);

/*
 * Diagnostics (no counterpart in the paper).
 * h2o_cache_export copies, for every unit u = s * n_heads + h, its slot table into
 * host arrays with a fixed row pitch: pos [units][pitch] (unused entries -1),
 * acc [units][pitch], count [units], t [units]; pitch >= max_s B_s.  Synchronises
 * the stream.  Any output pointer may be NULL.
 * h2o_cache_status synchronises the stream and returns the device status word
 * (H2O_OK, or the first H2O_ERR_* a kernel recorded).
 */
int h2o_cache_export(h2o_cache_t* cache, int32_t* pos, double* acc, int32_t* count, int32_t* t, int32_t pitch,
                     void* stream);
int h2o_cache_status(h2o_cache_t* cache, void* stream);
/*
 * Tuning knob (no counterpart in the paper): how the decode kernel is laid out.
 * split  = thread blocks (one cluster) sharing a unit: 1, 2, 4 or 8; 0 keeps the
 *          value chosen at create time from the number of units and the budgets.
 * stages = depth of the shared-memory ring of 16 KB (K tile + V tile) stages, 1..8
 *          (rounded down to a power of two); 0 = default.  Results do not depend on
 *          either value beyond summation order.
 */
int h2o_cache_set_decode_shape(h2o_cache_t* cache, int32_t split, int32_t stages);
/*
 * Diagnostics for the prefill (no counterpart in the paper).
 * h2o_cache_set_prefill_path: 0 = automatic (tensor-core kernels for bf16 with head_dim
 *   128, fp32-FMA kernels otherwise), 1 = always the fp32-FMA kernels.
 * h2o_prefill_scratch_layout: byte offset, inside the scratch buffer of
 *   h2o_prefill_select, of the column sums acc0 (double, [n_heads][total_tokens]); valid
 *   once the stream has finished the call.
 */
int h2o_cache_set_prefill_path(h2o_cache_t* cache, int32_t path);
/*
 * Which kernel runs a multi-head decode step (no counterpart in the paper; results differ by summation order
 * only): 0 = automatic, 1 = the online-softmax kernel (one pass over K and V tile pairs),
 * 2 = the two-pass streaming kernel (bf16, head_dim 128:
 * K stream with the scores on the tensor cores, exact softmax, V stream; H2O_ERR_UNSUPPORTED where it does not
 * apply: other dtypes, 4-bit slots, grouped caches (which have their own form of it),
 * budgets whose scores do not fit shared memory).  Automatic takes 2 for launches of more than two blocks per SM
 * whose mean budget is at least 100 slots; with "Top-K" attention set, for launches of at most two blocks per SM.
 */
int h2o_cache_set_decode_path(h2o_cache_t* cache, int32_t path);
/* The kind of kernel the next h2o_decode_step of this cache launches: 2 = two streaming passes, 1 = one pass
 * (online softmax; for 4-bit slots and for grouped caches outside the streaming kernel's reach: their own
 * one-block-per-unit kernels).  Negative: H2O_ERR_INVALID_ARG (null handle). */
int h2o_cache_get_decode_path(h2o_cache_t* cache);
/* h2o_decode_chunk: 0 = automatic (chunk kernel where it applies), 1 = one decode-step kernel per token. */
int h2o_cache_set_chunk_path(h2o_cache_t* cache, int32_t path);
/*
 * Score variants.
 *
 * h2o_cache_set_score_mode: how candidates are RANKED when heavy hitters are selected after the prompt
 *   and when a victim is chosen in a decode step.
 *     0 (default)  by the accumulated attention score (Algorithm 1 / Algorithm 2, h(z) = z);
 *     1            by the averaged attention score — the accumulated score divided by the number of queries
 *                  that attended the key (a key at position p, current query position t: t - p + 1; after a
 *                  prompt of n tokens: n - p) — the variant the paper's "Discussions and Limitations" reports
 *                  as an experiment against the bias towards old tokens.
 *   The stored scores are the accumulated ones in both modes; ties still go to the lowest position.
 *   Only on an empty cache (after create or reset, before the first prefill or decode call): H2O_ERR_STATE
 *   otherwise.  The mode survives h2o_cache_reset.  With mode 1, h2o_decode_chunk takes one decode-step
 *   kernel per token.
 *
 * h2o_cache_fscore: F_score of every unit, the sum of h(accumulated score) over the unit's kept keys (the
 *   score function in the paper's definition of the eviction policy; remark on h).
 *     hkind 0: h(z) = z,  1: h(z) = sqrt(z + 1),  2: h(z) = log(z + 1).
 *   Reporting only: for an increasing h the victim is the same.  out_dev: DEVICE pointer, [batch * n_heads]
 *   doubles in (sequence, head) order, written on `stream`; owned by the caller.
 *   Errors: H2O_ERR_INVALID_ARG (null pointer, hkind outside 0..2), H2O_ERR_CUDA.
 */
int h2o_cache_set_score_mode(h2o_cache_t* cache, int32_t mode);
/*
 * Heavy hitters combined with a sparse attention pattern (Section 5.1, the table that lists the strided and
 * the fixed Sparse Transformer patterns with and without H2; the paper gives the results, not the rule).  This
 * library's reading: the cache keeps what it keeps without a pattern — k_s heavy hitters by accumulated score
 * and the r_s most recent positions — and the pattern decides which entries of the RECENT region a query
 * attends.  For the query at position t and a key at position p:
 *     p == t         attended (the token itself);
 *     p <= t - r_s   attended (a heavy hitter, or the entry that has just left the window);
 *     t - r_s < p < t attended iff the pattern allows it:
 *       kind 1, strided(a = stride, b = local window): t - p < b or (t - p) mod a == 0;
 *       kind 2, fixed(a = block length, b = summary columns, b <= a): floor(p / a) == floor(t / a) or
 *                                                                    p mod a >= a - b.
 *   An entry that is not attended is absent from the softmax of that step and its score does not grow.  The
 *   prompt rows of h2o_prefill_select follow the same rule.  "Without H2" is k_s = 0; kind 0 switches the
 *   pattern off.
 * Only on an empty cache (H2O_ERR_STATE otherwise); the pattern survives h2o_cache_reset.  With a pattern,
 * h2o_prefill_select uses the fp32-FMA kernels and h2o_decode_chunk one decode-step kernel per token.
 * Errors: H2O_ERR_INVALID_ARG (kind outside 0..2, a < 1, b < 0, b > a for kind 2), H2O_ERR_UNSUPPORTED
 * (4-bit slots).
 */
int h2o_cache_set_mask(h2o_cache_t* cache, int32_t kind, int32_t a, int32_t b);
/*
 * Heavy hitters combined with "Top-K" attention (appendix "Enhancing the Top-K baseline", the table with and
 * without H2; results only, no rule).  This library's reading: in a decode step the query attends, of everything it
 * would otherwise attend (the kept entries, minus what a sparse pattern leaves out, and the token itself), only the
 * m entries with the largest scaled logits; equal logits: the higher position first.  The others get probability 0
 * and their accumulated score does not grow in that step; the cache policy itself is unchanged.  The kernel
 * streams the keys only and reads just the value rows of the attended entries.  m = 0 switches it off.
 * The prompt rows of h2o_prefill_select stay dense.
 * Only on an empty cache (H2O_ERR_STATE otherwise); the setting survives h2o_cache_reset.  A unit stays in one
 * thread block (budgets up to 8192 slots; H2O_ERR_UNSUPPORTED beyond, and for 4-bit slots); h2o_decode_chunk takes
 * one decode-step kernel per token.  Which of two logits closer than fp32 resolves is the larger one is decided in
 * fp32 here.
 */
int h2o_cache_set_topk(h2o_cache_t* cache, int32_t m);
int h2o_cache_fscore(h2o_cache_t* cache, int32_t hkind, double* out_dev, void* stream);
/*
 * Process-wide diagnostic switch (no counterpart in the paper).  A decode kernel launched right
 * after a decode / prefill / reset of a DIFFERENT cache on the same stream starts copying its own
 * cache tiles into shared memory before the preceding kernel has finished (inputs q/k/v are still
 * read only afterwards).  0 turns that off, so that every launch waits first; results must be
 * identical either way.  Returns the previous setting.
 */
int h2o_debug_set_early_prefetch(int32_t enabled);
/*
 * Diagnostic (no counterpart in the paper): enqueue a one-warp kernel that polls `polls` times
 * (1 .. 2^20, i.e. at most a few milliseconds) on a barrier nobody ever arrives at and then, like
 * every bounded wait of this library that gives up, records H2O_ERR_TIMEOUT in the cache's status
 * word and returns normally.  h2o_cache_status then reports the code; h2o_cache_reset clears it.
 * Shows that a timed-out wait costs a status code, not the context.
 */
int h2o_debug_wait_probe(h2o_cache_t* cache, int32_t polls, void* stream);
int h2o_prefill_scratch_layout(const h2o_config_t* cfg, int64_t total_tokens, size_t* acc0_offset);
/*
 * Diagnostic (no counterpart in the paper): per-kernel timing of the NEXT h2o_prefill_select call on this
 * cache.  `events`: host array of four cudaEvent_t (created by the caller with timing enabled; NULL entries
 * are skipped), recorded on that call's stream before the attention kernel (P1-P3 of the path), after it,
 * after the column-sum kernel (P4) and after selection and gather (P5-P6).  The handles are used by that one
 * call only; `events` == NULL cancels.  Recording between the kernels orders them strictly, so a timed call
 * can be a little slower than an untimed one.
 */
int h2o_debug_set_prefill_events(h2o_cache_t* cache, void* const* events);
/*
 * Diagnostic (no counterpart in the paper): 1 if this library was built with -DH2O_BOUNDS — every slot, unit and
 * prompt-row index of the kernels checked before use, a violation recorded as H2O_ERR_STATE in the status word
 * and the access skipped (the build the parity tests are also run against, in place of a memory checker) —
 * 0 for the normal build.
 */
int h2o_debug_bounds_checked(void);
const char* h2o_strerror(int code);

#ifdef __cplusplus
}
#endif
#endif /* H2O_B200_H_ */
