/*
 * efim.h - C ABI of the EFIM per-turn GPU path (NVIDIA B200, sm_100a).
 *
 * EFIM (Sec. 1; Sec. 2.2, Fig. 3) rewrites an infilling prompt from
 * `<P>prefix+inc<S>suffix<M>` to `<P>prefix<S>suffix<M>inc`.  The keys and
 * values of `<P>prefix<S>suffix<M>` (C tokens) then stay valid in the paged KV
 * cache from one turn to the next; each turn only has to
 *   1. rotate the N new `inc` tokens' q/k by their positions C..C+N-1 and store
 *      k/v into the cache pages                       -> efim_kv_append
 *   2. attend the N new queries causally over the C cached and N new keys
 *                                                     -> efim_append_prefill_attn
 *   3. decode the generated middle one token at a time -> efim_decode_attn
 * The paper changes nothing in the model (Sec. 3), so 2 and 3 are standard
 * softmax attention, o = sum_j softmax_j(scale * q.k_j) v_j.
 *
 * Conventions for every entry point
 *   - Pointers named d_* are DEVICE pointers, h_* are HOST pointers.  The caller
 *     owns all memory and the stream; the library allocates no device memory and never
 *     synchronises the device.  What it keeps between calls: the fixed array of
 *     efim_decode_attn_static (and its per-device address), the SM count of each device it
 *     has planned for, the driver entry point it encodes tensor maps with, the encoded maps
 *     of the pools each host thread used last and which devices have had a kernel's
 *     shared-memory limit raised - host-side look-ups made once; no call's result depends
 *     on an earlier call.
 *   - `stream` is a cudaStream_t passed as void* (NULL = default stream).  All
 *     work is enqueued on it; results are ready when the stream reaches that point.
 *   - Stream capture: calls that copy a work list from pageable host memory must not be
 *     issued while the stream is capturing - efim_append_prefill_attn, and
 *     efim_append_prefill_step without a plan.  The planned calls can be captured with
 *     lists_resident = 1 (they only launch), or with lists_resident = 0 and a blob in pinned
 *     memory that outlives the graph.  efim_kv_append, efim_decode_attn and efim_decode_step
 *     only launch.
 *   - bf16 tensors are raw 16-bit patterns.  Packed layouts, innermost last:
 *       q / out      [total_new_tokens][num_q_heads][head_dim]   bf16
 *       k_new/v_new  [total_new_tokens][num_kv_heads][head_dim]  bf16
 *       pools        [num_pages][num_kv_heads][page_size][head_dim] bf16 (K and V separate)
 *       block table  [batch][max_pages_per_seq] int32: token p of sequence s lives
 *                    in page block_table[s][p / page_size], slot p % page_size.
 *     Sequence s owns rows q_indptr[s] .. q_indptr[s+1]-1 of the packed tensors.
 *   - Grouped-query map: q head h reads kv head h / (num_q_heads / num_kv_heads).
 *   - Errors the host can see (null pointers, unsupported shapes, workspace too
 *     small) are returned before anything is launched.  Errors only the device can
 *     see are OR-ed into *d_status (EFIM_DEV_* bits) if d_status is not NULL, and the
 *     offending access is skipped; the kernels never trap.
 *   - Supported: page_size 16; head_dim 64 or 128; num_q_heads a multiple of
 *     num_kv_heads; base pointers 16-byte aligned (pools 128-byte aligned).
 */
#ifndef EFIM_H_
#define EFIM_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
  EFIM_OK = 0,
  EFIM_ERR_INVALID_ARG = 1,   /* null pointer, negative size, H_q % H_kv != 0, bad alignment */
  EFIM_ERR_UNSUPPORTED = 2,   /* head_dim / page_size outside the supported set; more than 32767 kv heads
                                 or num_pages * num_kv_heads above 2^31 - 1                  */
  EFIM_ERR_OUT_OF_RANGE = 3,  /* a host-visible length exceeds max_pages_per_seq*page_size  */
  EFIM_ERR_WORKSPACE = 4,     /* workspace_bytes smaller than the *_workspace_bytes() answer */
  EFIM_ERR_CUDA = 5,          /* a CUDA runtime/driver call failed (launch, copy, tensor map) */
  EFIM_ERR_TIMEOUT = 6        /* reserved: reported through d_status by bounded device waits */
} efim_status;

/* Bits OR-ed into *d_status by kernels. */
#define EFIM_DEV_BAD_PAGE      0x1   /* block-table entry outside [0, num_pages)           */
#define EFIM_DEV_BAD_POSITION  0x2   /* token position >= rope max_position, or beyond table */
#define EFIM_DEV_TIMEOUT       0x4   /* a bounded wait inside a kernel expired               */

const char* efim_strerror(efim_status s);
/* Text of the CUDA error behind the calling thread's most recent EFIM_ERR_CUDA. */
const char* efim_last_cuda_error(void);
int efim_version(void);

/* Paged KV cache of ONE layer. */
typedef struct {
  void* d_k_pool;            /* bf16 [num_pages][num_kv_heads][page_size][head_dim] */
  void* d_v_pool;            /* same shape                                         */
  int32_t num_pages;
  int32_t page_size;         /* 16 */
  int32_t num_q_heads;
  int32_t num_kv_heads;
  int32_t head_dim;          /* 64 or 128 */
} efim_cache_desc;

/* Ragged batch of one turn: sequence s has cached_len[s] tokens already in the
 * cache (`<P>prefix<S>suffix<M>`) and new_len[s] new tokens (`inc`). */
typedef struct {
  int32_t batch;
  int32_t max_pages_per_seq;
  int32_t total_new_tokens;          /* = q_indptr[batch]                             */
  const int32_t* d_cached_len;       /* [batch]                                       */
  const int32_t* d_new_len;          /* [batch]                                       */
  const int32_t* d_q_indptr;         /* [batch+1], exclusive prefix sum of new_len    */
  const int32_t* d_block_table;      /* [batch][max_pages_per_seq]                    */
  const int32_t* h_cached_len;       /* host mirrors, read during the call (planning) */
  const int32_t* h_new_len;
} efim_batch_desc;

/* Rotary embedding.  d_cos_sin row p holds cos(p*theta_f), f = 0..D/2-1, then
 * sin(p*theta_f), f = 0..D/2-1, theta_f = base^(-2f/D).  Pair (f, f+D/2) is
 * rotated, or (2f, 2f+1) when interleaved != 0.  d_cos_sin == NULL disables the
 * rotation (k is stored as given, q untouched). */
typedef struct {
  const float* d_cos_sin;    /* fp32 [max_position][head_dim] */
  int32_t max_position;
  int32_t interleaved;
} efim_rope_desc;

/* Fill a HOST table for efim_rope_desc (computed in double, rounded to float).
 * h_out: [max_position][head_dim] floats owned by the caller.  The paper fixes only the
 * token order (Sec. 1), hence each token's position; the rotary embedding itself is that of
 * the model families it serves (Sec. 4.1), read here as theta_f = base^(-2f/head_dim), no
 * scaling. */
efim_status efim_rope_table_build(double base, int32_t head_dim, int32_t max_position, float* h_out);

/*
 * Step 1 (EFIM Sec. 1: only `inc` is new; its k/v join the cache after
 * `<P>prefix<S>suffix<M>`).  For new token i of sequence s, position
 * p = cached_len[s] + i: q and k are rotated by p (fp32 math, one bf16
 * round-to-nearest-even), q is rewritten in place, k (rotated) and v (as is) are
 * stored at page block_table[s][p/page_size], slot p%page_size, all kv heads.
 * d_q may be NULL (only k/v are processed).  Sequences must not share a page that
 * is written.  A bad page id or position sets a bit in *d_status and skips that token.
 */
efim_status efim_kv_append(const efim_cache_desc* cache, const efim_batch_desc* batch,
                           const efim_rope_desc* rope,
                           void* d_q, const void* d_k_new, const void* d_v_new,
                           int32_t* d_status, void* stream);

/*
 * Step 2 (EFIM Sec. 1, Sec. 2.2: prefix and suffix KV are cache hits, so the
 * prefill that remains is the `inc` tokens attending over everything before
 * them).  The new tokens' k/v must already be in the pages (efim_kv_append).
 * A block-table entry outside [0, num_pages) among the pages a row sees sets
 * EFIM_DEV_BAD_PAGE; the 16 keys of that page are taken as zeros (the rows that see it are
 * finite and meaningless, all other rows unaffected).
 * New token i of sequence s (position C+i) sees keys j <= C+i:
 *   out[t,h,:] = sum_j softmax_j(sm_scale * q[t,h,:].k[j,h/G,:]) v[j,h/G,:]
 *   lse[t,h]   = log sum_j exp(sm_scale * q.k_j)         (natural log; optional)
 * bf16 operands, fp32 accumulation and softmax, bf16 output.
 * sm_scale <= 0 selects 1/sqrt(head_dim).  Sequences with new_len 0 are skipped.
 * The host mirrors h_cached_len/h_new_len are read during the call to build the
 * work list, which is copied into the workspace on `stream`.
 * Workspace: at least efim_prefill_workspace_bytes() bytes, 256-byte aligned,
 * exclusively this call's until the stream has passed it.
 */
size_t efim_prefill_workspace_bytes(const efim_cache_desc* cache, const efim_batch_desc* batch);
efim_status efim_append_prefill_attn(const efim_cache_desc* cache, const efim_batch_desc* batch,
                                     const void* d_q, void* d_out, float* d_lse, float sm_scale,
                                     void* d_workspace, size_t workspace_bytes,
                                     int32_t* d_status, void* stream);

/*
 * Step 2 with the planning taken out of the call.  The work list depends only on the batch's
 * lengths and the cache shape, not on the layer: a model runs step 2 once per layer on the
 * same batch, so it plans once and runs many times.  efim_prefill_plan() writes the plan - a
 * relocatable blob of efim_prefill_plan_bytes() bytes - into HOST memory of the caller;
 * efim_append_prefill_attn_planned() is efim_append_prefill_attn() with that blob in place of
 * the planning (same results bit for bit, same workspace size).  With lists_resident = 0 the
 * blob's lists are first copied to the head of the workspace on `stream`: keep the blob alive
 * and unchanged until the stream has passed the call (pinned memory makes the copy
 * asynchronous).  With lists_resident = 1 the call copies nothing and only launches: the head
 * of this workspace must still hold the lists from an earlier call with the same plan (the
 * kernels only read them; the partials live behind them) - upload once per batch, run per layer.
 * EFIM_ERR_INVALID_ARG if the blob was not made for this cache shape and these lengths
 * (checked against a hash of the host mirrors), EFIM_ERR_WORKSPACE if plan_bytes is too small.
 */
size_t efim_prefill_plan_bytes(const efim_cache_desc* cache, const efim_batch_desc* batch);
efim_status efim_prefill_plan(const efim_cache_desc* cache, const efim_batch_desc* batch,
                              void* h_plan, size_t plan_bytes);
efim_status efim_append_prefill_attn_planned(const efim_cache_desc* cache, const efim_batch_desc* batch,
                                             const void* h_plan, size_t plan_bytes, int32_t lists_resident,
                                             const void* d_q, void* d_out, float* d_lse, float sm_scale,
                                             void* d_workspace, size_t workspace_bytes,
                                             int32_t* d_status, void* stream);

/*
 * Steps 1 and 2 of a turn in one call (EFIM Sec. 1: the `inc` tokens join the cache after
 * `<P>prefix<S>suffix<M>` and attend over everything before them).  Equivalent to
 *     efim_kv_append(rope, d_q, d_k_new, d_v_new) ; efim_append_prefill_attn[_planned](d_q)
 * - out, lse and the pools bit for bit - but d_q is READ ONLY: the attention kernel rotates
 * each query row by its position cached_len[s] + i as it loads it (the same fp32 arithmetic
 * and single bf16 rounding), and the append moves only k and v.  The rotated q is never
 * written, which at equal head counts is two thirds of what efim_kv_append moves.
 * h_plan = NULL: the work list is planned inside the call (as efim_append_prefill_attn does);
 * otherwise h_plan / plan_bytes / lists_resident are those of
 * efim_append_prefill_attn_planned.  `rope` may be NULL or hold a NULL table (no rotation).
 * A query position >= rope->max_position sets EFIM_DEV_BAD_POSITION; that row attends with a
 * zero query (its output is finite and meaningless), its k/v are not appended.
 * d_k_new and d_v_new may both be NULL: the new tokens' k/v are then taken to be in the
 * pages already (an earlier efim_kv_append with d_q = NULL) and only the attention runs.
 * Two kernels are enqueued (three when the key range is split).
 */
efim_status efim_append_prefill_step(const efim_cache_desc* cache, const efim_batch_desc* batch,
                                     const efim_rope_desc* rope, const void* d_q,
                                     const void* d_k_new, const void* d_v_new, void* d_out, float* d_lse,
                                     float sm_scale, const void* h_plan, size_t plan_bytes,
                                     int32_t lists_resident, void* d_workspace, size_t workspace_bytes,
                                     int32_t* d_status, void* stream);

/*
 * Step 3 (decode of the generated middle, EFIM Sec. 2.2 / Fig. 4): one query
 * token per sequence over keys [0, ctx_len[s]) (ctx_len counts the token just
 * appended).  The key range is cut into fixed-length chunks; each chunk yields a
 * partial (o_c, lse_c) in the workspace and a second kernel merges them:
 *   lse = log sum_c exp(lse_c),  o = sum_c exp(lse_c - lse) o_c.
 * max_ctx_len is an upper bound on every ctx_len[s] (<= 0: max_pages_per_seq *
 * page_size); it fixes the chunking, so no host copy of the lengths is needed.
 * ctx_len[s] == 0 gives out = 0, lse = -inf.  Query-head groups of up to 7 per kv head read
 * the K/V pages once; larger groups are cut into tiles of 4 or 3 heads that each read them.
 * (The kernel works on fp32 FMAs; from about 5 heads per kv head on a batch of decode rows is
 * served faster by efim_append_prefill_attn as rows with new_len = 1, which is legal there.)  A device length beyond what the launch was
 * planned for (the chunks cover max_ctx_len rounded up to whole chunks, at most the block
 * table's capacity) is clamped to that and sets EFIM_DEV_BAD_POSITION; nothing outside the
 * workspace or the table is touched.
 */
size_t efim_decode_workspace_bytes(const efim_cache_desc* cache, int32_t batch, int32_t max_ctx_len);
/* Number of kernels the corresponding call enqueues for these arguments (the main
 * kernel, plus a merge kernel when the key range is split); 0 for invalid arguments.
 * Planning queries for profiling and launch accounting; they launch nothing. */
int32_t efim_prefill_launch_count(const efim_cache_desc* cache, const efim_batch_desc* batch);
int32_t efim_decode_launch_count(const efim_cache_desc* cache, int32_t batch, int32_t max_ctx_len);
efim_status efim_decode_attn(const efim_cache_desc* cache, int32_t batch,
                             const int32_t* d_ctx_len, int32_t max_ctx_len,
                             const int32_t* d_block_table, int32_t max_pages_per_seq,
                             const void* d_q, void* d_out, float* d_lse, float sm_scale,
                             void* d_workspace, size_t workspace_bytes,
                             int32_t* d_status, void* stream);

/*
 * Steps 1 and 3 of a decode step in one launch: the generated token of row s is the row's
 * last key, position ctx_len[s] - 1.  The kernel rotates its q and k by that position
 * (the same fp32 arithmetic and single bf16 rounding as efim_kv_append), stores k/v into
 * the page slot and attends over keys [0, ctx_len[s]) - the result of
 *     efim_kv_append(cached_len = ctx_len - 1, new_len = 1) ; efim_decode_attn(ctx_len)
 * bit for bit, with one kernel less per step.  Differences: d_q is read only (the rotated q
 * is not written back); `rope` may be NULL or hold a NULL table (no rotation); rows with
 * ctx_len[s] == 0 append nothing.  A position >= rope->max_position sets
 * EFIM_DEV_BAD_POSITION and skips the row (nothing appended, out = 0, lse = -inf); a length
 * that had to be clamped (see efim_decode_attn) appends nothing either and attends over the
 * clamped range.  d_k_new / d_v_new: [batch][num_kv_heads][head_dim]
 * bf16.  Workspace and every other argument as for efim_decode_attn.
 */
efim_status efim_decode_step(const efim_cache_desc* cache, int32_t batch,
                             const int32_t* d_ctx_len, int32_t max_ctx_len,
                             const int32_t* d_block_table, int32_t max_pages_per_seq,
                             const efim_rope_desc* rope, const void* d_q,
                             const void* d_k_new, const void* d_v_new, void* d_out, float* d_lse,
                             float sm_scale, void* d_workspace, size_t workspace_bytes,
                             int32_t* d_status, void* stream);

/*
 * Allocation-free variant of efim_decode_attn (the paper has no counterpart; this is
 * a convenience of this library).  For callers that cannot provide a workspace
 * because they may not allocate device memory at all - a serving loop that has
 * given every free byte to its KV pool, a plug-in handed only input and output
 * pointers, a latency-critical thread that must not block in the allocator.  The
 * chunk partials go to a fixed array of efim_decode_static_scratch_bytes() bytes
 * (8 MiB) that lives inside the library on every GPU that loads it, from load to
 * process exit.  Same arguments, results and errors as efim_decode_attn without the
 * workspace pair, plus:
 *   - EFIM_ERR_WORKSPACE if this (batch, heads, max_ctx_len) needs more than the
 *     fixed array, i.e. efim_decode_workspace_bytes() > efim_decode_static_scratch_bytes();
 *     use efim_decode_attn with your own workspace then.
 *   - The first call on each device looks up the array's device address (no
 *     allocation, but a runtime query): make that first call outside any stream
 *     capture, with the device current.
 *   - All calls on a device share the one array and it keeps the previous call's
 *     partials.  Nothing has to be cleared (each call overwrites what it reads back),
 *     but two calls whose kernels may overlap on the GPU - different streams without
 *     an ordering between them - race on it.  Issue them on one stream or order them.
 *   - Calls no cudaMalloc/cudaFree and no allocating library routine.
 */
size_t efim_decode_static_scratch_bytes(void);
efim_status efim_decode_attn_static(const efim_cache_desc* cache, int32_t batch,
                                    const int32_t* d_ctx_len, int32_t max_ctx_len,
                                    const int32_t* d_block_table, int32_t max_pages_per_seq,
                                    const void* d_q, void* d_out, float* d_lse, float sm_scale,
                                    int32_t* d_status, void* stream);

/*
 * Self-test of the bounded device wait (the paper has no counterpart).  Every wait inside
 * the kernels - on a bulk copy, on a tensor-core commit - gives up after a limit, sets
 * EFIM_DEV_TIMEOUT in *d_status and lets the kernel end normally.  This call runs that code
 * in isolation: one warp waits on a barrier that nothing will ever complete, with nothing in
 * flight, for limit_ns nanoseconds (1 .. 100,000,000).  Afterwards *d_status has
 * EFIM_DEV_TIMEOUT set and *d_waited_ns (optional, device) holds how long the warp waited.
 */
efim_status efim_selftest_bounded_wait(uint64_t limit_ns, int32_t* d_status, uint64_t* d_waited_ns, void* stream);

/* ------------------------------------------------------------------------------------
 * Host-side front end (no GPU work): what turns a stream of infilling requests into the
 * (cached_len, new_len, block table) triples the three calls above consume.
 *
 * 1. Prompt transformation, Sec. 3.1 (Fig. 7, steps 1-5).  A per-user session keeps the
 *    prefix and suffix as they were laid out in the user's last prompt.  For a request
 *    (user, prefix, suffix), all token ids:
 *      - no session (step 2):                    `<P>prefix<S>suffix<M>`, session created
 *      - prefix = session prefix + inc, inc not empty (step 4):
 *                                                `<P>session prefix<S>suffix<M>inc`  (EFIM, Sec. 1)
 *        the session keeps its prefix (so the next turn's prompt again starts with the same
 *        tokens) and takes the request's suffix
 *      - prefix unchanged (step 5, or a repeat): `<P>prefix<S>suffix<M>`, session takes the suffix
 *      - prefix edited or shortened:             `<P>prefix<S>suffix<M>`, session replaced
 *    `rebase_inc_tokens` > 0 bounds inc: a longer increment is folded back into the prefix
 *    with one PSM prompt (the paper states no bound; 0 = never).
 * 2. Cross-request KV reuse as Sec. 1 states it: the KV of a prompt can be reused for the
 *    tokens whose whole token prefix equals an earlier sequence's.  Reuse is per page:
 *    admit() pins the longest run of cached full pages at the start of the prompt (leaving at
 *    least one token to compute) and takes pages for the rest plus `reserve_tokens` of decode
 *    room - the lowest-numbered free page first, else the least recently used unpinned cached
 *    page (among equals the deepest one); finish() registers the full pages of the finished
 *    sequence, frees duplicates, the partial last page and unused room.
 * All pointers are HOST pointers; a front end is not thread safe; nothing here touches CUDA.
 */
typedef struct efim_frontend efim_frontend;

/* values of *format */
#define EFIM_FMT_PSM_NEW     0
#define EFIM_FMT_EFIM        1
#define EFIM_FMT_PSM_SUFFIX  2
#define EFIM_FMT_PSM_SAME    3
#define EFIM_FMT_PSM_RESET   4
#define EFIM_FMT_PSM_REBASE  5

/* NULL if num_pages <= 0 or page_size <= 0. */
efim_frontend* efim_frontend_create(int32_t tok_p, int32_t tok_s, int32_t tok_m, int32_t rebase_inc_tokens,
                                    int32_t num_pages, int32_t page_size);
void efim_frontend_destroy(efim_frontend* fe);

/* Builds the prompt for one request.  Needs capacity >= prefix_len + suffix_len + 3, else
 * EFIM_ERR_OUT_OF_RANGE (and the session is left as it was). */
efim_status efim_frontend_transform(efim_frontend* fe, int64_t user, const int32_t* h_prefix, int32_t prefix_len,
                                    const int32_t* h_suffix, int32_t suffix_len, int32_t* h_prompt,
                                    int32_t capacity, int32_t* prompt_len, int32_t* format, int32_t* inc_len);

/* Admits a prompt: *cached_len tokens are already in the pages named by the first entries of
 * h_block_table_row, *num_pages_out entries are written in all (ceil((prompt_len + reserve_tokens)
 * / page_size)); the rest of the row is set to -1.  EFIM_ERR_OUT_OF_RANGE if the row is too
 * short, EFIM_ERR_WORKSPACE if the pool has no page left to take (nothing is pinned then). */
efim_status efim_frontend_admit(efim_frontend* fe, const int32_t* h_prompt, int32_t prompt_len,
                                int32_t reserve_tokens, int32_t* h_block_table_row, int32_t max_pages_per_seq,
                                int32_t* cached_len, int32_t* num_pages_out, int64_t* handle);
/* The request is over; h_tokens[0..total_len) is the sequence whose KV its pages now hold
 * (the prompt followed by what was generated).  EFIM_ERR_INVALID_ARG for an unknown handle. */
efim_status efim_frontend_finish(efim_frontend* fe, int64_t handle, const int32_t* h_tokens, int32_t total_len);
/* h_out[0..4) = prompt tokens admitted, of which found cached, pages evicted, pages free now. */
void efim_frontend_stats(const efim_frontend* fe, int64_t* h_out);

/* ------------------------------------------------------------------------------------
 * Fragment tokenisation, Sec. 3.2 (Fig. 8: "the length of each segment follows uniform
 * distribution [1,200]"): the training-side data processing that teaches a model to emit
 * sub-word pieces anywhere.  The library decides where a text is cut; the caller
 * tokenises every segment on its own and concatenates the ids.  Host only.
 * Lengths count characters (the paper does not say) and are lo + z_i mod (hi - lo + 1)
 * with z_i the i-th draw of SplitMix64 under `seed`; the last segment is what is left.
 *
 * efim_fragment_cuts: writes the end offsets of the segments of a text of n characters
 * (the last one is n) into h_cuts, at most `capacity` of them, and returns how many there
 * are (so call with capacity 0 to size); -1 for invalid arguments (n < 0, lo < 1, hi < lo).
 * efim_fim_split: the two cut points 0 <= a <= b <= n of the FIM transformation of a
 * document (prefix [0,a), middle [a,b), suffix [b,n); Sec. 2.1), both uniform on [0, n].
 */
int64_t efim_fragment_cuts(uint64_t seed, int64_t n, int32_t lo, int32_t hi, int64_t* h_cuts, int64_t capacity);
efim_status efim_fim_split(uint64_t seed, int64_t n, int64_t* a, int64_t* b);

/*
 * One FIM training example with fragment tokenisation (Sec. 2.1 for the PSM layout
 * `<P>prefix<S>suffix<M>middle`, Sec. 3.2 for the segments): the document of n characters is
 * split by efim_fim_split(seed), each of the three parts is cut into segments on its own (a
 * segment never spans a special token; generator seeds seed+1 prefix, seed+2 suffix, seed+3
 * middle), and the example is the list of spans in the order they are emitted.  h_spans
 * receives up to `capacity` triples (kind, begin, end): kind EFIM_SPAN_TEXT = tokenise
 * characters [begin, end) of the document on their own; EFIM_SPAN_TOKEN_P/_S/_M = emit that
 * special token (begin = end = where the part starts).  Returns the number of spans (call
 * with capacity 0 to size), -1 for invalid arguments.
 */
#define EFIM_SPAN_TEXT     0
#define EFIM_SPAN_TOKEN_P  1
#define EFIM_SPAN_TOKEN_S  2
#define EFIM_SPAN_TOKEN_M  3
int64_t efim_fim_fragment_spans(uint64_t seed, int64_t n, int32_t lo, int32_t hi, int64_t* h_spans,
                                int64_t capacity);

#ifdef __cplusplus
}
#endif
#endif /* EFIM_H_ */
