/*
 * klpm.h -- C ABI of the device-resident k-LPM scheduling path (sm_100a).
 *
 * The library keeps a flattened radix tree of cached prompts in device memory and runs, on the GPU,
 * batched longest-prefix matching, the k-LPM / FCFS / LPM selection rule and the schedule replay
 * under the paper's prefix-reuse cost model.
 *
 * Conventions that hold for every entry point unless its comment says otherwise:
 *   - `d_*` arguments are DEVICE pointers owned by the caller (4-byte aligned for int32 data,
 *     8-byte aligned for int64 data).  The library never frees them and does not keep them after
 *     the work enqueued by the call has completed.  A pointer documented "nullable" may be NULL.
 *   - token buffers are read in aligned 16-byte units: the unit that holds a prompt's first token and
 *     the unit that holds its last token are loaded whole, so up to 12 bytes before and after the
 *     tokens a call names may be read (never written, never interpreted).  An aligned 16-byte unit
 *     never crosses a page, so this is safe for any pointer into an allocation; prompts may start
 *     at any 4-byte boundary.
 *   - prompts are int32 token strings in CSR form: prompt i is tokens[offsets[i] .. offsets[i+1]);
 *     offsets are int64, non-decreasing, offsets[0] may be non-zero.
 *   - `stream` is a cudaStream_t passed as void* (NULL = the default stream).  Work is enqueued on it;
 *     entry points return without waiting for the device, except where stated.
 *   - the return value reports argument and launch errors found on the host.  Conditions found on the
 *     device (capacity exhausted, budget too small, a bounded wait that ran out) are recorded in a
 *     status word inside the tree and returned by rt_sync_status(); nothing traps or aborts.
 *   - a tree may be used from one stream at a time; calls on one tree must not overlap on the GPU.
 *   - all arithmetic is integer; there is no floating point on this path.
 */
#ifndef KLPM_H_
#define KLPM_H_

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef int32_t rt_status;
enum {
    RT_OK = 0,
    RT_ERR_INVALID = -1,   /* bad argument (null pointer, negative count, k < 1, ...) */
    RT_ERR_CAPACITY = -2,  /* node, token-pool or clock capacity of the tree exhausted */
    RT_ERR_BUDGET = -3,    /* the KV budget cannot hold a prompt even after evicting everything evictable */
    RT_ERR_LIMIT = -4,     /* a bounded device-side wait or probe loop ran out */
    RT_ERR_CUDA = -5,      /* a CUDA runtime call failed */
    RT_ERR_TOO_LARGE = -6  /* a size is above a fixed limit of the entry point (klpm_select_noalloc) */
};

enum { KLPM_POLICY_FCFS = 0, KLPM_POLICY_LPM = 1, KLPM_POLICY_KLPM = 2 };

typedef struct rt_tree rt_tree; /* opaque; owned by the library from rt_build/rt_create until rt_destroy */

typedef struct {
    int32_t vocab;            /* informational: token ids are expected in [0, vocab) */
    int64_t max_nodes;        /* capacity in tree nodes (every processed prompt adds at most 2) */
    int64_t max_pool_tokens;  /* capacity of the append-only int32 token pool: the uncached tokens of every
                                 stored prompt plus up to 8 tokens of alignment padding per prompt */
    int64_t budget_tokens;    /* KV-cache budget in tokens with LRU eviction; 0 = unbounded */
    int64_t max_clock;        /* capacity in processed prompts over the tree's life; 0 = max_nodes */
} rt_config;

typedef struct {
    int32_t policy;      /* KLPM_POLICY_* ; LPM = every pick is a longest-match pick */
    int32_t k;           /* Algorithm 1's k (>= 1); used by KLPM only */
    int64_t c_num;       /* c_attn = c_num / c_den (Definition 2); times are in units of 1/c_den tick */
    int64_t c_den;       /* >= 1 */
    int64_t start_tick;  /* tick at which processing starts (R of the "previous" query for the first pick) */
} klpm_params;

/* ---- radix tree of cached prompts (RadixAttention as Section 1 describes it: processed prompts are
 *      kept in a radix tree so that later prompts reuse their shared prefixes; under a fixed memory
 *      budget the least recently used entries are evicted) ---- */

/* Create an empty tree.  Synchronous (allocates device memory). */
rt_status rt_create(const rt_config* cfg, rt_tree** out);

/* Create a tree and store n_prompts prompts in it, as if processed one after the other in index
 * order (prompt i is stamped with logical clock i+1 for LRU).  Equivalent to rt_create + rt_insert. */
rt_status rt_build(const int32_t* d_tokens, const int64_t* d_offsets, int32_t n_prompts,
                   const rt_config* cfg, void* stream, rt_tree** out);

/* Store n more prompts, one after the other in index order: each is matched against the tree as it
 * stands, a node boundary is put at its match end, its uncached tail is appended as a new leaf, the
 * logical clock advances by one, and (with a budget) least-recently-used leaves are evicted first to
 * make room.  d_new_tokens (nullable, int32[n]) receives |x_i| - match length at its own insertion.
 * If the device runs out of capacity the prompts before the failing one stay inserted and the tree
 * stays valid; the condition is reported by rt_sync_status.
 * When d_new_tokens is NULL, the tree has no budget and n >= 64, the prompts are inserted concurrently
 * in rounds instead (same resulting set of cached prefixes and node boundaries; node numbering may
 * differ from run to run).  The rounds run on the device (the later ones inside one cooperative kernel
 * whose grid-wide waits are bounded like every other wait); the call does not wait for them. */
rt_status rt_insert(rt_tree* tree, const int32_t* d_tokens, const int64_t* d_offsets, int32_t n,
                    int32_t* d_new_tokens, void* stream);

/* Batched longest-prefix match (Section 1.3 defines overlap(x, y); Section 1 has the tree matched
 * against each incoming prompt): d_match_len[i] = max over cached prompts y of overlap(q_i, y) = the longest
 * prefix of query i that lies on a root path of the tree, counted token by token (partial edges
 * count).  Read-only on the tree.  d_term_node / d_term_off (nullable, int32[nq]) receive where the
 * match ended: the node whose edge holds the last matched token (0 = root when nothing matched) and
 * how many tokens of that edge matched. */
rt_status rt_match_batch(const rt_tree* tree, const int32_t* d_q_tokens, const int64_t* d_q_offsets,
                         int32_t nq, int32_t* d_match_len, int32_t* d_term_node, int32_t* d_term_off,
                         void* stream);

/* What a batched match knows about one query beyond its match length (where in the token pool the match ended,
 * the run of pool tokens around it, the query token that follows), kept so that the scheduling loop can start from
 * the match instead of walking every query again.  Opaque: 32 bytes per query, 16-byte aligned. */
typedef struct { int64_t w[4]; } klpm_match_state;

/* rt_match_batch that also fills d_state (nullable, klpm_match_state[nq]) for a later klpm_run_ex on the same
 * queries.  The records are good for that one purpose while (a) the tree has not been changed by any call since
 * (rt_insert, klpm_replay, klpm_run*, rt_rollback), (b) d_q_tokens / d_q_offsets / nq are the ones passed here
 * and their contents have not changed, and (c) no later rt_match_batch_ex with a state buffer was made on this
 * tree.  On a tree with a budget the records are written but klpm_run_ex does not use them (the tree changes
 * under the loop).  Batches of 2,048 queries or more are taken in an order bucketed by first token, for which
 * the first such call allocates scratch (synchronously); results do not depend on the order. */
rt_status rt_match_batch_ex(rt_tree* tree, const int32_t* d_q_tokens, const int64_t* d_q_offsets, int32_t nq,
                            int32_t* d_match_len, int32_t* d_term_node, int32_t* d_term_off,
                            klpm_match_state* d_state, void* stream);

/* Counters of the tree (synchronises the stream the tree was last used on).  Any pointer may be NULL.
 * n_nodes: live nodes, root excluded; n_tokens: tokens held by live nodes; clock: prompts processed;
 * evictions: leaves evicted so far; pool_used: tokens appended to the pool so far. */
rt_status rt_stats(rt_tree* tree, int64_t* n_nodes, int64_t* n_tokens, int64_t* clock,
                   int64_t* evictions, int64_t* pool_used);

/* A second, independent tree with the same capacity and the same content (device-to-device copies enqueued on
 * `stream`; the allocation itself is synchronous).  Several clones can be scheduled at the same time on
 * different streams, e.g. to try several values of k on one stream of queries (the back-testing the paper
 * suggests for choosing k, Section 4.2). */
rt_status rt_clone(rt_tree* tree, void* stream, rt_tree** out);

/* Remember the tree as it is now (device-to-device copies of the node arrays, the child table and the
 * counters; the token pool is append-only and is not copied).  One checkpoint per tree; a later call replaces it. */
rt_status rt_checkpoint(rt_tree* tree, void* stream);

/* Put the tree back to its last checkpoint, undoing every insertion and eviction since.
 * RT_ERR_INVALID if there is no checkpoint. */
rt_status rt_rollback(rt_tree* tree, void* stream);

/* Wait for `stream` and return the tree's device-side status word (RT_OK or the first error recorded). */
rt_status rt_sync_status(rt_tree* tree, void* stream);

/* A number that says which device-side check recorded the status word (0 if none did): 101/104 a child entry
 * that should exist was not found, 102/112 a bounded wait of the scheduling loop / of the concurrent insertion ran out, 103/105/107 an internal
 * prediction did not hold, 106 a child lookup probed the whole table, 108 an order entry that is not a query
 * (or a prompt with a negative length), 109 a prompt too long for the hit-rate score.  A debugging aid;
 * synchronises like rt_stats. */
rt_status rt_status_detail(rt_tree* tree, int32_t* detail);

/* Free the tree and everything it owns.  Synchronous. */
rt_status rt_destroy(rt_tree* tree);

/* ---- scheduling (Algorithm 1 "k-LPM"; FCFS and LPM of Section 1 as its k = 1 and k = infinity limits) ---- */

/* One scheduling decision as a pure function of its inputs.  Among the queries with d_waiting[i] != 0:
 *   - oldest-first pick (FCFS; or KLPM when pick_counter % k == 0): the query with the smallest
 *     (arrival, index);
 *   - longest-match pick (LPM; or KLPM otherwise): the query with the largest d_match_len, ties to the
 *     smallest (arrival, index).
 * d_pick (int32[1]) receives the index, or -1 if no query is waiting.  Uses library-owned scratch that
 * is allocated on the first call on each device and shared by every later call on it: calls that overlap
 * on the GPU (different streams, no dependency) race on it -- issue them on one stream or order them
 * with events.  The same holds for klpm_select_topk. */
rt_status klpm_select(const int32_t* d_match_len, const int64_t* d_arrival, const uint8_t* d_waiting,
                      int32_t nq, int64_t pick_counter, const klpm_params* params, int32_t* d_pick,
                      void* stream);

/* The kk best longest-match candidates of one snapshot of the queue, best first: d_out[j] (int32[kk]) is the
 * waiting query that ranks j-th by (largest d_match_len, then smallest arrival, then smallest index), or -1
 * when fewer than kk queries are waiting.  1 <= kk <= 64.  These are the k-1 picks that follow an oldest-first
 * pick in Algorithm 1 *if match lengths did not move*; they do move when a processed prompt extends the cache
 * (klpm_run accounts for that, this call does not).  Uses library-owned scratch allocated on first use. */
rt_status klpm_select_topk(const int32_t* d_match_len, const int64_t* d_arrival, const uint8_t* d_waiting,
                           int32_t nq, int32_t kk, int32_t* d_out, void* stream);

/* klpm_select for callers that must not allocate device memory.  (The paper has no counterpart of this
 * entry point; it exists for how the library gets embedded, not for the method.)
 *
 * Some hosts of this library cannot let it call cudaMalloc: a serving engine that hands the whole GPU to
 * its own memory pool at start-up and treats any later allocation as a bug, code that runs where an
 * allocation would force a device-wide synchronisation in the middle of a latency-critical scheduling
 * tick, or a process whose memory accounting must stay fixed after initialisation.  klpm_select keeps the
 * per-block partial results of its reduction in a buffer it allocates on first use; this variant keeps
 * them in a small fixed array that is part of the library image, so it never allocates or frees anything.
 *
 * Same arguments, same result as klpm_select (bit for bit), with these differences:
 *   - nq must not exceed KLPM_SELECT_NOALLOC_MAX_QUERIES; a larger nq returns RT_ERR_TOO_LARGE (and says so
 *     on stderr) without launching anything.
 *   - the fixed array is 4 KiB plus a counter.  Every GPU on which the library is loaded holds it until the
 *     process exits, whether or not this entry point is ever called.
 *   - the first call on each device looks up the array's device address (with that device current) and
 *     remembers it; make that first call outside any stream capture.
 *   - all calls on a device share the one array, and it keeps whatever the previous call left in it; each
 *     call clears the counter it relies on before its kernel runs.  Two calls that overlap on the GPU
 *     (different streams, no dependency between them) race on the array and may both return wrong picks:
 *     issue calls on one stream, or order them with events. */
#define KLPM_SELECT_NOALLOC_MAX_QUERIES (1 << 22)
rt_status klpm_select_noalloc(const int32_t* d_match_len, const int64_t* d_arrival, const uint8_t* d_waiting,
                              int32_t nq, int64_t pick_counter, const klpm_params* params, int32_t* d_pick,
                              void* stream);

/* Definition 2 along a given processing order: for j = d_order[0], d_order[1], ...:
 *   m = longest prefix of x_j in the tree; uncached = |x_j| - m;
 *   R_j = max(R_prev, t_j) + (c_den + c_num |x_j|) * uncached;  TTFT_j = R_j - t_j;
 * then x_j is stored in the tree (as rt_insert does).  Outputs are indexed by query: d_uncached
 * (int32[n_queries]), d_ttft (int64[n_queries]), d_completion (nullable, int64[n_queries]); entries of
 * queries that are not in d_order are left untouched.  A query may appear in d_order once.  An entry outside
 * [0, n_queries), or one that names a query for the second time, stops the replay there: nothing of it is read or
 * written, the queries before it stay processed, and the status word reports RT_ERR_INVALID (detail 108).
 * The replay runs through the same device loop as klpm_run, with the order given instead of picked: every query
 * is matched once, a processed prompt re-matches only the queries tied with it, and the tree is written at the
 * end (what klpm_run says about capacity holds here too).  The debug setting "run_one_by_one" selects the plain
 * form instead: one CTA that walks, charges and stores one prompt after the other. */
rt_status klpm_replay(rt_tree* tree, const int32_t* d_order, int32_t n_order, const int32_t* d_q_tokens,
                      const int64_t* d_q_offsets, const int64_t* d_arrival, int32_t n_queries,
                      const klpm_params* params, int32_t* d_uncached, int64_t* d_ttft,
                      int64_t* d_completion, void* stream);

/* The whole scheduling loop on the device (Algorithm 1 with Definitions 1 and 2): until all n queries
 * are processed -- wait for the next arrival if nobody is waiting; pick by the policy among the queries
 * that have arrived (match lengths are those against the tree at that moment, which includes every
 * query processed so far); charge the pick by Definition 2; store it in the tree (LRU eviction under
 * the budget).  d_order[c] (int32[n]) = query processed at decision c; the other outputs are as in
 * klpm_replay.  The pick counter of KLPM never resets.
 * On a tree without a budget nothing is ever evicted, so a query's match length changes only when a prompt is
 * processed whose own match ended at the same place and goes on with the same token; the loop then keeps every
 * query's match state itself and stores all processed prompts in the tree at the end, concurrently (as rt_insert
 * does for large batches) -- same outputs, same cached prefixes and node boundaries.  A tree too small for the
 * queue still gets every output (they do not depend on the tree's capacity) while the status word reports
 * RT_ERR_CAPACITY and the tree, still valid, holds only part of the queue.  Like every other call, klpm_run only
 * enqueues work (the first call for a queue of a given size also allocates scratch, which synchronises). */
rt_status klpm_run(rt_tree* tree, const int32_t* d_q_tokens, const int64_t* d_q_offsets,
                   const int64_t* d_arrival, int32_t n, const klpm_params* params, int32_t* d_order,
                   int32_t* d_uncached, int64_t* d_ttft, int64_t* d_completion, void* stream);

/* Which loop the last klpm_run / klpm_run_ex on this tree took: 0 = none yet, 1 = one decision at a time on the
 * tree itself (trees with a budget), 2 = the grouped loop (trees without a budget; see klpm_run).  Both give the
 * same outputs.  The debug setting "run_one_by_one" makes trees without a budget take loop 1 too. */
int32_t klpm_run_path(const rt_tree* tree);

/* What the grouped loop of the last klpm_run / klpm_run_ex on this tree did (zeros if it has not run): out16[0] decisions
 * taken by a careful step, [1] groups dissolved by the whole CTA, [2] scans after an eviction of a leaf with queries
 * parked in it, [3] queries that fell back out of evicted leaves, [4] evictions, [5..7] clock cycles spent in tree
 * updates, in those scans, in dissolves by the whole CTA; once everybody had arrived: [8] CTA-wide batches tried,
 * [9] committed, [10] decisions they made, [11] warp-wide steps committed, [12] decisions they made, [13] decisions
 * made one at a time, [14..15] clock cycles in CTA-wide and in warp-wide attempts.  A debugging aid; synchronises
 * like rt_stats. */
rt_status rt_debug_counters(rt_tree* tree, int64_t* out16);

/* Settings for tests and debugging; process-wide, read when a later call is made; value < 0 restores the default.
 *   "run_one_by_one"   1: klpm_run takes the one-decision-at-a-time loop on every tree (default 0)
 *   "fast_max_blocks"  grouped loop: the most tournament leaf blocks it may use (default 0 = 8,192)
 *   "fast_smem_kb"     grouped loop: the shared memory it may use, in KiB (default 0 = 224)
 *   "wait_limit_ns"    one-by-one loop: how long a CTA waits for another before it gives up, records
 *                      RT_ERR_LIMIT (detail 102) and lets every CTA return (default 5e9; 0 = give up at once)
 * RT_ERR_INVALID for an unknown name. */
rt_status klpm_debug_set(const char* name, int64_t value);

/* klpm_run with two variants of the longest-match pick (the oldest-first picks are not affected):
 *   d_tie_priority (nullable, int64[n]): among waiting queries with the same score the one with the smallest
 *     priority wins; arrival and index decide only among equal priorities.  With priorities drawn uniformly at
 *     random by the caller this is the tie-breaking the paper assumes for LPM (footnote in Section 4.2).
 *   score_mode 0: the score is the match length in tokens (Algorithm 1 as klpm_run reads it).
 *   score_mode 1: the score is the prompt's hit rate match / length (0 for an empty prompt) -- the other
 *     reading of "maximizes the prefix cache hit rate".  It is held as floor(match * 2^31 / length), which
 *     orders prompts exactly as the rates do while no prompt is longer than 46,340 tokens (46,340^2 < 2^31);
 *     a longer prompt makes the status word report RT_ERR_INVALID (detail 109), and ties may then be wrong.
 *   d_match_state (nullable): the records rt_match_batch_ex wrote for exactly these queries on this tree, if no
 *     call has changed the tree since.  The loop then starts from that match; without them it matches every
 *     query itself first (the same kernel), so the outputs are identical.  RT_ERR_INVALID is returned, and nothing
 *     is enqueued, if the records are not the ones the last rt_match_batch_ex on this tree wrote for these
 *     arguments or the tree has changed since; records the caller has overwritten are caught on the device
 *     (status RT_ERR_INVALID, detail 110).
 * klpm_run(...) is klpm_run_ex(..., NULL, 0, NULL, ...). */
rt_status klpm_run_ex(rt_tree* tree, const int32_t* d_q_tokens, const int64_t* d_q_offsets,
                      const int64_t* d_arrival, int32_t n, const klpm_params* params,
                      const int64_t* d_tie_priority, int32_t score_mode,
                      const klpm_match_state* d_match_state, int32_t* d_order,
                      int32_t* d_uncached, int64_t* d_ttft, int64_t* d_completion, void* stream);

/* Batch size B (Section 2.1: the order is cut into consecutive bins of B queries, and a query is finished when
 * the last query of its bin is).  d_order (int32[n_order]) is a processing order and d_completion (int64, indexed
 * by query) its batch-size-one completion times, as klpm_run / klpm_replay produce them; d_completion_b and
 * d_ttft_b (int64, indexed by query; entries of queries not in d_order are left untouched) receive the
 * completion time of the query's bin and that minus its arrival.  The per-query arrays have n_queries entries;
 * a decision whose own entry of d_order, or the last entry of its bin, lies outside [0, n_queries) is skipped
 * (nothing is read or written for it) and counted in d_n_skipped (nullable, int32[1], set by the call).
 * batch_size >= 1; the outputs must not alias the inputs. */
rt_status klpm_batch_times(const int32_t* d_order, int32_t n_order, const int64_t* d_arrival,
                           const int64_t* d_completion, int32_t n_queries, int32_t batch_size,
                           int64_t* d_ttft_b, int64_t* d_completion_b, int32_t* d_n_skipped, void* stream);

/* Many independent queues at once under the cache model the paper's analysis uses: only the previously processed
 * prompt is cached (Definition 2 as printed; Section 2.1), so the match of a waiting prompt is its overlap with the
 * prompt processed last and nothing is kept between queues.  This is the setting of the worked example of
 * Section 4.2 and of Theorem 2; a Monte-Carlo over the random arrival orders of Definition 3 is one call.
 *   Queue r consists of prompts d_queue_offsets[r] .. d_queue_offsets[r+1]-1 (int32[n_queues+1], non-decreasing) of the
 *   CSR arrays d_tokens / d_offsets; d_arrival and d_tie_priority (nullable) are indexed like the prompts.  Each queue is
 *   scheduled on its own by params (FCFS / LPM / k-LPM, c_attn, start_tick), starting with an empty cache: wait for
 *   the next arrival if nobody is waiting; oldest-first pick = smallest (arrival, index); longest-match pick =
 *   largest overlap with the prompt processed last, ties to the smallest priority, then (arrival, index); charge by
 *   Definition 2.  d_order[d_queue_offsets[r] + c] = index WITHIN queue r of the prompt processed at its decision c;
 *   d_uncached, d_ttft, d_completion (nullable) are indexed like the prompts.
 * A queue of more than KLPM_LAST_ONLY_MAX_QUEUE prompts is left untouched and counted in d_n_skipped (nullable,
 * int32[1], set by the call).  One warp runs one queue; no scratch memory, no tree. */
#define KLPM_LAST_ONLY_MAX_QUEUE 1024
rt_status klpm_run_last_only_batch(const int32_t* d_tokens, const int64_t* d_offsets, const int64_t* d_arrival,
                                   const int64_t* d_tie_priority, const int32_t* d_queue_offsets, int32_t n_queues,
                                   const klpm_params* params, int32_t* d_order, int32_t* d_uncached,
                                   int64_t* d_ttft, int64_t* d_completion, int32_t* d_n_skipped, void* stream);

/* Version of the ABI (bumped when a signature changes). */
int32_t klpm_abi_version(void);

#ifdef __cplusplus
}
#endif
#endif /* KLPM_H_ */
