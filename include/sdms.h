/*
 * sdms - draft-token construction for multi-sample speculative decoding on one
 * NVIDIA B200 (sm_100a).  Method: arXiv 2503.05330, section "Method" and
 * Algorithm 1 ("Self-Consistency Draft Token Generation").
 *
 * A context holds G independent prompts with N reasoning paths each.  Every
 * decode step the caller
 *   1. asks for one draft per path            (sdms_build_drafts),
 *   2. lets its model verify the drafts       (not part of this library),
 *   3. reports the sampled tokens             (sdms_accept, which can also
 *      append them; or sdms_append directly).
 *
 * Conventions that hold for every entry point
 *   - "d_" pointers are DEVICE pointers owned by the caller; everything else is
 *     host memory.  The library allocates no device memory: all of its device
 *     state lives in the caller's workspace (sdms_workspace_bytes bytes, 256-byte
 *     aligned).  The context is a small host object.
 *   - Path index p = g * paths_per_group + n.  Rows of per-path arrays are
 *     contiguous ([P][x], row-major, int32/float32).
 *   - `stream` is a cudaStream_t passed as void* (NULL = default stream).  Calls
 *     only enqueue work; none waits for the device except sdms_create,
 *     sdms_get_status and sdms_profile_read.
 *   - Return value: 0 on success, a negative SDMS_ERR_* otherwise.  Nothing
 *     throws, aborts or traps.  Conditions only visible on the device set bits
 *     in a device status word (SDMS_STATUS_*); the offending item is clamped or
 *     skipped as described per call and the rest of the batch proceeds.
 *   - A context is not thread-safe; distinct contexts are independent.
 */
#ifndef SDMS_H_
#define SDMS_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define SDMS_OK                      0
#define SDMS_ERR_INVALID_ARG        -1
#define SDMS_ERR_WORKSPACE_TOO_SMALL -2
#define SDMS_ERR_CUDA               -3
#define SDMS_ERR_BAD_STATE          -4
#define SDMS_ERR_TOO_LARGE          -5

/* Device status bits (sticky until sdms_get_status clears them). */
#define SDMS_STATUS_BAD_COUNT      0x01u /* append count outside [0, row width]: clamped          */
#define SDMS_STATUS_CAPACITY       0x02u /* sdms_append beyond the path capacity: truncated       */
#define SDMS_STATUS_BAD_TOKEN      0x04u /* token outside [0, vocab): path keeps what came before */
#define SDMS_STATUS_BAD_LOGPROB    0x08u /* NaN logprob: stored as probability 0                  */
#define SDMS_STATUS_INDEX_FULL     0x10u /* n-gram table had no free bucket (cannot happen with the sized workspace) */
#define SDMS_STATUS_MATCH_OVERFLOW 0x20u /* match workspace exhausted: the affected paths get draft_len 0 */
#define SDMS_STATUS_SEARCH_FALLBACK 0x40u /* search_mode 2: a path had too many matches for shared memory (more than about
                                            24576 / (11 * max_draft_len)) and the table area had no room: greedy draft */
#define SDMS_STATUS_TIMEOUT        0x80u /* a bounded wait inside a kernel ran out (never expected): the build's matches are incomplete */
#define SDMS_STATUS_TABLES_FULL    0x100u /* sdms_get_beams: the table area of the workspace (wide_table_bytes) did not hold
                                             every path's node tables; the paths left out have no beam */

#define SDMS_MAX_K      16   /* largest supported k_max           */
#define SDMS_MAX_DRAFT  32   /* largest supported max_draft_len   */
#define SDMS_MAX_PATHS_PER_GROUP 1024
#define SDMS_MAX_DAG_NODES 32  /* largest dag_nodes_per_layer      */
#define SDMS_MAX_DAG_EDGES 16  /* largest dag_edges_per_node       */
#define SDMS_MAX_BEAMS  8      /* largest max_beams                 */

typedef struct sdms_ctx sdms_ctx;

typedef struct {
  uint32_t struct_size;          /* sizeof(sdms_config), for ABI checks                       */
  int32_t  num_groups;           /* G: independent prompts; matching never crosses prompts    */
  int32_t  paths_per_group;      /* N: parallel samples of one prompt (the paper's N)         */
  int32_t  capacity;             /* L: tokens kept per path; a path at L builds no more drafts
                                    but is still searched by the others                      */
  int32_t  vocab;                /* V: tokens must lie in [0, V)                              */
  int32_t  k_max;                /* largest query suffix length that will be asked for        */
  int32_t  max_draft_len;        /* D: the paper's maximum draft token length                 */
  int32_t  max_append;           /* most tokens a path may gain per sdms_accept commit        */
  int32_t  dag_nodes_per_layer;  /* B: nodes kept per layer by sdms_get_dag, 0 = no export     */
  int32_t  dag_edges_per_node;   /* Ke: out-edges kept per exported node                      */
  int32_t  search_mode;          /* 0: walk to the best successor of the current node;
                                    1: best node of each layer regardless of the previous one;
                                    2: not the paper's greedy walk but the path of the DAG with the
                                       largest sum of node weights (its introduction asks for the
                                       highest-likelihood sequence): best(d,v) = w(d,v) + max over
                                       successors of best(d+1,.), summed from the path's end; the
                                       walk follows the largest best(), ties to the smaller token.
                                       DAG pool only.  Paths with more matches than shared memory
                                       takes are searched by one more launch after the build, over
                                       node tables in the workspace's table area (wide_table_bytes);
                                       only if that is switched off or full do they keep the mode-0
                                       draft and raise SDMS_STATUS_SEARCH_FALLBACK               */
  float    alpha;                /* Eq. 5 mixing weight; the paper's experiments use 1        */
  int64_t  match_capacity;       /* match-list entries in the workspace, 0 = default          */
  int32_t  epsilon;              /* Eq. 4 edit-distance tolerance of the suffix match: 0 (exact)
                                    or 1.  With 1 the index is not used: small prompts (N*L <= 131072
                                    tokens and G*N*N*L <= match_capacity) are scanned by the single-launch
                                    build, larger ones in two passes (count, then fill)             */
  int32_t  pool_mode;            /* draft pool: 0 = weighted DAG (the method); the weaker pools of the
                                    paper's ablation: 1 = tree (merge identical prefixes only),
                                    2 = list (no merging: the heaviest single candidate)            */
  int32_t  max_matches_per_path; /* R: 0 = every match counts, as in Eq. 3.  R > 0: of the matches a
                                    query path has in ONE other path only the R with the largest end
                                    positions (the most recent ones) enter the pool - defined by
                                    position, so the result does not depend on the order in which
                                    matches are found.  Bounds the pool at (N-1)*R candidates per query:
                                    the paper's experiments stress a small candidate set and its
                                    limitations the cost of aggregating over many paths           */
  int32_t  max_beams;            /* largest number of drafts per path that sdms_get_beams will be asked for
                                    (0 = the call is not used; at most SDMS_MAX_BEAMS)               */
  int64_t  wide_table_bytes;     /* workspace set aside for node tables in global memory.  Two users: on
                                    prompts too large for the single-launch build, queries with more than 32
                                    matches are aggregated by all SMs together; and sdms_get_beams (max_beams
                                    > 0) and search_mode 2.  A slot costs 40 + 16 * max(max_beams, 1) bytes and a path with M matches
                                    needs between 2.5 and 5 * M * D slots (half of that for the beams).  0 = default (room for every position
                                    matching every query of its prompt, but at most 320 MiB), -1 = none.  A build
                                    whose queries need more falls back to one thread block for those that
                                    did not fit, with the same results                                    */
  int32_t  index_max_n;          /* n-gram lengths the index keeps tables for: 1..index_max_n (0 = k_max, every
                                    length that can be asked for).  A query with k > index_max_n looks up its last
                                    index_max_n tokens instead: that bucket lists a superset of the k-gram's
                                    occurrences, which are verified against all k tokens, or hands the query to the
                                    scan.  Fewer tables: 64 bytes less per token and dropped length, and fewer
                                    inserts per appended token; more queries scanned.  Results are the same      */
  int32_t  reserved1;            /* must be 0 */
} sdms_config;

/* Bytes of device workspace a context with this configuration needs (host only,
 * no CUDA call). */
int sdms_workspace_bytes(const sdms_config* cfg, size_t* bytes);

/* Create a context over caller-owned device memory.  Zero-fills the workspace on
 * the default stream and waits for it.  Starts with all paths empty. */
int sdms_create(const sdms_config* cfg, void* d_workspace, size_t bytes, sdms_ctx** out);

/* Forget every token (same effect as destroying and re-creating the context). */
int sdms_reset(sdms_ctx* ctx, void* stream);

/* Frees the host object only. */
int sdms_destroy(sdms_ctx* ctx);

/*
 * State update ("Dynamic Draft Pool Construction": the partial sequences
 * y_i^{1:t} grow every step).  Path p gains d_tokens[p][0 .. d_counts[p]) with
 * the model's log-probability of each of those tokens (the p_theta of Eq. 5 is
 * exp(logprob), stored as round_half_even(exp(logprob) * 2^30) in [0, 2^30]).
 * Rows are `row_width` wide (1 <= row_width; any width, e.g. a prefill chunk).
 * The new positions' n-grams (n = 1..k_max) enter the prompt's hash tables.
 * Clamping: count outside [0, row_width] -> BAD_COUNT; beyond capacity ->
 * CAPACITY, truncated; token outside [0, V) -> BAD_TOKEN, the path keeps the
 * tokens before it.
 */
int sdms_append(sdms_ctx* ctx, const int32_t* d_tokens, const float* d_logprobs,
                const int32_t* d_counts, int32_t row_width, void* stream);

/*
 * One draft per path (Algorithm 1):
 *   query      the last k tokens of path i                       (1 <= k <= k_max)
 *   match      Eq. 3: every end position e in every other path j of the same
 *              prompt with y_j[e-k+1..e] equal to the query and e <= len_j - 2
 *              With epsilon = 1 ("Fuzzy Suffix Matching", Eq. 4): every e <= len_j - 2
 *              at which some window of k-1, k or k+1 tokens (at least one) ends
 *              within edit distance 1 of the query; each e counts once.  The walk
 *              then starts from a virtual root in front of all matched windows.
 *              With max_matches_per_path = R > 0 only the R matches with the largest e
 *              per other path j are kept.
 *   candidates the up to D tokens that follow each match
 *   DAG        layer d = distinct d-th followers; edge (u,v) between layers d-1
 *              and d accumulates S = sum of fixed-point probabilities of v and
 *              cnt = number of instances; Eq. 5 weight = alpha*S/2^30 + (1-alpha)*cnt
 *              evaluated in binary64; a node's score is Eq. 5 on its summed in-edges
 *   search     greedy walk from the query's last token, ties to the smaller token
 *              id, until D tokens or a node without successor.
 * Outputs: d_draft_tok [P][D] (unused entries -1), d_draft_len [P],
 * d_draft_score [P][D] = score of each chosen node, d_draft_edge_w [P][D] =
 * weight of the edge taken (unused 0; either float array may be NULL).
 * Paths shorter than k, full paths and paths without a match get draft_len 0.
 * Read-only with respect to the path histories.
 */
int sdms_build_drafts(sdms_ctx* ctx, int32_t k, int32_t* d_draft_tok, int32_t* d_draft_len,
                      float* d_draft_score, float* d_draft_edge_w, void* stream);

/*
 * The same with a suffix length that backs off: every path uses the longest k in
 * [1, k_hi] for which it has at least one match (the paper names k but never fixes
 * it; longer suffixes give fewer, more specific candidates).  d_used_k [P] (may be
 * NULL) receives that k, 0 for paths without a draft.  One launch on prompts small
 * enough for the single-launch build (N*L <= 131072 tokens and G*N*N*L <=
 * match_capacity); on larger ones one round of launches per suffix length, longest
 * first (a path that has found matches keeps them; sdms_debug_read_query_modes then
 * reports 3 for it).  With epsilon = 1 a path that gets down to k = 1 matches every
 * position of its prompt (one substitution away from any token): on such a large
 * prompt that is more than a match list holds, the path gets no draft and
 * SDMS_STATUS_MATCH_OVERFLOW is raised.
 */
int sdms_build_drafts_backoff(sdms_ctx* ctx, int32_t k_hi, int32_t* d_draft_tok, int32_t* d_draft_len,
                              float* d_draft_score, float* d_draft_edge_w, int32_t* d_used_k, void* stream);

/*
 * "Draft acceptance": d_accept_len[p] = longest t <= d_draft_len[p] with
 * d_draft_tok[p][0..t) == d_sampled[p][0..t), d_sampled being [P][D+1] tokens
 * sampled by the model at the draft positions plus one more.
 * If d_sampled_logprobs ([P][D+1]) is not NULL the call also commits: path p
 * appends d_sampled[p][0 .. min(tau_p + 1, max_append)) exactly as sdms_append
 * would, except that reaching capacity silently truncates.
 */
int sdms_accept(sdms_ctx* ctx, const int32_t* d_draft_tok, const int32_t* d_draft_len,
                const int32_t* d_sampled, const float* d_sampled_logprobs,
                int32_t* d_accept_len, void* stream);

/*
 * One decode step in one call: sdms_accept with commit on the drafts that
 * d_draft_tok / d_draft_len hold on entry (the previous call's output), then
 * sdms_build_drafts(k) into the same arrays ("Draft acceptance" followed by
 * Eq. 3, Eq. 5 and the greedy search on the extended histories).  The results
 * are identical to those two calls made one after the other.
 * d_sampled and d_sampled_logprobs ([P][D+1]) are both required.
 * When a prompt's paths fit one thread-block cluster (paths_per_group <= 16, the
 * single-launch build applies and the device can hold the clusters of all prompts
 * at once) the step is ONE kernel launch: the paths of a prompt commit, meet at a cluster
 * barrier, and build (search_mode 2 adds the launch that searches the paths with many
 * matches).  Otherwise the call issues the separate launches.
 * sdms_step_is_single_launch reports which (1 / 0).
 */
int sdms_step(sdms_ctx* ctx, int32_t k, const int32_t* d_sampled, const float* d_sampled_logprobs,
              int32_t* d_accept_len, int32_t* d_draft_tok, int32_t* d_draft_len, float* d_draft_score,
              float* d_draft_edge_w, void* stream);
/* sdms_step with the suffix length backing off as in sdms_build_drafts_backoff. */
int sdms_step_backoff(sdms_ctx* ctx, int32_t k_hi, const int32_t* d_sampled, const float* d_sampled_logprobs,
                      int32_t* d_accept_len, int32_t* d_draft_tok, int32_t* d_draft_len, float* d_draft_score,
                      float* d_draft_edge_w, int32_t* d_used_k, void* stream);
int sdms_step_is_single_launch(sdms_ctx* ctx, int32_t* yes);
/* Thread blocks (= consecutive paths of one prompt) that share the scan of their prompt in the single-launch
 * build: 1 = every query scans for itself (also on contexts that do not take that build). */
int sdms_build_cluster_size(sdms_ctx* ctx, int32_t* paths);

/*
 * Sliding window for runs longer than the capacity (the paper's runs end long
 * before any limit; this call is not part of its method).  Path p forgets all but
 * its newest d_keep[p] tokens: they move to the front of its store, the path has
 * room again, and every later call sees exactly the shorter history, as if only
 * those tokens had ever been appended.  d_keep[p] >= the path's length changes
 * nothing; d_keep[p] < 0 raises SDMS_STATUS_BAD_COUNT and changes nothing.
 * The n-gram tables of every prompt with a trimmed path are emptied and filled
 * again from the histories (three launches; cost proportional to the prompt's
 * tokens * k_max), so call it every few hundred steps with a generous cut, not
 * every step.  Drafts built before the call refer to the old positions: build
 * again before the next sdms_accept.
 */
int sdms_trim(sdms_ctx* ctx, const int32_t* d_keep, void* stream);

/*
 * Zero-copy callers.  The per-step arrays of sdms_step / sdms_accept / sdms_build_drafts
 * (sampled tokens and logprobs, drafts, accept lengths) may live in page-locked
 * host memory that is mapped into the device's address space: the kernel then
 * reads its inputs and writes its results over the host link itself and no copy
 * is enqueued around the call (a step's inputs and outputs are about 2 KB).
 * This call checks that host_ptr is such memory (cudaHostAlloc, or registered
 * with the mapped flag) and returns in *device_ptr the address to pass instead;
 * SDMS_ERR_INVALID_ARG for pageable, device or unknown memory.  The host may read
 * the results after the stream (or an event recorded after the call) has completed.
 */
int sdms_host_pointer(const void* host_ptr, void** device_ptr);

/* ---- inspection (used by the parity tests; not part of a decode step) ------- */

/* Matches of the last sdms_build_drafts: d_offsets [P+1] (exclusive prefix sums)
 * and d_gpos = global positions j*L + e of every match, grouped per query path,
 * in no particular order inside a group.  At most `cap` positions are written;
 * d_offsets always holds the true counts. */
int sdms_get_matches(sdms_ctx* ctx, int32_t* d_offsets, int32_t* d_gpos, size_t cap, void* stream);

/* DAG export of the last sdms_build_drafts (needs dag_nodes_per_layer > 0).  The
 * call aggregates the same matches once more and this time ranks and writes out
 * the nodes and edges; the histories must not have changed since that build
 * (an append or a committing accept in between gives SDMS_ERR_BAD_STATE).
 * Layer index d-1 for d = 1..D.  Per layer the B best nodes by (score desc,
 * token asc): node_tok/node_S/node_cnt [P][D][B] (unused token -1), the true
 * number of nodes node_count [P][D].  Per kept node of layer d its Ke best
 * out-edges to layer d+1 by (weight desc, destination asc): edge_dst/edge_S/
 * edge_cnt [P][D][B][Ke] and the true out-degree out_degree [P][D][B].
 * S values are int64 sums of fixed-point probabilities. */
int sdms_get_dag(sdms_ctx* ctx, int32_t* d_node_tok, int64_t* d_node_S, int32_t* d_node_cnt,
                 int32_t* d_node_count, int32_t* d_edge_dst, int64_t* d_edge_S,
                 int32_t* d_edge_cnt, int32_t* d_out_degree, void* stream);

/*
 * Several drafts per path (e.g. for tree verification; the paper's method extracts one sequence, its
 * introduction asks for the highest-likelihood one): the num_beams best paths of the DAG of the last
 * sdms_build_drafts, 1 <= num_beams <= max_beams.  A path of the DAG is worth the sum of the Eq. 5
 * in-weights of its nodes, added from its end towards its start in binary64 (the value search_mode 2
 * maximises), and only paths that run on to a node without successor or to layer D count.  Every node
 * keeps its num_beams best continuations - leaf: its own weight; otherwise the best of { own weight +
 * a kept continuation of a successor }, ordered by value (larger first), then by the successor's token
 * (smaller first), then by the continuation's rank - and the beams are the root's.  Unless two different
 * sums round to the same double (never with alpha = 1) that is the order "value, then token sequence".
 * The first beam is the search_mode 2 draft.
 * Outputs: d_beam_tok [P][num_beams][D] (unused -1), d_beam_len [P][num_beams] (0 = no such beam),
 * d_beam_value [P][num_beams].  DAG pool only; the histories must not have changed since the build
 * (SDMS_ERR_BAD_STATE otherwise, also when max_beams = 0).  Paths whose tables do not fit the table area
 * of the workspace get no beam and raise SDMS_STATUS_TABLES_FULL.
 */
int sdms_get_beams(sdms_ctx* ctx, int32_t num_beams, int32_t* d_beam_tok, int32_t* d_beam_len,
                   float* d_beam_value, void* stream);

/* Copies the stores: d_tok / d_pq [P][L], d_len [P] (any may be NULL). */
int sdms_debug_read_history(sdms_ctx* ctx, int32_t* d_tok, int32_t* d_pq, int32_t* d_len, void* stream);

/* How each path's query of the last sdms_build_drafts was answered: d_modes [P],
 * 0 = no query or no index entry, 1 = from the index bucket, 2 = by scanning. */
int sdms_debug_read_query_modes(sdms_ctx* ctx, int32_t* d_modes, void* stream);

/* Every wait inside a kernel (grid barrier of the wide pass, copy barriers of the streaming scan) is bounded:
 * when it runs out, the kernel raises SDMS_STATUS_TIMEOUT and returns, and the context stays usable.  This call
 * shows what that looks like without anything going wrong: one thread waits, with the same bounded wait, about
 * half a millisecond for a count that nobody raises, sets the status bit and returns. */
int sdms_debug_wait_timeout(sdms_ctx* ctx, void* stream);

/* Waits for `stream`, returns the status bits in *host_flags and clears them. */
int sdms_get_status(sdms_ctx* ctx, uint32_t* host_flags, void* stream);

/* ---- for callers that cannot allocate device memory ------------------------- */

/*
 * The paper has no counterpart of this call; it exists for one kind of caller.
 * A sampler plug-in that runs inside a serving engine usually finds the GPU's
 * memory already handed out: the engine reserves almost all free HBM for its
 * KV-cache pool at start-up, a later cudaMalloc may fail or stall every stream of
 * the device, and the plug-in has no access to the engine's own allocator.  Such
 * a caller cannot provide the workspace a context needs.  This call finds the
 * Eq. 3 matches straight from path histories the caller already holds, and the
 * only extra device memory it uses - two int32 counters per path - is a fixed
 * 128 KiB array inside the library image (present on every GPU that loads the
 * library, until the process exits).  It calls no cudaMalloc / cudaFree and no
 * allocating routine of any library.
 *
 *   d_tok [P][capacity], d_len [P] : the histories (inputs, P = groups * paths)
 *   d_offsets [P+1], d_gpos [cap]  : same meaning as in sdms_get_matches; a path
 *       shorter than k, or full, has no query and therefore no matches
 *
 * Limits and sharing: P <= SDMS_NOALLOC_MAX_PATHS and P * paths_per_group *
 * capacity < 2^31 (the largest number of matches there can be, so that the int32
 * offsets cannot wrap), otherwise SDMS_ERR_TOO_LARGE and nothing is launched;
 * paths_per_group <= SDMS_MAX_PATHS_PER_GROUP as for a context.  All calls on a device share the one array; each call
 * zeroes the counters it uses before counting, so calls in sequence on a stream
 * are independent of each other, but two calls whose kernels overlap on the GPU
 * (different streams, different threads) race and give wrong results.  The first
 * call on each device looks up the array's device address; make that first call
 * outside any stream capture.
 */
#define SDMS_NOALLOC_MAX_PATHS 16384
int sdms_match_noalloc(const int32_t* d_tok, const int32_t* d_len, int32_t num_groups,
                       int32_t paths_per_group, int32_t capacity, int32_t k, int32_t* d_offsets,
                       int32_t* d_gpos, size_t cap, void* stream);

/* ---- measurement hooks (no counterpart in the paper) ----------------------- */

#define SDMS_KERNEL_APPEND 0
#define SDMS_KERNEL_PROBE  1
#define SDMS_KERNEL_SCAN   2
#define SDMS_KERNEL_DAG    3
#define SDMS_KERNEL_ACCEPT 4
#define SDMS_KERNEL_BUILD_FUSED 5   /* probe + scan + dag in one launch (small prompts) */
#define SDMS_KERNEL_STEP   6        /* accept + commit + build in one launch (sdms_step) */
#define SDMS_KERNEL_TRIM   7        /* the three launches of sdms_trim */
#define SDMS_KERNEL_DAG_WIDE 8      /* aggregation and search of queries with many matches, all SMs */
#define SDMS_NUM_KERNELS   9

/* Number of kernels this context has launched since creation. */
int sdms_launch_count(sdms_ctx* ctx, uint64_t* launches);

/* When enabled every kernel launch is bracketed by CUDA events on its stream. */
int sdms_profile_enable(sdms_ctx* ctx, int32_t on);

/* Waits for the recorded events; adds up per kernel the elapsed milliseconds and
 * the launches since the last read (arrays of SDMS_NUM_KERNELS). */
int sdms_profile_read(sdms_ctx* ctx, float* ms, uint64_t* launches);

const char* sdms_strerror(int code);
const char* sdms_kernel_name(int kernel);

#ifdef __cplusplus
}
#endif
#endif  /* SDMS_H_ */
