/*
 * dynakv.h -- C ABI of libdynakv: cluster-based KV-cache retrieval with migration-free
 * cluster adaptation (arXiv 2511.07427, "DynaKV"), with the whole index and KV store
 * resident in the HBM of one sm_100a GPU.
 *
 * Vocabulary (paper, Section 4.1).  A *unit* is one KV head of one layer of one
 * sequence: the cache K_t that the paper partitions into M_t disjoint clusters
 * (Eq. 1-3), each with a representative r_j = mean of its members (Eq. 4).  Every call
 * below works on all U units of a context at once; units never interact.
 * G = query heads sharing one KV head, d = head dimension, n = tokens in a unit.
 *
 * Pointers.  Unless a parameter says "host", data pointers are DEVICE pointers owned by
 * the caller; the library reads or writes them on the context's stream and never frees
 * them.  Everything else (cluster arenas, tables, scratch) is owned by the context and
 * released by dynakv_destroy().  Calls enqueue work on the context's stream and return
 * without synchronising unless stated.
 *
 * Errors.  Host-detectable problems (NULL pointer, size mismatch, wrong call order)
 * return a negative code and enqueue nothing.  Conditions only the device can see
 * (budget smaller than the best cluster, cluster-id or token capacity reached, page pool
 * exhausted) never trap: the kernel skips the step it cannot do, sets a sticky bit in a
 * device status word, and dynakv_get_status() reports it.
 */
#ifndef DYNAKV_H_
#define DYNAKV_H_

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define DYNAKV_F32 0
#define DYNAKV_BF16 1
/* DYNAKV_FP8: K and V are PASSED as bf16 arrays (like DYNAKV_BF16) and kept in the precision the paper evaluates in
 * (Section 8.1): every row is rounded, where it enters the library, to e4m3 values (OCP 8-bit float: 4 exponent
 * bits, 3 mantissa bits, largest value 448) times one power-of-two scale per row, the smallest 2^e with
 * max|x| / 2^e <= 448, round to nearest even.  All arithmetic of the method then runs on those rounded values
 * (they are exact in bf16), and the gather-attention kernel streams a one-byte-per-element copy of the pages: half
 * the bytes of DYNAKV_BF16 per retrieved token.  The bytes and one scale exponent per row are all the context keeps of
 * a row (the paths that re-read keys decode them, exactly), so the pages take half the memory they take with
 * DYNAKV_BF16.  head_dim 128 only. */
#define DYNAKV_FP8 2

#define DYNAKV_INIT_KMEANSPP 0
#define DYNAKV_INIT_RANDOM 1

#define DYNAKV_OK 0
#define DYNAKV_ERR_ARG (-1)     /* NULL pointer or value out of range            */
#define DYNAKV_ERR_STATE (-2)   /* call order: e.g. decode before build_index    */
#define DYNAKV_ERR_CUDA (-3)    /* a CUDA runtime call failed                    */
#define DYNAKV_ERR_NOMEM (-4)   /* device allocation failed                      */
#define DYNAKV_ERR_TOO_LARGE (-5) /* dynakv_attend_rows_noalloc: more work than its fixed scratch holds */

/* sticky device status bits */
#define DYNAKV_ST_BUDGET_EXCEEDED 1u  /* best cluster alone larger than the budget; taken whole */
#define DYNAKV_ST_MAX_CLUSTERS 2u     /* a split was skipped: max_clusters ids in use            */
#define DYNAKV_ST_MAX_TOKENS 4u       /* an append was dropped: unit holds max_tokens            */
#define DYNAKV_ST_PAGE_POOL 8u        /* a split or append was skipped: no free page             */
#define DYNAKV_ST_INTERNAL 16u        /* an internal bound was hit (bounded wait ran out, ...)   */
#define DYNAKV_ST_BOUNDS 64u          /* checked build only: an index taken from a table was out of range; the access
                                         was skipped (dynakv_status.bounds_site names the first such place)       */
#define DYNAKV_ST_TIER_CACHE 32u      /* two-tier mode: a step's clusters did not fit a unit's cache; that unit's output
                                         of the step is meaningless                              */

typedef struct dynakv_ctx dynakv_ctx;

typedef struct dynakv_config {
    int32_t n_units;           /* U = sequences x layers x KV heads                              */
    int32_t gqa_group;         /* G, 1..8                                                        */
    int32_t head_dim;          /* d: 64 or 128                                                   */
    int32_t kv_dtype;          /* DYNAKV_F32, DYNAKV_BF16 or DYNAKV_FP8 for K, V; q, out, centroids are fp32 */
    int32_t max_tokens;        /* capacity per unit (prefill + decode)                           */
    int32_t max_clusters;      /* cluster ids per unit, <= 4096                                  */
    int32_t kmeans_iters;      /* T: Lloyd rounds at build time (all are run, no early exit)     */
    int32_t init_mode;         /* DYNAKV_INIT_KMEANSPP or DYNAKV_INIT_RANDOM                     */
    float split_size_factor;   /* gamma: split when n_j * M_live > gamma * N; <= 0 disables      */
    float split_var_factor;    /* alpha: tau = alpha * mean live sigma_j^2 at build; <= 0 disables */
    int32_t split_min_size;    /* clusters smaller than this are never split                     */
    int32_t split_iters;       /* cap on 2-means rounds in a split                               */
    int32_t trace;             /* 1: keep every Lloyd round's assignment for dynakv_get_build_trace */
    int32_t assign_mode;       /* 0: auto (tensor-core distance GEMM for bf16, d=128), 1: force fp32 path */
    int32_t attn_mode;         /* 0: auto (tensor-core gather-attention for bf16 K/V), 1: force the plain fp32 kernel */
    int32_t update_mode;       /* DYNAKV_MODE_ADAPTIVE (0, the paper's method), _STATIC, _LOCAL or _DELAYED          */
    int32_t local_max;         /* DYNAKV_MODE_LOCAL: a cluster born during decoding splits above this size (>= 2)    */
    int32_t det_sums;          /* 1: the build's centroid sums (Eq. 4) accumulate in 64-bit fixed point, units of 2^-24:
                                  the sum does not depend on the order in which keys arrive, so the centroids and every
                                  Lloyd round's assignment are reproducible bit for bit from run to run (the order of a
                                  cluster's rows inside its pages still follows arrival).  Needs |key element| < 2^18 (else DYNAKV_ST_INTERNAL is
                                  set and the element is clamped) and at most 2^20 keys per cluster.  0: fp32 atomic adds
                                  in arrival order (last bits of the centroids may differ between runs)             */
    int32_t buf_max;           /* DYNAKV_MODE_DELAYED: B_max of Algorithm 1, per unit -- entries buffered for flagged
                                  clusters that force a split (>= 1)                                                  */
    int32_t tier;              /* 1: two memory tiers (Section 6; Section 7 on CPU-GPU platforms).  The page pool lives in
                                  pinned host memory; device memory holds a cache of cache_pages page frames per unit.
                                  Each step's selected clusters are brought into the cache whole before the attention
                                  reads them, replacing whole clusters (Section 6.2); results are those of tier = 0.
                                  Any kv_dtype (FP8: pool and frames hold the one-byte rows and their exponents)      */
    int32_t cache_pages;       /* tier = 1: 32-token page frames per unit in device memory (< 2^20); must hold the clusters of
                                  any one step (about token_budget / 32 plus one per selected cluster)                */
} dynakv_config;

/* How the partition follows the decode stream (Section 3.1; the baselines of Section 8.1):
 *   ADAPTIVE  append to the nearest cluster; split_check splits clusters by the variance and size rules;
 *   STATIC    append to the nearest cluster; split_check never splits ("static update");
 *   LOCAL     new entries are clustered among themselves only ("local update"): the clusters of the build never
 *             change; append joins the nearest cluster born during decoding (the first new entry founds one), and
 *             split_check splits such a cluster by the same 2-means once it holds more than local_max entries. */
#define DYNAKV_MODE_ADAPTIVE 0
#define DYNAKV_MODE_STATIC 1
#define DYNAKV_MODE_LOCAL 2
/*   DELAYED   the adaptive rule with the delayed split of Algorithm 1 / Section 4.2 (there it saves the transfer of a
 *             cluster that is not in fast memory; here every cluster is resident and the mode only reproduces the
 *             policy): at a split check a cluster whose trigger fires is split only if the last decode step retrieved
 *             it; otherwise it is flagged, the entries it takes from then on count as buffered, and it is split at the
 *             first later check at which it is among the retrieved clusters.  When the buffered entries of a unit's
 *             flagged clusters reach buf_max, the flagged cluster with the most of them (lowest id among equals) is
 *             split as well, after the others.  Flags are not part of a checkpoint. */
#define DYNAKV_MODE_DELAYED 3

typedef struct dynakv_status {
    uint32_t error_bits;       /* OR of DYNAKV_ST_*                                              */
    int32_t bounds_site;       /* checked build: first place whose index test failed, 0 = none (else always 0) */
    int64_t n_appended;        /* appends stored, summed over units                              */
    int64_t n_splits;          /* splits performed, summed over units                            */
    int64_t tokens_selected;   /* tokens attended in the last decode step, summed over units     */
    int64_t clusters_selected; /* clusters selected in the last decode step, summed over units   */
    int64_t pages_in_use;      /* 32-token pages holding data, summed over units                 */
    int64_t assign_rechecked;  /* keys whose tensor-core argmin was re-decided in fp32 (build)   */
    int64_t tokens_attended_total;   /* tokens attended, summed over units and all decode steps  */
    int64_t clusters_selected_total; /* clusters selected, summed over units and all decode steps */
} dynakv_status;

/* Counters of the two-tier mode since dynakv_create, summed over units (dynakv_get_tier_stats):
 * a selected cluster is a hit (its copy in the cache is current), refreshed (it only took appends since it was copied:
 * the rows added since are copied) or fetched (all its rows are copied); evicted counts clusters that made room,
 * dropped_stale copies made void by a split. */
typedef struct dynakv_tier_stats {
    int64_t pages_fetched;     /* pages touched by a copy (whole or in part) */
    int64_t clusters_hit;
    int64_t clusters_fetched;
    int64_t clusters_refreshed;
    int64_t clusters_evicted;
    int64_t copies_dropped_stale;
    int64_t frames_in_use;     /* now, summed over units */
    int64_t frames_total;      /* n_units * cache_pages  */
    int64_t rows_fetched;      /* K/V rows copied: of a page only the rows that hold entries, of a refreshed cluster's
                                  former last page only the rows appended since the copy */
} dynakv_tier_stats;

/* Create a context on the current CUDA device; all later work runs on `cuda_stream`
 * (a cudaStream_t passed as void*, NULL = the legacy default stream).  Allocates the
 * arenas: about max_tokens * 4 * d * sizeof(kv) bytes per unit plus tables. */
int dynakv_create(const dynakv_config* cfg, void* cuda_stream, dynakv_ctx** out);

/* Prefill: NewCluster of Algorithm 1 / the k-means partition of Section 4.1 (Eq. 3) with
 * centroid representatives (Eq. 4).  K, V: [U][n][d] row-major in cfg.kv_dtype.
 * Seeded init (k-means++ by exponential race, or the n_clusters keys with the smallest
 * counter-based uniforms), then cfg.kmeans_iters rounds of nearest-centre assignment
 * (squared Euclidean, ties to the lowest id) and mean update (an empty cluster keeps its
 * centre).  Then the members of each cluster are stored contiguously in 32-token pages
 * (Section 5.1, intra-cluster placement), n_j, r_j and M2_j = sum ||k - r_j||^2 are
 * initialised (Algorithm 1, the initialisation of size, centroid and variance) and the unit's
 * variance threshold tau is set.  Token id = row index.  Requires
 * n_clusters <= n <= max_tokens, n_clusters <= max_clusters, d == head_dim.
 * May be called once per context. */
int dynakv_build_index(dynakv_ctx* ctx, const void* K, const void* V, int64_t n, int32_t d,
                       int32_t n_clusters, uint64_t seed);

/* dynakv_build_index followed by the correlation-aware placement of Section 5.1 (Eq. 8): the reference queries q_ref
 * (DEVICE, [n_ref][U][G][d] fp32 -- the paper uses the initial input) are scored and selected under token_budget on
 * the finished index, every pair of clusters retrieved by the same query is counted (the adjacency matrix of retrieval
 * frequencies; Eq. 8 divides it by one constant, which does not change an ordering), and the clusters' pages are
 * laid out again so that a cluster is followed by the not yet placed cluster it was co-retrieved with most often
 * (greedy chain from the most co-retrieved cluster; lowest id among equals).  Clusters stay contiguous page by page;
 * only the order of the clusters in the page pool changes, so every later call gives the results it gives after
 * dynakv_build_index.  In HBM the order of pages has no cost of its own (there is no seek, and a copy never spans two
 * pages); the call exists so that the placement can be run and its effect on access contiguity measured
 * (dynakv_get_work_list).  Needs n_clusters^2 * 4 bytes of scratch per unit during the call.  Counters and status
 * word are left as a plain build leaves them. */
int dynakv_build_index_placed(dynakv_ctx* ctx, const void* K, const void* V, int64_t n, int32_t d,
                              int32_t n_clusters, uint64_t seed, const float* q_ref, int64_t n_ref,
                              int32_t token_budget);

/* Algorithm 1, nearest-cluster assignment of the new entry, UpdateVar, AddEntry,
 * UpdateStats: for every unit, the new key k [U][d] joins the live cluster with the
 * nearest representative; n_j, r_j, M2_j are updated incrementally and the (k, v) row is
 * written into the tail page of that cluster (no existing entry moves).  The new token id
 * is the unit's token count before the call. */
int dynakv_append(dynakv_ctx* ctx, const void* k, const void* v);

/* Section 4.1 / Algorithm 1, retrieval of the top clusters by query-centroid similarity, then
 * attention over the retrieved entries only (Section 2.1).  q: [U][G][d] fp32.
 * score_j = mean over the G heads of q_g . r_j; clusters are taken in (score descending,
 * id ascending) order while their sizes sum to <= token_budget (the best cluster is taken
 * whole if it alone is larger, with DYNAKV_ST_BUDGET_EXCEEDED).  out: [U][G][d] fp32 =
 * softmax(q_g . k_i / sqrt(d)) v_i over the members of the selected clusters; zeros when
 * nothing is selected.  selected_ids: [U][max_clusters] int32, selection in score order,
 * -1 padded; may be NULL. */
int dynakv_decode_step(dynakv_ctx* ctx, const float* q, int32_t token_budget, float* out,
                       int32_t* selected_ids);

/* Algorithm 1's split decision and SplitCluster (Section 4.2, 5.2).  A live cluster with
 * n_j >= split_min_size splits when sigma_j^2 = M2_j / n_j > tau (variance rule) or
 * n_j * M_live > gamma * N (size rule), triggers evaluated on the state at entry, each
 * triggered cluster once, in ascending id.  2-means over its members: centre A = member
 * farthest from r_j, B = member farthest from A, up to split_iters rounds, ties to A.
 * The child holding the smallest token id keeps the id and its pages, compacted in place;
 * the other child moves to fresh pages under the next free id.  A split that leaves a
 * side empty is abandoned and not retried until the cluster's next append. */
int dynakv_split_check(dynakv_ctx* ctx);

/* n_steps iterations of { decode_step(q_t); append(k_t, v_t); split_check() } (the order
 * of Algorithm 1's loop body), replayed from CUDA graphs (of 8, 4, 2 and 1 iterations,
 * captured once per token budget) whose kernels read the step index and the addresses of
 * the caller's arrays from device memory, so later calls may pass other arrays at no cost.  q_steps: [n_steps][U][G][d] fp32, k_steps,
 * v_steps: [n_steps][U][d] kv_dtype, out_steps: [n_steps][U][G][d] fp32, all device.
 * All n_steps inputs must be complete before the call: units are independent, so a unit's
 * centroid pass for step t+1 (query scores, new key's distances) runs as soon as that
 * unit's own append of step t is done, while other units may still be splitting; results
 * are those of the stated order.  The context must have been created on a non-default
 * stream (stream capture), else DYNAKV_ERR_STATE. */
int dynakv_decode_loop(dynakv_ctx* ctx, const float* q_steps, const void* k_steps,
                       const void* v_steps, int64_t n_steps, int32_t token_budget,
                       float* out_steps);

/* One loop iteration as above with HOST buffers (pinned memory recommended): copies
 * q, k, v to the device, runs the three calls and copies out back.  Returns when out_host
 * holds the step's result; the step's append and split check may still be running on the
 * context's stream then, and every later call on the context is ordered behind them (a call
 * that synchronises, e.g. dynakv_get_status, sees them complete).  q_host, k_host, v_host
 * must stay unchanged until the call returns.  q_host [U][G][d] fp32, k_host, v_host
 * [U][d] kv_dtype, out_host [U][G][d]. */
int dynakv_step_host(dynakv_ctx* ctx, const float* q_host, const void* k_host,
                     const void* v_host, int32_t token_budget, float* out_host);

/* dynakv_decode_loop with HOST arrays (same shapes; pinned memory for the copies to overlap): the steps are taken in
 * chunks of up to 32 (shorter ones at both ends of the call, so that the first copy in and the last copy out are
 * short); while the loop runs one chunk on the device, the next chunk's q, k, v are copied in and the
 * previous chunk's outputs copied out on two more streams.  Returns when every output is in out_steps.  For a
 * caller that has its inputs step by step, dynakv_step_host is the call. */
int dynakv_decode_loop_host(dynakv_ctx* ctx, const float* q_steps, const void* k_steps, const void* v_steps,
                            int64_t n_steps, int32_t token_budget, float* out_steps);

/* Synchronises the stream and fills *host_out (host memory). */
int dynakv_get_status(dynakv_ctx* ctx, dynakv_status* host_out);

/* Synchronises and copies the index state to HOST arrays; any pointer may be NULL.
 *   tok_cluster [U][max_tokens] int32  cluster id of each token id (-1 beyond n)
 *   centroids   [U][max_clusters][d] fp32
 *   counts      [U][max_clusters] int32 (0 = dead or unused id)
 *   M2          [U][max_clusters] fp32
 *   n_tokens    [U] int32,  n_ids [U] int32 (ids handed out),  tau [U] fp32 */
int dynakv_export_state(dynakv_ctx* ctx, int32_t* tok_cluster, float* centroids, int32_t* counts,
                        float* M2, int32_t* n_tokens, int32_t* n_ids, float* tau);

/* Checkpoint and resume (the paper keeps its KV store on flash but describes no resume; these two calls make the
 * index restartable).  dynakv_export_kv synchronises and writes the first n tokens' K and V rows of every unit,
 * in token-id order, to DEVICE arrays [U][n][d] of cfg.kv_dtype (n = the units' common token count).  Together
 * with dynakv_export_state's tok_cluster, n_ids and tau that is a complete checkpoint.
 * dynakv_import_state takes such a checkpoint into a freshly created context INSTEAD of dynakv_build_index:
 * K, V and tok_cluster [U][n] are DEVICE arrays, n_ids [U] and tau [U] HOST arrays; n_build_clusters is the
 * n_clusters of the original build (ids below it are the build's clusters, which matters in
 * DYNAKV_MODE_LOCAL).  Members are laid out cluster by cluster in pages as after a build, and n_j, r_j
 * (member means, Eq. 4) and M2_j are recomputed from the members, so they equal the exported ones up to
 * fp32 rounding; ids without members stay unused; a split that had been abandoned may be tried again. */
int dynakv_export_kv(dynakv_ctx* ctx, void* K_out, void* V_out, int64_t n);
int dynakv_import_state(dynakv_ctx* ctx, const void* K, const void* V, int64_t n, const int32_t* tok_cluster,
                        const int32_t* n_ids, const float* tau, int32_t n_build_clusters);

/* Synchronises and copies the last decode step's selection sizes to HOST arrays:
 * n_selected [U], tokens_selected [U]; either may be NULL. */
int dynakv_get_selection(dynakv_ctx* ctx, int32_t* n_selected, int32_t* tokens_selected);

/* The last decode step's gather list, to HOST arrays: n_entries [U] and, if entries is not NULL, entries
 * [U][entries_per_unit][2] = (first row in the unit's page pool, rows <= 32) of every run of rows the attention kernel
 * copied, in the order it took them; entries_per_unit >= dynakv_work_list_capacity(ctx).  With tier = 1 the rows are
 * rows of the unit's cache frames.  Synchronises. */
int dynakv_get_work_list(dynakv_ctx* ctx, int32_t* n_entries, int32_t* entries, int64_t entries_per_unit);

/* Two-tier mode: the cache counters (HOST struct).  DYNAKV_ERR_STATE when the context has tier = 0.  Synchronises.
 * Section 6.2 defines the replacement policy by two principles (small clusters are the ones worth caching; recently
 * updated clusters are retained); the order this library evicts in: copies made void by a split, then clusters
 * unchanged since they were copied -- more pages first, the longest unused first among equals, then the lowest id --
 * then clusters that took appends since.  Clusters the current step selected are never evicted. */
int dynakv_get_tier_stats(dynakv_ctx* ctx, dynakv_tier_stats* host_out);

int dynakv_work_list_capacity(dynakv_ctx* ctx);

/* With cfg.trace = 1: HOST arrays picks [U][n_clusters] (token ids chosen as initial
 * centres, in centre order) and assign [T][U][n] (assignment of every Lloyd round);
 * either may be NULL.  Returns DYNAKV_ERR_STATE if tracing was off. */
int dynakv_get_build_trace(dynakv_ctx* ctx, int32_t* picks, int32_t* assign);

/* Self-test of the device-side bounded waits (no counterpart in the paper).  Every wait on a shared-memory barrier in
 * this library gives up after a bounded number of polls, sets DYNAKV_ST_INTERNAL and lets the kernel return.  This
 * call runs a one-thread kernel that waits, with a limit of 4096 polls, on a barrier nobody arrives at: *gave_up
 * (HOST) becomes 1, DYNAKV_ST_INTERNAL is set in the status word, and the context stays usable.  Synchronises. */
int dynakv_selftest_wait_expiry(dynakv_ctx* ctx, int32_t* gave_up);

/* Measurement aid (no counterpart in the paper).  Runs the gather-attention kernel `reps` times back to back on the
 * selection of the LAST dynakv_decode_step (same work lists, q as given, results to out), as ordinary launches
 * bracketed by two CUDA events on the context's stream, after one untimed launch.  *ms_per_launch (HOST) = elapsed
 * time / reps: the kernel's duration without the cost of an event pair around every launch.  bf16 K/V only.
 * Synchronises. */
int dynakv_time_gather_attention(dynakv_ctx* ctx, const float* q, float* out, int32_t reps, float* ms_per_launch);

/* Measurement aid (no counterpart in the paper).  With timing on, every kernel launched
 * by a direct call (not by dynakv_decode_loop's graph replay) is bracketed by CUDA events on
 * the context's stream.  dynakv_get_kernel_times synchronises and returns, per kernel class,
 * the summed event time in ms and the number of launches since the last reset, into HOST
 * arrays of DYNAKV_KC_COUNT entries. */
#define DYNAKV_KC_INIT 0
#define DYNAKV_KC_ASSIGN 1
#define DYNAKV_KC_UPDATE 2
#define DYNAKV_KC_FINALIZE 3
#define DYNAKV_KC_SELECT 4
#define DYNAKV_KC_ATTN 5
#define DYNAKV_KC_COMBINE 6
#define DYNAKV_KC_APPEND 7
#define DYNAKV_KC_SPLIT 8
#define DYNAKV_KC_FRONT 9
#define DYNAKV_KC_TIER 10       /* two-tier mode: cache bookkeeping and the page copies of a step */
#define DYNAKV_KC_COUNT 11
int dynakv_set_timing(dynakv_ctx* ctx, int32_t on);
int dynakv_get_kernel_times(dynakv_ctx* ctx, double* ms_total, int64_t* launches, int32_t reset);

/* Number of kernels this context has launched so far (graph replays count their nodes). */
int64_t dynakv_launch_count(dynakv_ctx* ctx);

/* Test aid (no counterpart in the paper).  1 if the library was compiled with -DDYNAKV_CHECKED, else 0.  In a checked
 * build every index a kernel takes out of a table and turns into an address (a cluster id, a page of a chain, a row of
 * the gather list, a token slot) is tested against the array it indexes; a failing test sets DYNAKV_ST_BOUNDS, records
 * its place in dynakv_status.bounds_site, and the access is skipped or replaced by an in-range one.  Results are those
 * of the ordinary build; it is slower and exists for the test suite. */
int dynakv_checked_build(void);

/* Text of the last CUDA error seen by this library on the calling thread ("" if none). */
const char* dynakv_last_error(void);

void dynakv_destroy(dynakv_ctx* ctx);

/* Attention without any allocation (the paper has no counterpart: this is a service entry of the
 * library, not a step of the method).  For callers that may not call cudaMalloc: code running
 * inside a serving stack or memory pool that has already claimed the whole device, code in a
 * latency-critical section that cannot afford the synchronisation an allocation implies, or a
 * sandboxed component that may only launch kernels on buffers it was handed.  Needs no context.
 *
 * For every unit u < n_units and head g < gqa_group:
 *     out[u][g] = softmax_i(q[u][g] . K[u][i] / sqrt(d)) V[u][i]   over ALL rows i < n,
 * which is what dynakv_decode_step returns when the token budget covers every cluster.
 * q [n_units][gqa_group][d] fp32, K and V [n_units][n][d] row-major in kv_dtype (DYNAKV_F32 or
 * DYNAKV_BF16), out [n_units][gqa_group][d] fp32: DEVICE pointers owned by the caller.  d is 64 or
 * 128, gqa_group 1..8, n >= 0 (n == 0 gives zeros).  Work is enqueued on cuda_stream
 * (a cudaStream_t, NULL = default stream) of the CURRENT device and the call returns at once.
 *
 * Scratch.  The split-K partial sums live in one fixed array of DYNAKV_NOALLOC_SCRATCH_BYTES that
 * is part of the library image: every GPU that loads the library holds it until the process ends.
 * The call needs n_units * 16 * gqa_group * (d + 2) floats of it and returns DYNAKV_ERR_TOO_LARGE,
 * enqueuing nothing, when that is more than the array holds (or n_units > 65535): split the units
 * over several calls.  With d = 128 and gqa_group = 4 the limit is 126 units per call.
 * The array is shared by all calls and keeps the previous call's contents; every record a call
 * reads is first written by that same call, so nothing needs clearing, but two calls whose
 * kernels overlap on the GPU (different streams, several host threads) race on it: issue calls
 * on one stream, or order them yourself.
 * The first call on each device looks up the array's device address (cudaGetSymbolAddress, with
 * that device current); make that first call before any stream capture begins.
 * Calls cudaMalloc / cudaFree never.  Returns DYNAKV_OK, DYNAKV_ERR_ARG, DYNAKV_ERR_TOO_LARGE or
 * DYNAKV_ERR_CUDA. */
#define DYNAKV_NOALLOC_SCRATCH_BYTES (4 * 1024 * 1024)
int dynakv_attend_rows_noalloc(const float* q, const void* K, const void* V, int32_t n_units, int64_t n,
                               int32_t gqa_group, int32_t d, int32_t kv_dtype, float* out, void* cuda_stream);

#ifdef __cplusplus
}
#endif
#endif /* DYNAKV_H_ */
