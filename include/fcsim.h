/*
 * fcsim -- batched Monte-Carlo evaluation of the token-level LLM-serving model on one GPU.
 *
 * Each replica is an independent copy of the discrete-time single-worker system of Section 2.1:
 * requests (l, o, t_arr) arrive n_t per slot into a FIFO waiting queue, are activated into an active
 * set whose KV-cache usage U_t = sum (l_i + j_i(t)) must stay <= M, generate one output token per
 * slot, and leave at the end of the slot in which the last token is produced.  Activation follows
 * Algorithm 2 (flow control: at most B_t activations per slot, E[B_t] = b, Theorem 3.6) with
 * last-in-first-out eviction on overflow (Section 3.3), or one of two baselines named in the
 * Introduction: greedy prefill-first admission (the b -> infinity limit of Algorithm 2) and chunked
 * prefill.  Metrics are those of Section 2.2: token throughput, prompt throughput, latency.
 *
 * All simulation state and arithmetic are integers.  Random words come from Philox4x32-10 with key =
 * seed and counter = (slot, replica id, stream, index); stream 0 (index 0) gives the slot's words
 * (word 0 -> n_t, word 1 -> B_t, word 2 -> arrival-state switch), stream 1 (index i) gives arrival i
 * of the slot (word 0 -> class, word 1 -> l, word 2 -> o).
 *
 * Conventions: every function returns 0 (FCSIM_OK) or a negative error code; nothing throws, aborts
 * or traps.  "HOST" / "DEVICE" says where a pointer must live.  Device output buffers are allocated
 * and owned by the caller; the library only allocates small private device copies of the tables.
 * One GPU; a handle is bound to the device that is current in fcsim_create, and fcsim_run / fcsim_stats
 * return FCSIM_EINVAL when called with another device current.  A handle is not thread-safe: calls on the
 * same handle must not overlap.  Different handles may be driven from different threads.
 */
#ifndef FCSIM_H
#define FCSIM_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

enum {
    FCSIM_OK = 0,
    FCSIM_EINVAL = -1, /* bad field, non-monotone table, vmin < 1 for a length table, max l + max o > M, ... */
    FCSIM_ECAP = -2,   /* Qcap/Acap need more shared memory than one warp can be given */
    FCSIM_ESIZE = -3,  /* a required buffer is NULL or too small */
    FCSIM_ERANGE = -4, /* steps beyond T_max */
    FCSIM_ECUDA = -5,  /* CUDA runtime error; code via fcsim_last_cuda_error */
    FCSIM_ENOMEM = -6, /* host allocation failed */
    FCSIM_ETOOBIG = -7 /* fcsim_stats_noalloc: the group rows exceed the library's fixed device scratch */
};

/* ALPHA is the alpha-protection greedy baseline of Section 4.1: prefill-first greedy admission that keeps
 * the usage within (1 - alpha) M when a prompt (initial memory l + 1) joins, and evicts ALL active
 * requests back to the waiting queue when the slot would overflow M. */
/* CLASSFLOW is Algorithm 1 (known output length): every slot, for each class k in turn, up to b_k waiting
 * requests of that class are activated, first come first served within the class.  The memory gate, the
 * token budget and the last-in-first-out eviction are those of Algorithm 2 (they never act when the
 * condition of Theorem 3.3 holds); a pick that does not fit ends the loop of its class only. */
/* MC is the memory-constrained benchmark of Section 4.1: first come first served, a request starts only if,
 * with every running request and the candidate run to completion and nothing else started, the usage of every
 * future slot stays within M (so no slot can overflow and nothing is evicted).  With mc_worst_case = 1 every
 * request is projected with the longest output length of its class (the unknown-length adaptation). */
enum {
    FCSIM_POLICY_FLOW = 0, FCSIM_POLICY_GREEDY = 1, FCSIM_POLICY_CHUNKED = 2, FCSIM_POLICY_ALPHA = 3,
    FCSIM_POLICY_CLASSFLOW = 4, FCSIM_POLICY_MC = 5
};

/* Integer inverse-CDF table.  Support {vmin .. vmin+n-1}; cdf[k] = floor(P(X <= vmin+k) * 2^32) clamped
 * to 2^32-1, non-decreasing; cdf[n-1] is a catch-all whose value is ignored.  A 32-bit word u maps to
 * vmin + min{k < n-1 : u < cdf[k]}, or vmin+n-1 if there is none.  `cdf` is a HOST pointer borrowed only
 * for the duration of fcsim_create / fcsim_query_sizes / fcsim_simulate_host. */
typedef struct {
    uint32_t n;
    int32_t vmin;
    const uint32_t* cdf;
} fcsim_table;

/* Law of the arrival count n_t (Section 2.1: n_t drawn from a known law with mean lambda).
 * n_states = 1: one count table.  n_states = 2: two-state modulated law; each slot the state s flips
 * first iff word 2 of the slot < switch_thr[s], then n_t is drawn from count[s].  Initial state 0.
 * Count values must lie in [0, 255]. */
typedef struct {
    uint32_t n_states;
    fcsim_table count[2];
    uint32_t switch_thr[2];
} fcsim_arrivals;

/* A group of replicas sharing policy and parameters; replicas are laid out group after group.
 * b_fp: Q16.16 activation rate b of Algorithm 2; B_t = (b_fp >> 16) + [ (word1 >> 16) < (b_fp & 0xffff) ],
 *       i.i.d., mean b_fp / 65536, bounded by (b_fp >> 16) + 1 (the law asked for by Theorem 3.6).
 * chunk: prefill chunk size c (CHUNKED only, >= 1).
 * rng_replica_base: generator replica id of the group's first replica (equal bases in two groups give
 *       common random numbers).
 * m_admit: ALPHA only, the admission limit floor((1 - alpha) M) in tokens, 1 .. M.
 * b_class: CLASSFLOW only, HOST array [n_classes] of the integer budgets b_k (0 .. 65535), borrowed during
 *       fcsim_create / fcsim_query_sizes; NULL otherwise.
 * mc_worst_case: MC only, 0 = output lengths known, 1 = project with the class's longest output length.
 * preempt_keep: what an evicted request loses.  0 = all progress: it re-enters the queue "refreshed", with
 *       its original (l, o) and nothing generated (Sections 2.1 and 3.3; the paper's model).  1 = only its place
 *       in the cache: the j output tokens it has generated stay with it as prompt, (l, o) <- (l + j, o - j), so
 *       they are loaded again at its next activation instead of being generated again.  The paper has no such
 *       variant.  The kept tokens are final, so completed_tokens grows by j and sum_w_completed by
 *       l*j + j(j+1)/2 at the eviction (a request's workload is the sum over its segments), wasted_tokens
 *       stays 0, and a completion record describes the last segment only.  Needs l_max + o_max <= 65536;
 *       not accepted with MC, which never evicts (FCSIM_EINVAL). */
typedef struct {
    int32_t policy;
    uint32_t b_fp;
    int32_t chunk;
    int32_t arrivals_id;
    uint32_t rng_replica_base;
    int32_t n_replicas;
    int32_t m_admit;
    const int32_t* b_class;
    int32_t mc_worst_case;
    int32_t preempt_keep;
} fcsim_group;

/* M: KV capacity in tokens (1 .. 2^30).  K: prefill-token budget per slot, 0 = none (the paper's model).
 * T_max: horizon (1 .. 2^24-1).  Qcap: waiting room; a new arrival finding |Q| >= Qcap is dropped and
 * counted (evicted requests always re-enter).  Acap: storage bound of the active set; when it is full,
 * activation stops for the slot and acap_blocked_steps counts it.  Lengths l, o must lie in [1, 65535],
 * n_classes in [1, 256].  All table/array pointers are HOST pointers. */
typedef struct {
    int32_t M, K, T_max, Qcap, Acap;
    uint64_t seed;
    int32_t n_classes;
    fcsim_table class_law;     /* values 0 .. n_classes-1 */
    const fcsim_table* prompt; /* [n_classes] law of l per class */
    const fcsim_table* decode; /* [n_classes] law of o per class */
    int32_t n_arrivals;
    const fcsim_arrivals* arrivals;
    int32_t n_groups;
    const fcsim_group* groups;
    int32_t trace_stride; /* record {U_t, |Q_t|} when t % stride == 0; 0 = no trace */
    int32_t hist_bins;    /* 0 = no latency histogram; bin = min(latency >> hist_shift, hist_bins-1) */
    int32_t hist_shift;
    int32_t complog_cap;  /* completions logged per replica; 0 = no log */
    int32_t trace_bulk;   /* 0 = trace records leave the registers with plain coalesced stores (default, faster as
                             measured); 1 = they are staged in shared memory and every block of 32 records leaves
                             with one 256-byte bulk asynchronous copy (needs 512 more bytes of shared memory per
                             warp).  Same results either way. */
} fcsim_config;

/* Per-replica counters, all int64, accumulated over the slots run so far (R = number of replicas).
 * Latency of a request = t_done - t_arr + 1 slots (arrival to completion, Section 2.2).
 * sum_w_completed adds l*o + o(o+1)/2 per completion (the per-request workload of Prop. 3.2).
 * status: bit 0 = Acap was hit, bit 1 = completion log overflowed.  q_final, p_final, resid_age
 * (sum over unfinished requests of t - t_arr + 1), resid_j (output tokens held by active requests) and
 * mmpp_state describe the state at the last slot run. */
typedef struct {
    int64_t steps_done, status, arrived, dropped, admitted, completed, evictions, overflow_steps,
        gate_blocked_steps, budget_blocked_steps, acap_blocked_steps, tokens_generated, prefill_tokens,
        completed_tokens, wasted_tokens, sum_lat, max_lat, sum_U, max_U, sum_N, max_Q, sum_w_completed,
        n_logged, q_final, p_final, resid_age, resid_j, mmpp_state;
} fcsim_counters;

/* Where a summary's p95/p99 come from. */
enum { FCSIM_PCT_NONE = 0, FCSIM_PCT_HISTOGRAM = 1, FCSIM_PCT_EXACT = 2 };

/* Per-group summary: `total` combines the group's replicas field by field (sum; max for max_lat, max_U,
 * max_Q and steps_done; bitwise or for status).  With n = replicas in the group and T = slots run:
 * mean_latency = sum_lat / completed; mean_utilisation = sum_U / (n T M); request_throughput =
 * completed / (n T); token_throughput = tokens_generated / (n T) (Section 2.2).
 * p95/p99 of the end-to-end latency (Section 2.2; the "95% latency" of Section 4.1's figures), q = 95, 99:
 *  - FCSIM_PCT_EXACT, when there is a completion log and no replica of the group overflowed it: the
 *    ceil(q * completed / 100)-th smallest latency of the group's completions, selected on the device from
 *    the log's latency words;
 *  - FCSIM_PCT_HISTOGRAM otherwise, when there is a histogram: the smallest bin k whose cumulative count
 *    reaches ceil(q * completed / 100), reported as the bin's largest latency ((k+1) << hist_shift) - 1, or
 *    max_lat for the open last bin;
 *  - FCSIM_PCT_NONE (values 0) when nothing completed or neither output exists.
 * percentile_source says which. */
typedef struct {
    fcsim_counters total;
    double mean_latency, p95_latency, p99_latency, mean_utilisation, request_throughput, token_throughput;
    int32_t percentile_source;
    int32_t reserved;
} fcsim_summary;

/* DEVICE buffers, caller-owned, each at least the size fcsim_query_sizes reports and 16-byte aligned.
 * workspace: per replica, the simulator state between launches and the waiting queue (a ring of the next power of
 *            two >= Qcap + Acap entries of 8 bytes, read and written during launches); opaque.
 * counters:  [R] fcsim_counters.
 * trace:     [R][T_max / trace_stride] {int32 U_t, int32 |Q_t|}, or NULL when trace_stride = 0.
 * hist:      [R][hist_bins] int32, or NULL when hist_bins = 0.
 * complog:   [R][complog_cap] {int32 t_done, int32 latency}, or NULL when complog_cap = 0.
 * scratch:   per-group reduction area used by fcsim_stats (opaque; with a completion log it includes the digit
 *            counts of the percentile selection, 3 * 4096 + 8 words of 8 bytes per group). */
typedef struct {
    void* workspace;
    void* counters;
    void* trace;
    void* hist;
    void* complog;
    void* scratch;
} fcsim_buffers;

typedef struct {
    size_t workspace, counters, trace, hist, complog, scratch;
} fcsim_sizes;

/* Launch geometry chosen for a handle (for reporting).  A configuration whose groups use several policies is
 * advanced by one kernel per policy; the figures are those of the policy with the most replicas. */
typedef struct {
    int32_t grid, block, warps_per_block, blocks_per_sm, sm_count;
    int32_t smem_per_block, smem_per_warp, max_steps_per_launch;
} fcsim_launch_info;

typedef struct fcsim fcsim_t; /* opaque host object */

/* Validates `cfg` and reports the bytes the caller must allocate for each device buffer. */
int fcsim_query_sizes(const fcsim_config* cfg, fcsim_sizes* out);

/* Validates, copies the tables to the device, zeroes workspace/counters/hist/complog/trace and returns a
 * handle positioned before slot 1.  Synchronous (default stream).  The buffers must outlive the handle. */
int fcsim_create(const fcsim_config* cfg, const fcsim_buffers* device_buffers, fcsim_t** out);

/* Advances every replica by n_steps slots (steps_done + n_steps <= T_max, else FCSIM_ERANGE).
 * Asynchronous on `cuda_stream` (a cudaStream_t; NULL = default stream).  Resumable: run(a) then run(b)
 * gives bit for bit the state and outputs of run(a+b).  Long runs are split into several launches.
 * The groups of each policy are advanced by a kernel compiled for that policy.  With several policies the
 * kernels run side by side: the first on `cuda_stream`, the others on streams owned by the handle that are
 * forked from and joined back to `cuda_stream` with events, so work enqueued on `cuda_stream` after the call
 * sees all of them finished. */
int fcsim_run(fcsim_t* h, int32_t n_steps, void* cuda_stream);

/* Reduces counters and histograms per group on the device, then synchronises `cuda_stream` and copies:
 * host_out (HOST, [R], may be NULL) <- per-replica counters; per_group_out (HOST, [n_groups], may be
 * NULL) <- summaries. */
int fcsim_stats(fcsim_t* h, void* cuda_stream, fcsim_counters* host_out, fcsim_summary* per_group_out);

/* Group summaries for callers that must not allocate.  (The paper has no counterpart: this is a
 * deployment convenience of the library.)
 *
 * Some hosts of this library cannot obtain device memory when they want statistics: a serving process
 * whose memory manager has already claimed the whole GPU and hands none back, a monitoring thread that
 * must not trigger the implicit device-wide synchronisation an allocation or free causes, or an embedding
 * that simply forbids the CUDA allocator after start-up.  fcsim_stats needs a caller-allocated `scratch`
 * buffer for its per-group rows; this variant needs none.  It runs the same two reduction kernels, but
 * their group rows live in a fixed array inside the library's device image
 * (FCSIM_NOALLOC_SCRATCH_WORDS 64-bit words = 1 MiB, held by every GPU that loads the library until the
 * process exits), and the rows come back through a fixed host array inside the library.  It calls no
 * device or host allocator and frees nothing.
 *
 * per_group_out: HOST, [n_groups], receives exactly what fcsim_stats would write there.
 * Limit: n_groups * (28 + hist_bins), or n_groups * (28 + hist_bins + 8 + 3 * 4096) with a completion log (the
 * digit counts of the percentile selection), must not exceed FCSIM_NOALLOC_SCRATCH_WORDS, otherwise
 * FCSIM_ETOOBIG is returned and nothing is launched.
 * First call on a device: the library looks up the device address of its array (one runtime query, no
 * allocation) and remembers it; make that first call outside any stream capture, with the handle's
 * device current.
 * Sharing: every call, from every handle, uses the one array; it still holds the previous call's rows,
 * so each call clears the part it needs on `cuda_stream` before reducing.  Two calls whose GPU work
 * overlaps (different streams or threads) race on the array and on the host staging array: serialise them.
 * Synchronises `cuda_stream` before returning. */
#define FCSIM_NOALLOC_SCRATCH_WORDS 131072
int fcsim_stats_noalloc(fcsim_t* h, void* cuda_stream, fcsim_summary* per_group_out);

int fcsim_destroy(fcsim_t* h);

int32_t fcsim_steps_done(const fcsim_t* h);
int fcsim_get_launch_info(const fcsim_t* h, fcsim_launch_info* out);
int fcsim_last_cuda_error(const fcsim_t* h); /* cudaError_t of the last FCSIM_ECUDA, else 0 */
const char* fcsim_last_cuda_error_name(const fcsim_t* h); /* its symbolic name */

/* Diagnostics.  A library compiled with -DFCSIM_CHECKED compares every shared-memory and output index of
 * the step kernel with its bound; the first violation is recorded instead of performed.  fcsim_debug_read
 * copies the record to HOST out[8] = {source line (0 = none), index, bound, replica, 0, 0, 0, 0}
 * (synchronous).  In a normal build the record is always zero. */
int fcsim_debug_read(fcsim_t* h, uint32_t out[8]);
int fcsim_is_checked_build(void);
const char* fcsim_strerror(int code);

/* Whole job with HOST buffers: allocates device memory (one cudaMalloc), runs slots 1..n_steps, copies the
 * outputs to the given HOST arrays (each may be NULL; shapes as in fcsim_buffers with T_max = cfg->T_max; trace
 * records of slots that were not run read as zero; of a completion-log row only the first n_logged entries are
 * meaningful, and entries beyond the longest row's n_logged may be left untouched) and frees the device memory.
 * Synchronous.
 * A trace of 256 MB or more does not wait for the end of the run: the device holds only two windows of the
 * horizon (2048 records per replica or more each), and every filled window is copied into the caller's rows
 * with one strided copy on a second stream while the kernels fill the other.  The copies overlap the run only
 * when host_trace is page-locked memory; with pageable memory the result is the same, later. */
int fcsim_simulate_host(const fcsim_config* cfg, int32_t n_steps, fcsim_counters* host_counters,
                        void* host_trace, void* host_hist, void* host_complog, fcsim_summary* per_group_out);

#ifdef __cplusplus
}
#endif
#endif /* FCSIM_H */
