/*
 * libdisco -- batched, trace-driven evaluation of DiSCo's cost-aware dispatch
 * and token-level migration policy (arXiv 2502.11417) on one NVIDIA B200.
 *
 * For every (request, policy) pair the library derives the dispatch decision
 * (server only, device only, wait-then-race; Sec. 4.2, Algorithms 1-3), plays
 * the decode stream out token by token with per-token jitter, paced delivery
 * and buffer-based migration (Sec. 4.3, Eq. 4-6), prices it (Appendix E,
 * Eq. 8), reduces the pairs to per-policy QoE statistics (Sec. 5.1: mean and
 * tail TTFT, P99 TBT, cost) and picks a policy under a cost cap.
 *
 * Conventions
 *  - Plain C ABI.  Every function returns 0 on success or a negative status:
 *    DISCO_EINVAL (bad argument or input value), DISCO_ENOMEM, DISCO_ECUDA
 *    (a CUDA call failed), DISCO_EINFEASIBLE (selection only).  Nothing aborts
 *    or throws across the boundary; disco_last_error() describes the last
 *    failure of the calling thread.
 *  - "host" / "device" on a pointer says where the memory must live.  Inputs
 *    are never modified.  The context owns every byte it allocates; per-pair
 *    output arrays are allocated and owned by the caller.
 *  - `stream` is a cudaStream_t passed as void* (NULL = default stream).
 *  - Time is kept internally in integer microsecond ticks, so that results do
 *    not depend on the order of the parallel reductions.
 *  - There is no CPU fallback: without a CUDA device every call fails.
 */
#ifndef DISCO_H
#define DISCO_H

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define DISCO_NBINS 864          /* histogram bins: 32 per octave of ticks */
#define DISCO_MAX_PROMPT 4096
#define DISCO_MAX_OUTPUT 8192

#define DISCO_EINVAL (-1)
#define DISCO_ENOMEM (-2)
#define DISCO_ECUDA (-3)
#define DISCO_EINFEASIBLE (-4)

/* dispatch decisions (per-pair output `decision`) */
#define DISCO_SERVER_ONLY 0      /* device never started: the server answered within the wait */
#define DISCO_DEVICE_ONLY 1      /* Algorithm 3: prompt shorter than l_th */
#define DISCO_RACE 2             /* both endpoints ran; the first token won */

/* policy flags */
#define DISCO_FLAG_MIGRATION 1u  /* token-level migration on (Sec. 4.3) */
#define DISCO_FLAG_PACING 2u     /* delivery buffer: tokens handed over no faster than r_c */
#define DISCO_FLAG_STOCHASTIC 16u /* Stoch-S / Stoch-D baseline (Sec. 5.1): each request goes to the constrained
                                    endpoint with probability b, else to the other one; no race, no migration */
#define DISCO_FLAG_BETA_RULE 32u  /* device-constrained phase 2 as in Sec. 4.2, Eq. 1-2: wait 0 for prompts up to
                                    l_immediate, min(beta l, w_tail) above, beta the smallest whole number of ticks
                                    per prompt token that keeps the device's expected input-token share within b */
#define DISCO_MODE_AUTO (0u << 2)               /* Algorithm 1 decides from the costs */
#define DISCO_MODE_DEVICE_CONSTRAINED (1u << 2) /* force Algorithm 2 */
#define DISCO_MODE_SERVER_CONSTRAINED (2u << 2) /* force Algorithm 3 */

/* Server endpoint (Sec. 4.1 cost model; Sec. 3 decode characteristics). */
typedef struct {
    float tbt_s;       /* mean time between decode tokens, seconds, > 0 */
    float jitter;      /* per-token TBT varies uniformly by +- this fraction, in [0,1] */
    float c_prefill;   /* c^p_s, cost per prompt token */
    float c_decode;    /* c^d_s, cost per generated token */
} disco_server_profile_t;

/* Device endpoint: TTFT is linear in the prompt length, T_d(l) = l / prefill_tps + intercept (Sec. 4.2). */
typedef struct {
    float prefill_tps;        /* prompt tokens per second, > 0 */
    float ttft_intercept_s;   /* c of T_d = k l + c, >= 0 */
    float decode_tps;         /* generated tokens per second, > 0 */
    float jitter;             /* as for the server */
    float c_prefill;          /* c^p_d, energy cost per prompt token */
    float c_decode;           /* c^d_d */
    float lambda;             /* exchange rate energy -> money (Eq. 8) */
} disco_device_profile_t;

/* A request trace.  A request belongs to group (server_profile, device_profile);
 * each group has its own prompt-length distribution p(l) and server-TTFT
 * distribution F (Algorithm 1 inputs), both taken from the group's own rows. */
typedef struct {
    uint64_t n;                       /* requests, may be 0, < 2^31 */
    const int32_t* prompt_len;        /* [n], 1..DISCO_MAX_PROMPT */
    const int32_t* output_len;        /* [n], 1..DISCO_MAX_OUTPUT */
    const float*   server_ttft_s;     /* [n], finite, > 0, <= 2000 */
    const uint8_t* server_profile;    /* [n] or NULL (all 0) */
    const uint8_t* device_profile;    /* [n] or NULL (all 0) */
    const disco_server_profile_t* servers;  /* host, [n_servers] */
    uint32_t n_servers;               /* >= 1; n_servers * n_devices <= 64 */
    const disco_device_profile_t* devices;  /* host, [n_devices] */
    uint32_t n_devices;
    uint32_t arrays_on_device;        /* 0: the five [n] arrays are host memory; 1: device memory.  Host arrays that
                                         are all page-locked (cudaHostAlloc, cudaHostRegister) are read by the
                                         ingestion kernel in place; pageable ones are copied to the device first.
                                         Either way they may be reused as soon as disco_load_trace returns.
                                         2: host memory that is always copied first, by the copy engine: the transfer
                                         then leaves the multiprocessors free, so that it can run beside the kernels
                                         of another context (a second worker evaluating the previous trace). */
    uint64_t first_index;             /* index, in the whole trace, of request 0 of these arrays: 0 unless the arrays
                                         are a contiguous range (a shard) of a larger trace.  The per-token jitter hash
                                         is keyed by the request's index in the whole trace, so a shard loaded with its
                                         first_index draws what the whole trace would draw for its rows;
                                         first_index + n <= 2^32.  Per-pair output columns stay local (0 .. n-1). */
} disco_trace_desc_t;

/* One policy setting (Algorithm 1 inputs b, alpha; Eq. 4 overhead; Eq. 6 t_m, r_c). */
typedef struct {
    float budget;          /* b in [0,1] */
    float alpha;           /* tail ratio in (0,1) */
    float mig_threshold;   /* Overhead_migration of Eq. 4, cost units, >= 0; +INF = never migrate */
    float t_m_s;           /* estimated migration time, seconds; buffer B = ceil(r_c t_m) tokens */
    float r_c;             /* consumption rate, tokens/s, > 0 */
    uint32_t flags;        /* DISCO_FLAG_* | DISCO_MODE_* */
    uint32_t expected_len; /* Eq. 4's remaining length: 0 = the trace's true remainder n - m; else what is left of
                              this expected total output length, max(expected_len - m, 0) */
    uint32_t l_immediate;  /* DISCO_FLAG_BETA_RULE: prompts up to this length start the device at once (Eq. 1's l_th) */
} disco_policy_t;

/* Optional per-pair outputs, device memory, each [P][n] with requests
 * contiguous (index p * n + i, i = position in the caller's trace); any
 * member may be NULL. */
typedef struct {
    float *ttft_s, *tbt_mean_s, *tbt_max_s, *cost;
    uint32_t *tok_server, *tok_device;   /* generated tokens per endpoint; they sum to output_len */
    uint32_t *mig_at;                    /* hand-off index m (source generated tokens 1..m), 0 = no migration */
    uint16_t *delayed;                   /* tokens generated after their delivery slot during a migration */
    uint8_t *decision;                   /* DISCO_SERVER_ONLY / DEVICE_ONLY / RACE */
} disco_pair_out_t;

typedef struct {
    double mean_ttft_s, total_cost;
    float p50_ttft_s, p95_ttft_s, p99_ttft_s;   /* lower edge of the histogram bin holding the nearest rank */
    float p99_tbt_s;                            /* pooled over every inter-token interval of every request */
    int32_t bin_p50_ttft, bin_p95_ttft, bin_p99_ttft, bin_p99_tbt;
    uint64_t n_requests, n_intervals;
    uint64_t n_server_only, n_device_only, n_race, n_device_started, n_device_won, n_migrations;
    uint64_t tok_server, tok_device, prefill_tok_server, prefill_tok_device, delayed_tokens;
} disco_policy_stats_t;

/* What Algorithms 1-3 return for one (group, policy), for inspection. */
typedef struct {
    int32_t device_constrained;   /* Algorithm 1 */
    int32_t l_th;                 /* Algorithm 3 / Eq. 3: prompts shorter than this run on the device only */
    int32_t l_star;               /* Algorithm 2: shorter prompts wait 0, this length waits w_star, longer ones w_tail */
    int32_t B;                    /* Eq. 6 buffer, tokens */
    int64_t w_star, w_tail, tau;  /* ticks (microseconds) */
    int32_t beta_rule;            /* Eq. 1-2 variant in force (device-constrained groups of DISCO_FLAG_BETA_RULE policies) */
    int32_t l_immediate;          /* its immediate-start threshold (0 when b <= alpha) */
    int64_t beta;                 /* its slope, ticks per prompt token */
} disco_prep_t;

typedef struct disco_ctx disco_ctx_t;

/* Loads a trace (Algorithm 1's inputs): copies the arrays to the device if
 * they are host memory, converts times to ticks and builds, per group, the
 * prompt-length histogram p(l) and the sorted server-TTFT sample F.
 * *ctx must be NULL (a context is created) or a context from an earlier call
 * (it is reloaded in place, reusing its memory).  Synchronises `stream`.
 * DISCO_EINVAL if a value is out of the ranges above or a profile is invalid. */
int disco_load_trace(disco_ctx_t** ctx, const disco_trace_desc_t* desc, void* stream);

/* Evaluates every (request, policy) pair: dispatch (Sec. 4.2), play-out and
 * migration (Sec. 4.3), cost (Eq. 8); accumulates the per-policy sums and
 * histograms inside the context and, if `out` is not NULL, writes the per-pair
 * arrays.  pol is host memory [P], P >= 1.  `seed` keys the per-token jitter
 * hash.  Asynchronous on `stream`; results are read with disco_reduce_stats.
 * DISCO_EINVAL for a bad policy, or when a stream could outlast 2^31 ticks. */
int disco_eval_policies(disco_ctx_t* ctx, const disco_policy_t* pol, uint32_t P, uint64_t seed,
                        const disco_pair_out_t* out, void* stream);

/* Finishes the reductions of the last evaluation (Sec. 5.1 metrics) and copies
 * P records to host memory `stats`.  Synchronises `stream`. */
int disco_reduce_stats(disco_ctx_t* ctx, disco_policy_stats_t* stats, void* stream);

/* Picks, among P statistics records (host memory; those of disco_reduce_stats,
 * or records the caller merged itself), the policy whose total cost is within
 * cost_cap and whose P99 TBT is within tbt_slo_s that has the smallest P99 TTFT
 * (by histogram bin; then mean TTFT, then cost, then index) -- the objectives
 * of Sec. 4.1.  *best (host) receives its index.  If none is feasible, returns
 * DISCO_EINFEASIBLE and *best is the cheapest policy.  Runs on the host: the
 * records are already there, so no launch and no synchronisation. */
int disco_select_policy(const disco_policy_stats_t* stats, uint32_t P, double cost_cap, float tbt_slo_s,
                        int32_t* best);

/* The same selection by a kernel over the records the last disco_reduce_stats
 * left in the context's device memory.  Synchronises `stream`. */
int disco_select_policy_device(disco_ctx_t* ctx, double cost_cap, float tbt_slo_s, int32_t* best, void* stream);

/* Copies policy p's TTFT and pooled TBT histograms (host, DISCO_NBINS each; either may be NULL). */
int disco_get_histograms(disco_ctx_t* ctx, uint32_t p, uint64_t* ttft_hist, uint64_t* tbt_hist, void* stream);

/* Copies what Algorithms 1-3 produced for group g = server_profile * n_devices + device_profile, policy p. */
int disco_get_prep(disco_ctx_t* ctx, uint32_t g, uint32_t p, disco_prep_t* out, void* stream);

/* Copies group g's tables out (any may be NULL): requests per prompt length
 * cnt[DISCO_MAX_PROMPT+1] (host memory), the 257 equally spaced order statistics
 * of F and up to `n_sorted` of the smallest sorted TTFT ticks (host or device
 * memory, each).  Synchronises `stream`.  Returns the number of
 * requests behind the group's tables (the group's own requests, or what
 * disco_set_group_tables gave), or a negative status. */
int64_t disco_get_group_tables(disco_ctx_t* ctx, uint32_t g, int64_t* cnt, int32_t* knots,
                               int32_t* sorted_ticks, uint64_t n_sorted, void* stream);

/* ---- Evaluating one trace in several contexts (request-range shards, e.g. one per GPU) -------------------
 * Requests are independent given the tables of Algorithm 1 (p(l) and F per group), and every per-policy
 * accumulator is an integer sum over requests.  A shard is loaded with its first_index; it is then given
 * the tables of the WHOLE trace with disco_set_group_tables (its own tables, from disco_get_group_tables,
 * summed / merged with the other shards' by the caller), evaluated, and its accumulators exported; the
 * element-wise sum of all shards' accumulator words, imported into any one context, is reduced by
 * disco_reduce_stats to exactly the records one context holding the whole trace produces. */

/* Replaces the tables Algorithms 1-3 read by the caller's: cnt[G][DISCO_MAX_PROMPT+1] requests per prompt
 * length (host memory) and, group after group, the server-TTFT ticks behind F: n_ticks[g] (host) of them for
 * group g, in any order within the group, `ticks` in host or device memory (for instance the shards' sorted
 * ticks one after the other).  The library sorts them per group and rebuilds the cumulative token mass
 * (Eq. 3) and the 257 knots of F.  The context keeps its own requests.  DISCO_EINVAL if a group's length
 * counts do not add up to n_ticks[g] or a tick is negative (the context must then be reloaded).  Lasts until
 * the next disco_load_trace.  Synchronises `stream`. */
int disco_set_group_tables(disco_ctx_t* ctx, const int64_t* cnt, const int32_t* ticks, const uint64_t* n_ticks,
                           void* stream);

/* The accumulators of the last evaluation as additive 64-bit words: per (policy, group) counters, the
 * TTFT and pooled TBT histograms per policy, and per group the output tokens and requests they cover.
 * disco_accumulator_words gives their number (0 before an evaluation); export copies them to `words`,
 * import overwrites the context's with `words` (host or device memory; for example the sum over shards).
 * Both synchronise `stream`.  disco_reduce_stats then works on what was imported. */
uint64_t disco_accumulator_words(disco_ctx_t* ctx);
int disco_export_accumulators(disco_ctx_t* ctx, uint64_t* words, void* stream);
int disco_import_accumulators(disco_ctx_t* ctx, const uint64_t* words, void* stream);

/* Measurement aids.  disco_set_timing(ctx, 1) makes each evaluation record CUDA events on its stream around
 * its four main kernels; after disco_reduce_stats, disco_get_timing fills ms4[0..3] with the device
 * durations in milliseconds of: the play-out of clamp-free requests, the general play-out, the pair
 * reductions, the per-pair row writer (only for evaluations whose policies share one pacing / buffer
 * setting).  disco_kernel_launch_count returns how many kernels this library has launched in this process. */
int disco_set_timing(disco_ctx_t* ctx, int on);
int disco_get_timing(disco_ctx_t* ctx, float* ms4);
uint64_t disco_kernel_launch_count(void);

/* How the last evaluation's pairs were reduced (host counts4[4]): pairs settled zone by zone (a request against
 * the runs of neighbouring policies of a family of up to 128 policies that dispatch it alike); pairs evaluated
 * one by one; requests settled zone by zone, counted once per policy family; sweeps the zone kernel's blocks made
 * over segments of their request chunks.  The first two add up to requests x policies.  Synchronises `stream`. */
int disco_get_work_counts(disco_ctx_t* ctx, uint64_t* counts4, void* stream);

/* Checked build.  Compiled with -DDISCO_DEBUG the library checks every index its kernels derive (request, policy,
 * group, chunk, knot, histogram bin, window and staging slot, table entry) against its bound before the access; an
 * index out of range is recorded and the access skipped -- nothing traps -- and the next call that synchronises
 * returns DISCO_ECUDA with the kernel's name and the index in disco_last_error().  disco_debug_selftest shows that
 * the checks are live: it has a kernel offer an out-of-range index (the access is never made) and returns the
 * DISCO_ECUDA that follows; in an ordinary build it returns DISCO_EINVAL. */
int disco_debug_selftest(void* stream);

/* Measures what the GPU sustains on the integer instruction mix of the token loop (Sec. 4.3 play-out: per
 * token one counter add, the hash finaliser's three shift-xor pairs and two multiplies, one multiply-high
 * range map, one compare and one multiply-add into the sum = 13 lane-instructions) with every SM full of
 * independent lanes and nothing else to do: the ceiling the play-out's roofline fraction is quoted against.
 * Runs for a few milliseconds on `stream` and synchronises it.  lane_instr_per_s receives token-steps per
 * second x 13; token_steps_per_s (may be NULL) the token-steps per second themselves. */
int disco_measure_alu_peak(double* lane_instr_per_s, double* token_steps_per_s, void* stream);

/* Sorting without allocating.  (The paper has no counterpart to this call; it exists for the sake of
 * callers, not of the method.)
 *
 * Some programs that use this library may not allocate device memory at the point where they need a
 * result: a serving loop whose memory pool already owns the whole GPU and treats any further cudaMalloc
 * as an error, code that runs between the launches of a latency-critical stream where the implicit
 * synchronisation of cudaMalloc/cudaFree is unacceptable, or a plug-in that is handed device pointers
 * but no allocator.  disco_load_trace is closed to them, because it sizes and allocates a context.
 *
 * This call does the part of the load step that turns server TTFTs into the empirical distribution F of
 * Algorithm 1 -- seconds to microsecond ticks (nearest, ties to even), then an ascending sort -- for ONE
 * group of at most DISCO_NOALLOC_MAX_N requests.  Input and output are the caller's device arrays
 * (server_ttft_s[n] in, sorted_ticks[n] out); the sort's working memory is a fixed array of about 4.5 MB
 * that is part of the library image, so it occupies that much memory on every GPU the library is loaded
 * on, from load until the process exits.  The call makes no cudaMalloc, cudaFree or other allocating
 * call.  It returns the same ticks, in the same order, as disco_load_trace followed by
 * disco_get_group_tables on a one-group trace.
 *
 *  - n > DISCO_NOALLOC_MAX_N is refused with DISCO_EINVAL (use disco_load_trace); a TTFT that is not
 *    finite, not positive or above 2000 s gives DISCO_EINVAL after the kernels have run.
 *  - The first call on each device looks up the device address of the working array; make that first
 *    call during start-up, on the device you will use (cudaSetDevice first) and before any stream
 *    capture begins.
 *  - All calls on a device share the one working array, which still holds the previous call's data
 *    (the call clears what it needs cleared).  Two calls whose kernels could run at the same time on
 *    one GPU -- different streams, different host threads -- race on it: serialise them.
 *  - Synchronises `stream` before returning. */
#define DISCO_NOALLOC_MAX_N 262144u
int disco_sort_ttft_ticks_noalloc(const float* server_ttft_s /* device */, uint32_t n,
                                  int32_t* sorted_ticks /* device */, void* stream);

void disco_free_trace(disco_ctx_t* ctx);
const char* disco_last_error(void);

#ifdef __cplusplus
}
#endif
#endif
