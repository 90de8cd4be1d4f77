/*
 * CPU oracle for batched, trace-driven evaluation of DiSCo's dispatch and
 * migration policy (arXiv 2502.11417, Sec. 4 and Appendix F pseudocode).
 *
 * TEST INFRASTRUCTURE ONLY.  This is a plain, single-threaded, deliberately
 * slow restatement of the method, one (policy, request, token) at a time.  It
 * shares no code, header, table or helper with the CUDA library and must never
 * be linked into, imported by, or called from the product path.  Only the test
 * suite, the smoke check and the benchmark's CPU-baseline leg use it.
 *
 * All floating-point work is fp64 on the widened fp32 inputs; all times are
 * signed 64-bit microsecond ticks.
 */
#ifndef DISCO_ORACLE_H
#define DISCO_ORACLE_H

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define ORC_NBINS 864
#define ORC_MAX_PROMPT 4096
#define ORC_MAX_OUTPUT 8192
#define ORC_NKNOTS 257

enum { ORC_SERVER_ONLY = 0, ORC_DEVICE_ONLY = 1, ORC_RACE = 2 };
enum { ORC_FLAG_MIGRATION = 1, ORC_FLAG_PACING = 2, ORC_FLAG_STOCHASTIC = 16, ORC_FLAG_BETA_RULE = 32 };

typedef struct { float tbt_s, jitter, c_prefill, c_decode; } orc_server_t;
typedef struct { float prefill_tps, ttft_intercept_s, decode_tps, jitter, c_prefill, c_decode, lambda; } orc_device_t;
typedef struct { float budget, alpha, mig_threshold, t_m_s, r_c; uint32_t flags; uint32_t expected_len; uint32_t l_immediate; } orc_policy_t;

/* Dispatch rule of one (group, policy): what Algorithms 1-3 return, plus the
 * constants of the migration controller (Eq. 4-6). */
typedef struct {
    int32_t device_constrained;  /* Algorithm 1 */
    int32_t l_th;                /* Algorithm 3 / Eq. 3 */
    int32_t l_star;              /* Algorithm 2: first length class not fully funded */
    int32_t B;                   /* Eq. 6, tokens */
    int64_t w_star, w_tail;      /* Algorithm 2, ticks */
    int64_t tau, t_m;            /* ticks */
    int32_t candidate_winner;    /* 0 none, 1 server winner may migrate, 2 device winner may migrate */
    float   delta_c;             /* Eq. 5 */
    double  funded_fraction;     /* f of the class l_star (Algorithm 2), for tests */
    double  budget_A;            /* funded input tokens beyond the tail share, for tests */
    int32_t beta_rule;           /* Eq. 1: w(l) = 0 for l <= l_immediate, else min(beta l, w_tail) */
    int32_t l_immediate;
    int64_t beta;                /* ticks per prompt token */
} orc_prep_t;

typedef struct {
    double *ttft_s, *tbt_mean_s, *tbt_max_s, *cost;          /* [P][n] or NULL */
    uint32_t *tok_server, *tok_device, *mig_at;
    uint16_t *delayed;
    uint8_t *decision;
} orc_pair_out_t;

typedef struct {
    /* additive part */
    uint64_t n_requests, n_intervals;
    double sum_ttft_s, total_cost;
    uint64_t n_server_only, n_device_only, n_race, n_device_started, n_device_won, n_migrations;
    uint64_t tok_server, tok_device, prefill_tok_server, prefill_tok_device, delayed_tokens;
    uint64_t ttft_hist[ORC_NBINS], tbt_hist[ORC_NBINS];
    /* derived by orc_finish */
    double mean_ttft_s;
    double p50_ttft_s, p95_ttft_s, p99_ttft_s, p99_tbt_s;   /* lower edge of the bin holding the rank */
    int32_t bin_p50_ttft, bin_p95_ttft, bin_p99_ttft, bin_p99_tbt;
    /* exact order statistics (by sorting), filled by orc_eval when want_exact != 0 */
    double exact_p50_ttft_s, exact_p95_ttft_s, exact_p99_ttft_s, exact_p99_tbt_s;
} orc_stats_t;

typedef struct orc_trace orc_trace_t;

/* --- building blocks, exported so that tests can pin each one --- */
uint32_t orc_mix(uint32_t x);
uint32_t orc_hash(uint64_t seed, uint32_t request, uint32_t token);
int64_t  orc_jitter(uint32_t h, int64_t amplitude);
int32_t  orc_bin(int64_t ticks);
int64_t  orc_bin_lower_edge(int32_t bin);
int64_t  orc_seconds_to_ticks(float seconds);
int64_t  orc_rate_to_ticks(float per_second);

/* --- the path --- */
orc_trace_t* orc_load(uint64_t n, const int32_t* prompt_len, const int32_t* output_len,
                      const float* server_ttft_s, const uint8_t* server_profile,
                      const uint8_t* device_profile, const orc_server_t* servers, uint32_t n_servers,
                      const orc_device_t* devices, uint32_t n_devices);
void orc_free(orc_trace_t*);
const char* orc_last_error(void);

uint32_t orc_n_groups(const orc_trace_t*);
/* copies of the group tables: cnt[4097], sorted[N_g] (pass NULL to query N_g), knots[257] */
int64_t orc_group_tables(const orc_trace_t*, uint32_t g, int64_t* cnt, int64_t* sorted, int64_t* knots);
int64_t orc_inverse_cdf(const orc_trace_t*, uint32_t g, double q);

int orc_prep(const orc_trace_t*, const orc_policy_t* pol, uint32_t g, orc_prep_t* out);

/* One request under one policy; writes the generation and delivery times
 * g[1..n], d[1..n] (index 0 unused; arrays of n+1) and the hand-off index
 * (0 = none).  Returns the decision, or a negative error. */
int orc_play(const orc_trace_t*, const orc_policy_t* pol, uint64_t seed, uint64_t i,
             int64_t* g, int64_t* d, int64_t* ttft, int32_t* winner_is_device, int32_t* mig_at,
             int64_t* mig_latency, int32_t* delayed);

/* Requests [i0, i1) under every policy.  stats[P] is ADDED to (zero it first);
 * out may be NULL.  want_exact != 0 also sorts this call's TTFTs and TBTs. */
int orc_eval(const orc_trace_t*, const orc_policy_t* pol, uint32_t P, uint64_t seed,
             uint64_t i0, uint64_t i1, const orc_pair_out_t* out, orc_stats_t* stats, int want_exact);
/* The same with compact per-pair arrays: row p holds out_stride entries, request i goes to column
 * i - out_first (orc_eval: out_stride = n, out_first = 0). */
int orc_eval_cols(const orc_trace_t*, const orc_policy_t* pol, uint32_t P, uint64_t seed,
                  uint64_t i0, uint64_t i1, const orc_pair_out_t* out, uint64_t out_stride, uint64_t out_first,
                  orc_stats_t* stats, int want_exact);
void orc_finish(orc_stats_t* stats, uint32_t P);

int orc_select(const orc_stats_t* stats, uint32_t P, double cost_cap, double tbt_slo_s, int32_t* best);

#ifdef __cplusplus
}
#endif
#endif
