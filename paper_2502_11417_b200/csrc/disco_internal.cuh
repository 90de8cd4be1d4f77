// Internal declarations shared by the translation units of libdisco.
#pragma once

#include <cuda_runtime.h>
#include <stdint.h>

#include "disco.h"

namespace disco {

constexpr int kNBins = DISCO_NBINS;
constexpr int kMaxPrompt = DISCO_MAX_PROMPT;
constexpr int kMaxOutput = DISCO_MAX_OUTPUT;
constexpr int kNKnots = 257;
constexpr int kMaxGroups = 64;

// ---- per-group constants, ticks and costs (one per (server, device) profile pair) ----
struct GroupConst {
    int32_t T_srv, J_srv;        // server decode interval and jitter amplitude, ticks
    int32_t T_dev, J_dev;        // device decode interval and jitter amplitude
    int32_t kappa, c0;           // device TTFT = kappa * l + c0
    int32_t auto_device_constrained;   // Algorithm 1 evaluated on this group's costs
    int32_t candidate;           // 0 none, 1 a winning server may migrate (it is the dearer decoder), 2 a winning device may
    float delta_c;               // |c^d_s - lambda c^d_d|  (Eq. 5)
    float cps, cds, lcpd, lcdd;  // fp32 cost rates, device ones already in money
    double cps_d, cds_d, cpd_d, cdd_d, lambda_d;   // fp64 rates for the totals
};

// ---- per-policy constants derived on the host ----
struct PolicyConst {
    float budget, alpha, theta;
    uint32_t flags;
    int32_t tau, B;
    int32_t cls;                 // timeline class (policies with equal tau, B, pacing share play-outs)
    int32_t mode;                // 0 Algorithm 1 decides, 1 device-constrained, 2 server-constrained
    uint32_t expected_len;       // 0 = true remainder in the migration trigger
    uint32_t route_thr;          // stochastic routing: constrained endpoint iff hash < route_thr (or route_all)
    int32_t route_all;
    uint32_t l_immediate;        // Eq. 1's immediate-start threshold (beta rule)
};

// ---- what Algorithms 1-3 produce for one (group, policy) ----
struct Prep {
    int32_t device_constrained;
    int32_t l_th;
    int32_t l_star;
    int32_t w_star, w_tail;
    float theta;
    int32_t mig_on;
    int32_t stochastic;          // random routing instead of Algorithms 2-3
    uint32_t expected_len, route_thr;
    int32_t route_all;
    int32_t beta_rule;           // Eq. 1-2 variant: l_star holds the immediate-start threshold, w_star the slope beta
};

// ---- a timeline class: the parameters a play-out depends on besides the request ----
struct ClassConst {
    int32_t tau_eff;             // tau when pacing is on, else 0 (then delivery = generation)
    int32_t tau;                 // tau of the policies (for the "equals tau" fast count)
    int32_t B;
    int32_t pacing, mig_any;
    // dense windows of histogram bins that regular inter-token intervals can fall in
    int32_t W[3];                // bins per request for the server, device and migrated timelines
    int32_t lo[kMaxGroups][3];   // first bin of each window, per group
    int32_t ktau[kMaxGroups][3]; // index of bin(tau) inside the window, or -1
};

// Per-request summaries of the up to three distinct decode timelines of a class.
struct TimelineRec {
    uint32_t *sum[3], *max[3];   // d_n - d_1 and the largest TBT, ticks ([n] each)
    uint32_t* stall;             // TBT of the first token after a hand-off
    uint16_t *m, *delayed;       // hand-off index (0 = buffer never fills) and delayed tokens
    uint32_t* win[3];            // [n][W[c]] counts per window bin
};

struct TraceDev {
    uint32_t n;
    int32_t n_groups;
    const int32_t* S;            // server TTFT ticks, internal order: by group, inside a group by prompt length
    const uint16_t *l, *nout;
    const uint32_t* orig;        // caller's index of each request
    const uint32_t* inv;         // place of each of the caller's requests in the internal order
    const uint32_t* len_end;     // [G][4097]: where the group's requests of each prompt length end (the next length starts)
    const uint32_t* grp_off;     // [G+1]
};

struct Chunk { uint32_t start, len; int32_t g; int32_t pad; };

enum AccSlot { A_SERVER_ONLY = 0, A_DEVICE_ONLY, A_RACE, A_STARTED, A_DEVICE_WON, A_MIGR, A_TOK_DEVICE,
               A_PRE_SERVER, A_PRE_DEVICE, A_DELAYED, A_TTFT_SUM, A_TAU_CNT, kNAcc };

// ---- device helpers -------------------------------------------------------------------------------------

// Jitter hash: xorshift-multiply finaliser over a per-request key plus token counter.
__host__ __device__ __forceinline__ uint32_t mix32(uint32_t x) {
    x ^= x >> 16; x *= 0xA54FF53Bu;
    x ^= x >> 15; x *= 0x510E527Fu;
    x ^= x >> 16;
    return x;
}
constexpr uint32_t kHashSeed = 0x6A09E667u, kHashReq = 0xBB67AE85u, kHashTok = 0x3C6EF373u;

__host__ __device__ __forceinline__ uint32_t seed_key(uint64_t seed) {
    return mix32((uint32_t)seed ^ kHashSeed) ^ (uint32_t)(seed >> 32);
}

#ifdef __CUDACC__
// Histogram bin of a tick count: exact below 32, then 32 bins per octave.  The exponent and the five
// leading mantissa bits come from the float representation (round-toward-zero keeps them exact).
__device__ __forceinline__ int bin_of_ticks(uint32_t t) {
    if (t < 32u) return (int)t;
    int b = (int)(__float_as_uint(__uint2float_rz(t)) >> 18) - ((127 + 4) << 5);
    return min(b, kNBins - 1);
}
#endif

// Host-side bin (same partition of the axis, integer arithmetic).
inline int host_bin_of_ticks(int64_t t) {
    if (t < 0) t = 0;
    if (t < 32) return (int)t;
    int e = 63 - __builtin_clzll((unsigned long long)t);
    int64_t b = 32 * (int64_t)(e - 4) + ((t >> (e - 5)) & 31);
    return (int)(b < kNBins - 1 ? b : kNBins - 1);
}

// Lower edge of a bin, ticks.
inline int64_t host_bin_edge_ticks(int b) {
    return b < 32 ? (int64_t)b : (int64_t)(32 + (b & 31)) << ((b >> 5) - 1);
}

#ifdef __CUDACC__
// Launch that lets the grid be scheduled while its predecessor in the stream is still draining (programmatic
// stream serialisation).  Every kernel launched this way calls grid_dependency_wait() before it reads or
// writes global memory; the wait returns once the preceding grids have completed and their writes are visible.
template <class... KArgs, class... Args>
inline cudaError_t launch_after(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t st,
                                Args&&... args) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid; cfg.blockDim = block; cfg.dynamicSmemBytes = smem; cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr; cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, kernel, KArgs(args)...);
}
__device__ __forceinline__ void grid_dependency_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
#endif

// Records the calling thread's error message (read back by disco_last_error) and returns `code`.
int set_error(int code, const char* msg);

// ---- checked build (-DDISCO_DEBUG) -----------------------------------------------------------------------
// Every index a kernel derives from data or from its launch geometry -- request, policy, group, chunk, knot,
// histogram bin, window slot, staging slot, table entry -- goes through DBG_OK(index, bound, kernel, what) before
// the access.  An index outside [0, bound) is recorded (first one wins) and the access is skipped: nothing traps,
// the context stays usable, and the next call that synchronises returns DISCO_ECUDA naming kernel and index.
// In the ordinary build DBG_OK is the constant true and the checks vanish.
enum DbgKernel { DBG_K_INGEST = 1, DBG_K_RADIX, DBG_K_GATHER, DBG_K_TABLES, DBG_K_PREP, DBG_K_PLAYOUT_FAST, DBG_K_PLAYOUT,
                 DBG_K_PAIRS_ACC, DBG_K_PAIRS_ZONES, DBG_K_PAIRS_ROWS, DBG_K_FINALIZE, DBG_K_SELECT, DBG_K_SELFTEST,
                 DBG_K_COUNT };
enum DbgWhat { DBG_REQUEST = 1, DBG_POLICY, DBG_GROUP, DBG_CHUNK, DBG_KNOT, DBG_BIN, DBG_WINDOW, DBG_SLOT, DBG_TABLE,
               DBG_COUNTER, DBG_ELEMENT, DBG_WHAT_COUNT };
#ifdef DISCO_DEBUG
#ifdef __CUDACC__
static __device__ int32_t dbg_word[4];          // one per translation unit: kernel, what, index, bound
__device__ __forceinline__ bool dbg_in(long long i, long long n, int kernel, int what) {
    if (i >= 0 && i < n) return true;
    if (atomicCAS(&dbg_word[0], 0, kernel) == 0) {
        dbg_word[1] = what;
        dbg_word[2] = (int32_t)(i < -2147483647LL ? -2147483647LL : (i > 2147483647LL ? 2147483647LL : i));
        dbg_word[3] = (int32_t)(n > 2147483647LL ? 2147483647LL : n);
    }
    return false;
}
#define DBG_OK(i, n, kernel, what) (::disco::dbg_in((long long)(i), (long long)(n), (kernel), (what)))
// Reads (and clears) this translation unit's record; registered with the host side once per unit that has kernels.
void dbg_register(cudaError_t (*reader)(int32_t*));
struct DbgRegistrar { explicit DbgRegistrar(cudaError_t (*r)(int32_t*)) { dbg_register(r); } };
#define DBG_TRANSLATION_UNIT()                                                                         \
    namespace {                                                                                        \
    cudaError_t dbg_read_unit(int32_t* out) {                                                          \
        cudaError_t e = cudaMemcpyFromSymbol(out, ::disco::dbg_word, 16);                              \
        if (e == cudaSuccess && out[0]) { const int32_t z[4] = {0, 0, 0, 0}; e = cudaMemcpyToSymbol(::disco::dbg_word, z, 16); } \
        return e;                                                                                      \
    }                                                                                                  \
    ::disco::DbgRegistrar dbg_registrar_unit(dbg_read_unit);                                           \
    }
#endif
#else
#define DBG_OK(i, n, kernel, what) true
#define DBG_TRANSLATION_UNIT()
#endif

// ---- launch wrappers (defined in the kernel translation units) -------------------------------------------
cudaError_t launch_prep(const PolicyConst* pol, uint32_t P, int G, const GroupConst* gc, const int64_t* cum_mass,
                        const uint32_t* cnt, const int32_t* sorted, const uint32_t* grp_off, Prep* prep,
                        cudaStream_t st);
cudaError_t launch_prep_beta(const PolicyConst* pol, uint32_t P, int G, const int64_t* cum_mass, const uint32_t* cnt,
                             const int32_t* sorted, const uint32_t* grp_off, Prep* prep, cudaStream_t st);
cudaError_t launch_timeline(const TraceDev& tr, const GroupConst* gc, const ClassConst* cc, bool pacing,
                            const int32_t* knots, uint32_t k0 /* hash key base: seed_key(seed) + first_index * kHashReq */,
                            TimelineRec rec, int32_t* err, uint32_t* todo,
                            uint32_t* todo_count /* two words, zero on entry: length of the list, batch tickets */,
                            bool never_clamps /* pacing on and tau >= T + J for both endpoints of every group */,
                            bool long_outputs /* mean output length of 512 tokens or more */,
                            cudaEvent_t mid /* recorded between its two kernels, or null */,
                            int sms /* multiprocessors of the device */, cudaStream_t st);
cudaError_t launch_pairs(const TraceDev& tr, const GroupConst* gc, const ClassConst* cc, const Prep* prep, uint32_t P,
                         const uint32_t* pol_list, uint32_t n_list, const Chunk* chunks, uint32_t n_chunks,
                         TimelineRec rec, disco_pair_out_t out, uint64_t* acc, uint64_t* hist_ttft,
                         uint64_t* hist_tbt,
                         uint32_t* left_mask /* [n][ceil(tiles / 32)] scratch for the requests the zone kernel leaves to
                         the pair kernel, or null: every pair is evaluated one by one */,
                         uint32_t* left_count /* [n_chunks][tiles] scratch */,
                         uint32_t* left_lists /* [n_chunks][tiles][kLeftList] scratch, or null */,
                         uint32_t zone_blocks /* blocks the zone kernel may run: one per multiprocessor */,
                         uint32_t* zone_ticket /* one word, zero: the zone kernel's blocks draw their work from it */,
                         uint64_t* work /* [4], added to: pairs settled zone by zone, pairs evaluated one by one,
                         requests settled per policy family, sweeps over segments of a chunk */,
                         uint32_t k0, bool extras /* some policy routes at random or uses an
                         expected length */, bool wide /* some window W of the class spans several bins */,
                         cudaEvent_t mid /* recorded between its two kernels, or null */,
                         cudaStream_t st);
cudaError_t launch_pairs_zones(const TraceDev& tr, const GroupConst* gc, const ClassConst* cc, const Prep* prep,
                               uint32_t P, const uint32_t* pol_list, uint32_t n_list, int PL, const Chunk* chunks,
                               uint32_t n_chunks, TimelineRec rec, uint64_t* acc, uint64_t* hist_ttft,
                               uint64_t* hist_tbt, uint32_t* left_mask, uint32_t* left_count, uint32_t* left_lists,
                               uint32_t max_blocks, uint32_t* ticket, uint64_t* work, cudaStream_t st);
cudaError_t launch_finalize(uint32_t P, int G, const GroupConst* gc, const uint64_t* acc, const uint64_t* hist_ttft,
                            const uint64_t* hist_tbt,
                            const uint64_t* fin_totals /* [2G]: output tokens per group, then requests per group */,
                            disco_policy_stats_t* stats /* [P] + 16 bytes */,
                            disco_policy_stats_t* stats_host /* pinned host mirror of the same size, written by the kernel */,
                            const int32_t* err, cudaStream_t st);
cudaError_t launch_select(const disco_policy_stats_t* stats, uint32_t P, double cost_cap, float tbt_slo_s,
                          int32_t* result /* [2]: status, index; may be pinned host memory */, cudaStream_t st);
// Cumulative token mass and knots from tables given by the caller (F_off[g] .. F_off[g+1] delimit group g's ticks).
cudaError_t launch_tables_imported(int G, const uint32_t* cnt, int64_t* cum_mass, uint32_t* ng_exact,
                                   const int32_t* F_sorted, const uint32_t* F_off, int32_t* knots, cudaStream_t st);
// Sorts ticks stored group after group (off[g] .. off[g+1], device memory) ascending within each group into `out`;
// keys_a / keys_b: scratch of `total` 64-bit words each, counts: 256 * 1024 + 256 words; err[0..1]: set to (3, index) on
// a negative tick.  Launches 2 + 3 * (G > 1 ? 5 : 4) kernels.
cudaError_t sort_grouped_ticks(const int32_t* ticks, const uint32_t* off, int G, uint32_t total, uint64_t* keys_a,
                               uint64_t* keys_b, uint32_t* counts, int32_t* err, int32_t* out, int sms, cudaStream_t st);
// Checked build: 0, or DISCO_ECUDA (error string set) if a kernel refused an index since the last call.  Always 0 in
// an ordinary build.  To be called after the stream has been synchronised.
int check_debug_record();
#ifdef DISCO_DEBUG
// Launches a kernel whose only access uses an index beyond its bound (refused by the check, never made).
cudaError_t run_debug_selftest(cudaStream_t st);
#endif
// Times the token loop's instruction mix on every multiprocessor; *token_steps_per_s receives the rate.
cudaError_t run_alu_peak(int sms, double* token_steps_per_s, cudaStream_t st);

}  // namespace disco
