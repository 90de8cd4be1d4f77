// Final reductions per policy (Sec. 5.1 metrics: mean and tail TTFT, P99 TBT, cost) and policy selection.
#include "disco_internal.cuh"

namespace disco {

namespace {

__device__ __forceinline__ double bin_edge_seconds(int b) {
    long long edge = b < 32 ? b : ((long long)(32 + (b & 31)) << ((b >> 5) - 1));
    return __dmul_rn((double)edge, 1e-6);
}

// Nearest-rank quantiles of one 864-bin histogram by a warp: lane i owns bins [27 i, 27 i + 27); the bin
// holding the ceil(q*M)-th smallest item is found from the lanes' prefix counts.  All lanes return the bins.
constexpr int kBinsPerLane = kNBins / 32;
static_assert(kBinsPerLane * 32 == kNBins, "864 bins split evenly over a warp");

__device__ void warp_quantile_bins(const unsigned long long* hist, unsigned long long M, const double* qs, int nq,
                                   int* out) {
    const int lane = threadIdx.x & 31;
    unsigned long long mine[kBinsPerLane], sum = 0;
#pragma unroll
    for (int i = 0; i < kBinsPerLane; ++i) { mine[i] = hist[lane * kBinsPerLane + i]; sum += mine[i]; }
    unsigned long long incl = sum;
#pragma unroll
    for (int off = 1; off < 32; off <<= 1) {
        const unsigned long long v = __shfl_up_sync(0xFFFFFFFFu, incl, off);
        if (lane >= off) incl += v;
    }
    const unsigned long long excl = incl - sum;
    for (int k = 0; k < nq; ++k) {
        int bin = 0;
        if (M) {
            unsigned long long rank = (unsigned long long)ceil(__dmul_rn(qs[k], (double)M));
            if (rank < 1) rank = 1;
            int found = -1;
            if (rank > excl && rank <= incl) {
                unsigned long long acc = excl;
#pragma unroll
                for (int i = 0; i < kBinsPerLane; ++i) {
                    acc += mine[i];
                    if (found < 0 && acc >= rank) found = lane * kBinsPerLane + i;
                }
            }
            const unsigned owner = __ballot_sync(0xFFFFFFFFu, found >= 0);
            bin = owner ? __shfl_sync(0xFFFFFFFFu, found, __ffs(owner) - 1) : kNBins - 1;
            if (!DBG_OK(bin, kNBins, DBG_K_FINALIZE, DBG_BIN)) bin = kNBins - 1;
        }
        out[k] = bin;
    }
}

// One block of 32 threads per policy.
__global__ void k_finalize(uint32_t P, int G, const GroupConst* __restrict__ gc,
                           const unsigned long long* __restrict__ acc, const unsigned long long* __restrict__ hist_ttft,
                           const unsigned long long* __restrict__ hist_tbt,
                           const unsigned long long* __restrict__ fin_totals,
                           disco_policy_stats_t* __restrict__ stats, disco_policy_stats_t* __restrict__ stats_host,
                           const int32_t* __restrict__ err) {
    // stats_host: the caller's pinned mirror, written straight from here (no copy operation behind the kernel)
    const uint32_t p = blockIdx.x;
    grid_dependency_wait();
    if (p == 0 && threadIdx.x < 4) {                                                           // error word rides along
        ((int32_t*)(stats + P))[threadIdx.x] = err[threadIdx.x];
        ((int32_t*)(stats_host + P))[threadIdx.x] = err[threadIdx.x];
    }
    __shared__ unsigned long long tot[kNAcc];
    __shared__ int qb[4];
    // fin_totals: output tokens and requests per group behind the accumulators (this trace's, or what a caller
    // merged from several shards)
    const unsigned long long* grp_sum_n = fin_totals;
    unsigned long long N = 0;
    for (int g = 0; g < G; ++g) N += fin_totals[G + g];
    if (threadIdx.x < kNAcc) {
        unsigned long long s = 0;
        for (int g = 0; g < G; ++g) s += acc[((size_t)p * G + g) * kNAcc + threadIdx.x];
        tot[threadIdx.x] = s;
    }
    unsigned long long sum_n = 0;
    for (int g = 0; g < G; ++g) sum_n += grp_sum_n[g];
    {
        const double q_ttft[3] = {0.50, 0.95, 0.99}, q_tbt[1] = {0.99};
        int b3[3], b1[1];
        warp_quantile_bins(hist_ttft + (size_t)p * kNBins, N, q_ttft, 3, b3);
        warp_quantile_bins(hist_tbt + (size_t)p * kNBins, sum_n - N, q_tbt, 1, b1);
        if (threadIdx.x == 0) { qb[0] = b3[0]; qb[1] = b3[1]; qb[2] = b3[2]; qb[3] = b1[0]; }
    }
    __syncthreads();
    if (threadIdx.x != 0) return;
    // Eq. 8 on the exact integer token totals of each group
    double cost = 0.0;
    unsigned long long tok_dev = 0;
    for (int g = 0; g < G; ++g) {
        const unsigned long long* a = acc + ((size_t)p * G + g) * kNAcc;
        const double dts = (double)(grp_sum_n[g] - a[A_TOK_DEVICE]), dtd = (double)a[A_TOK_DEVICE];
        const double pts = (double)a[A_PRE_SERVER], ptd = (double)a[A_PRE_DEVICE];
        const GroupConst& c = gc[g];
        const double srv = __dadd_rn(__dmul_rn(c.cps_d, pts), __dmul_rn(c.cds_d, dts));
        const double dev = __dadd_rn(__dmul_rn(c.cpd_d, ptd), __dmul_rn(c.cdd_d, dtd));
        cost = __dadd_rn(cost, __dadd_rn(srv, __dmul_rn(c.lambda_d, dev)));
        tok_dev += a[A_TOK_DEVICE];
    }
    disco_policy_stats_t s;
    const unsigned long long ttft_ticks = tot[A_TTFT_SUM];
    s.mean_ttft_s = N ? __ddiv_rn(__dmul_rn((double)ttft_ticks, 1e-6), (double)N) : 0.0;
    s.total_cost = cost;
    s.bin_p50_ttft = qb[0]; s.bin_p95_ttft = qb[1]; s.bin_p99_ttft = qb[2]; s.bin_p99_tbt = qb[3];
    s.p50_ttft_s = (float)bin_edge_seconds(qb[0]); s.p95_ttft_s = (float)bin_edge_seconds(qb[1]);
    s.p99_ttft_s = (float)bin_edge_seconds(qb[2]); s.p99_tbt_s = (float)bin_edge_seconds(qb[3]);
    s.n_requests = N; s.n_intervals = sum_n - N;
    s.n_device_only = tot[A_DEVICE_ONLY]; s.n_race = tot[A_RACE];
    s.n_server_only = N - s.n_device_only - s.n_race;          // every request takes exactly one decision
    s.n_device_started = s.n_device_only + s.n_race;           // the device ran in both of these
    s.n_device_won = tot[A_DEVICE_WON]; s.n_migrations = tot[A_MIGR];
    s.tok_device = tok_dev; s.tok_server = sum_n - tok_dev;
    s.prefill_tok_server = tot[A_PRE_SERVER]; s.prefill_tok_device = tot[A_PRE_DEVICE];
    s.delayed_tokens = tot[A_DELAYED];
    stats[p] = s;
    stats_host[p] = s;
}

// Lexicographic objective of the selection: (tail TTFT bin, mean TTFT, cost, index), feasible policies only.
struct Pick { int feasible; int bin; double mean, cost; int idx; };

__device__ __forceinline__ bool better(const Pick& a, const Pick& b) {
    if (b.idx < 0) return a.idx >= 0;
    if (a.idx < 0) return false;
    if (a.feasible != b.feasible) return a.feasible > b.feasible;
    if (a.feasible) {
        if (a.bin != b.bin) return a.bin < b.bin;
        if (a.mean != b.mean) return a.mean < b.mean;
        if (a.cost != b.cost) return a.cost < b.cost;
    } else {
        if (a.cost != b.cost) return a.cost < b.cost;        // none feasible: cheapest
    }
    return a.idx < b.idx;
}

__global__ void k_select(const disco_policy_stats_t* __restrict__ stats, uint32_t P, double cost_cap, double tbt_slo,
                         int32_t* __restrict__ result) {
    __shared__ Pick best[256];
    Pick mine = {0, 0, 0.0, 0.0, -1};
    for (uint32_t p = threadIdx.x; p < P; p += blockDim.x) {
        const disco_policy_stats_t& s = stats[p];
        Pick c;
        c.feasible = (s.total_cost <= cost_cap) && (bin_edge_seconds(s.bin_p99_tbt) <= tbt_slo);
        c.bin = s.bin_p99_ttft; c.mean = s.mean_ttft_s; c.cost = s.total_cost; c.idx = (int)p;
        if (better(c, mine)) mine = c;
    }
    best[threadIdx.x] = mine;
    __syncthreads();
    for (int off = 128; off > 0; off >>= 1) {
        if ((int)threadIdx.x < off && better(best[threadIdx.x + off], best[threadIdx.x]))
            best[threadIdx.x] = best[threadIdx.x + off];
        __syncthreads();
    }
    if (threadIdx.x == 0) {
        result[0] = best[0].feasible ? 0 : DISCO_EINFEASIBLE;
        result[1] = best[0].idx;
    }
}

}  // namespace

DBG_TRANSLATION_UNIT()

cudaError_t launch_finalize(uint32_t P, int G, const GroupConst* gc, const uint64_t* acc, const uint64_t* hist_ttft,
                            const uint64_t* hist_tbt, const uint64_t* fin_totals,
                            disco_policy_stats_t* stats, disco_policy_stats_t* stats_host, const int32_t* err,
                            cudaStream_t st) {
    return launch_after(k_finalize, P, 32, 0, st, P, G, gc, (const unsigned long long*)acc,
                        (const unsigned long long*)hist_ttft, (const unsigned long long*)hist_tbt,
                        (const unsigned long long*)fin_totals, stats, stats_host, err);
}

cudaError_t launch_select(const disco_policy_stats_t* stats, uint32_t P, double cost_cap, float tbt_slo_s,
                          int32_t* result, cudaStream_t st) {
    k_select<<<1, 256, 0, st>>>(stats, P, cost_cap, (double)tbt_slo_s, result);
    return cudaGetLastError();
}

}  // namespace disco
