// Policy preparation: Algorithms 1-3 for every (group, policy).
#include "disco_internal.cuh"

namespace disco {

namespace {

// ------------------------------------------------------------------------------------------------------
// Algorithms 1-3, one thread per (group, policy).  All fp64 steps use explicit round-to-nearest
// operations so that no multiply-add is contracted.
// ------------------------------------------------------------------------------------------------------
__device__ int32_t inverse_cdf(const int32_t* sorted, uint32_t N, double q) {
    if (N == 0) return 0;
    double r = ceil(__dmul_rn(q, (double)N)) - 1.0;
    long long k = (long long)r;
    if (k < 0) k = 0;
    if (k > (long long)N - 1) k = (long long)N - 1;
    return sorted[k];
}

__global__ void k_prep(const PolicyConst* __restrict__ pol, uint32_t P, int G, const GroupConst* __restrict__ gc,
                       const int64_t* __restrict__ cum_mass, const uint32_t* __restrict__ cnt,
                       const int32_t* __restrict__ sorted, const uint32_t* __restrict__ grp_off,
                       Prep* __restrict__ prep) {
    const uint32_t idx = blockIdx.x * blockDim.x + threadIdx.x;
    if (idx >= P * (uint32_t)G) return;
    const int g = (int)(idx / P);
    const uint32_t p = idx % P;
    const PolicyConst pc = pol[p];
    const int64_t* cum = cum_mass + (size_t)g * (kMaxPrompt + 2);     // cum[L] = sum_{l<L} l*cnt[l]
    const uint32_t* c = cnt + (size_t)g * (kMaxPrompt + 1);
    const uint32_t off = grp_off[g], N = grp_off[g + 1] - off;
    const int32_t* srt = sorted + off;
    const double b = (double)pc.budget, alpha = (double)pc.alpha;
    const double Total = (double)cum[kMaxPrompt + 1];

    Prep r;
    r.device_constrained = pc.mode == 1 ? 1 : pc.mode == 2 ? 0 : gc[g].auto_device_constrained;
    r.l_th = 0; r.l_star = 0; r.w_star = 0; r.w_tail = 0;
    r.theta = pc.theta;
    r.mig_on = (pc.flags & DISCO_FLAG_MIGRATION) ? 1 : 0;
    r.stochastic = (pc.flags & DISCO_FLAG_STOCHASTIC) ? 1 : 0;
    r.expected_len = pc.expected_len; r.route_thr = pc.route_thr; r.route_all = pc.route_all;
    r.pad = 0;

    if (!r.device_constrained) {
        // Eq. 3: smallest L with device-only mass sum_{l<L} l cnt[l] >= (1-b) Total
        const double target = __dmul_rn(__dsub_rn(1.0, b), Total);
        int lo = 0, hi = kMaxPrompt + 1;                              // answer in [0, 4097]
        while (lo < hi) {
            const int mid = (lo + hi) >> 1;
            if ((double)cum[mid] >= target) hi = mid; else lo = mid + 1;
        }
        r.l_th = lo;
    } else {
        // Algorithm 2, phase 1: tail protection
        const double q_tail = __dsub_rn(1.0, fmin(alpha, b));
        r.w_tail = inverse_cdf(srt, N, q_tail);
        if (b <= alpha) {
            r.l_star = 0; r.w_star = r.w_tail;
        } else {
            // phase 2: A input tokens may start the device at once; shortest prompts first
            const double A = __dmul_rn(__ddiv_rn(__dsub_rn(b, alpha), __dsub_rn(1.0, alpha)), Total);
            int lo = 0, hi = kMaxPrompt + 1;                          // first length whose cumulative mass exceeds A
            while (lo < hi) {
                const int mid = (lo + hi) >> 1;
                if ((double)cum[mid + 1] > A) hi = mid; else lo = mid + 1;
            }
            r.l_star = lo;                                             // 4097 = every class is funded
            if (lo <= kMaxPrompt) {
                const double f = __ddiv_rn(__dsub_rn(A, (double)cum[lo]), __dmul_rn((double)lo, (double)c[lo]));
                r.w_star = inverse_cdf(srt, N, __dmul_rn(__dsub_rn(1.0, alpha), __dsub_rn(1.0, f)));
            }
        }
    }
    prep[(size_t)g * P + p] = r;
}

}  // namespace

cudaError_t launch_prep(const PolicyConst* pol, uint32_t P, int G, const GroupConst* gc, const int64_t* cum_mass,
                        const uint32_t* cnt, const int32_t* sorted, const uint32_t* grp_off, Prep* prep,
                        cudaStream_t st) {
    const uint32_t total = P * (uint32_t)G;
    k_prep<<<(total + 127) / 128, 128, 0, st>>>(pol, P, G, gc, cum_mass, cnt, sorted, grp_off, prep);
    return cudaGetLastError();
}

}  // namespace disco
