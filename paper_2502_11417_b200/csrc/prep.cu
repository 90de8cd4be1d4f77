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
    return DBG_OK(k, N, DBG_K_PREP, DBG_ELEMENT) ? sorted[k] : 0;
}

// Smallest x in [lo, hi) with pred(x), or hi if there is none; pred is false up to some point and true from
// there on.  Fifteen probes a round instead of one: the probes of a round are independent loads, so the search
// over the 4098 cumulative masses takes four rounds of memory latency instead of thirteen.
template <class F>
__device__ __forceinline__ int first_true(int lo, int hi, F pred) {
    while (hi - lo > 16) {
        const int step = (hi - lo + 15) >> 4;
        bool f[15];
#pragma unroll
        for (int k = 0; k < 15; ++k) { const int x = lo + (k + 1) * step; f[k] = x < hi ? pred(x) : true; }
        int k0 = 15;                                                  // first probe that holds
#pragma unroll
        for (int k = 14; k >= 0; --k) if (f[k]) k0 = k;
        const int nlo = k0 == 0 ? lo : lo + k0 * step + 1;            // the probe before it failed
        const int nhi = k0 == 15 ? hi : min(hi, lo + (k0 + 1) * step);
        lo = nlo; hi = nhi;
    }
    bool f[16];
#pragma unroll
    for (int k = 0; k < 16; ++k) { const int x = lo + k; f[k] = x < hi ? pred(x) : true; }
    int k0 = 16;
#pragma unroll
    for (int k = 15; k >= 0; --k) if (f[k]) k0 = k;
    return min(lo + k0, hi);
}

__global__ void k_prep(const PolicyConst* __restrict__ pol, uint32_t P, int G, const GroupConst* __restrict__ gc,
                       const int64_t* __restrict__ cum_mass, const uint32_t* __restrict__ cnt,
                       const int32_t* __restrict__ sorted, const uint32_t* __restrict__ grp_off,
                       Prep* __restrict__ prep) {
    const uint32_t idx = blockIdx.x * blockDim.x + threadIdx.x;
    if (idx >= P * (uint32_t)G) return;
    const int g = (int)(idx / P);
    const uint32_t p = idx % P;
    if (!DBG_OK(g, G, DBG_K_PREP, DBG_GROUP)) return;
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
    r.beta_rule = 0;

    if (!r.device_constrained) {
        // Eq. 3: smallest L with device-only mass sum_{l<L} l cnt[l] >= (1-b) Total
        const double target = __dmul_rn(__dsub_rn(1.0, b), Total);
        r.l_th = first_true(0, kMaxPrompt + 1, [&](int L) {                                         // in [0, 4097]
            return DBG_OK(L, kMaxPrompt + 2, DBG_K_PREP, DBG_TABLE) ? (double)cum[L] >= target : true; });
    } else {
        // Algorithm 2, phase 1: tail protection
        const double q_tail = __dsub_rn(1.0, fmin(alpha, b));
        r.w_tail = inverse_cdf(srt, N, q_tail);
        if (pc.flags & DISCO_FLAG_BETA_RULE) {
            // Eq. 1-2 variant: the slope is found by k_prep_beta; until then every wait is w_tail
            r.beta_rule = 1;
            r.l_star = b <= alpha ? 0 : (int32_t)pc.l_immediate;
            r.w_star = r.w_tail + 1;
        } else if (b <= alpha) {
            r.l_star = 0; r.w_star = r.w_tail;
        } else {
            // phase 2: A input tokens may start the device at once; shortest prompts first
            const double A = __dmul_rn(__ddiv_rn(__dsub_rn(b, alpha), __dsub_rn(1.0, alpha)), Total);
            // first length whose cumulative mass exceeds A; 4097 = every class is funded
            const int lo = first_true(0, kMaxPrompt + 1, [&](int l) {
                return DBG_OK(l + 1, kMaxPrompt + 2, DBG_K_PREP, DBG_TABLE) ? (double)cum[l + 1] > A : true; });
            r.l_star = lo;
            if (lo <= kMaxPrompt && DBG_OK(lo, kMaxPrompt + 1, DBG_K_PREP, DBG_TABLE)) {
                const double f = __ddiv_rn(__dsub_rn(A, (double)cum[lo]), __dmul_rn((double)lo, (double)c[lo]));
                r.w_star = inverse_cdf(srt, N, __dmul_rn(__dsub_rn(1.0, alpha), __dsub_rn(1.0, f)));
            }
        }
    }
    prep[(size_t)g * P + p] = r;
}

// Eq. 1-2 variant of phase 2, one block per (group, policy): the smallest whole slope beta (ticks per prompt
// token) with  sum_l l cnt[l] #{S > w(l)} <= b Total N,  w(l) = 0 for l <= l_immediate, min(beta l, w_tail) above.
// The sum is exact (it is below Total N < 2^63); it does not grow with beta, so beta is found by bisection.
__global__ void __launch_bounds__(256)
k_prep_beta(const PolicyConst* __restrict__ pol, uint32_t P, const int64_t* __restrict__ cum_mass,
            const uint32_t* __restrict__ cnt, const int32_t* __restrict__ sorted, const uint32_t* __restrict__ grp_off,
            Prep* __restrict__ prep) {
    __shared__ long long part[8];
    __shared__ long long total_s;
    const int g = (int)(blockIdx.x / P);
    const uint32_t p = blockIdx.x % P;
    Prep& out = prep[(size_t)g * P + p];
    const Prep pr = out;
    const PolicyConst pc = pol[p];
    if (!pr.beta_rule || !pr.device_constrained || (double)pc.budget <= (double)pc.alpha) return;   // block-uniform
    const uint32_t off = grp_off[g], N = grp_off[g + 1] - off;
    const int32_t* srt = sorted + off;
    const uint32_t* c = cnt + (size_t)g * (kMaxPrompt + 1);
    const double Total = (double)cum_mass[(size_t)g * (kMaxPrompt + 2) + kMaxPrompt + 1];
    const double limit = __dmul_rn(__dmul_rn((double)pc.budget, Total), (double)N);
    const long long w_tail = pr.w_tail, l_imm = pr.l_star;

    auto started_tokens = [&](long long beta) -> long long {
        long long acc = 0;
        for (int l = 1 + (int)threadIdx.x; l <= kMaxPrompt; l += 256) {
            const uint32_t k = c[l];
            if (k == 0) continue;
            const long long w = l <= l_imm ? 0 : min(beta * (long long)l, w_tail);
            uint32_t lo = 0, hi = N;                                  // requests with S <= w
            while (lo < hi) {
                const uint32_t mid = (lo + hi) >> 1;
                if (!DBG_OK(mid, N, DBG_K_PREP, DBG_ELEMENT)) break;
                if ((long long)srt[mid] <= w) lo = mid + 1; else hi = mid;
            }
            acc += (long long)l * (long long)k * (long long)(N - lo);
        }
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) acc += __shfl_xor_sync(0xFFFFFFFFu, acc, o);
        __syncthreads();
        if ((threadIdx.x & 31) == 0) part[threadIdx.x >> 5] = acc;
        __syncthreads();
        if (threadIdx.x == 0) { long long t = 0; for (int k = 0; k < 8; ++k) t += part[k]; total_s = t; }
        __syncthreads();
        return total_s;
    };
    long long lo = 0, hi = w_tail + 1;                                // beyond hi every wait is w_tail
    if ((double)started_tokens(hi) <= limit) {
        while (lo < hi) {
            const long long mid = lo + (hi - lo) / 2;
            if ((double)started_tokens(mid) <= limit) hi = mid; else lo = mid + 1;
        }
    } else {
        lo = hi;                                                      // not even the longest waits fit
    }
    if (threadIdx.x == 0) out.w_star = (int32_t)lo;
}

}  // namespace

DBG_TRANSLATION_UNIT()

cudaError_t launch_prep(const PolicyConst* pol, uint32_t P, int G, const GroupConst* gc, const int64_t* cum_mass,
                        const uint32_t* cnt, const int32_t* sorted, const uint32_t* grp_off, Prep* prep,
                        cudaStream_t st) {
    const uint32_t total = P * (uint32_t)G;
    k_prep<<<(total + 127) / 128, 128, 0, st>>>(pol, P, G, gc, cum_mass, cnt, sorted, grp_off, prep);
    return cudaGetLastError();
}

cudaError_t launch_prep_beta(const PolicyConst* pol, uint32_t P, int G, const int64_t* cum_mass, const uint32_t* cnt,
                             const int32_t* sorted, const uint32_t* grp_off, Prep* prep, cudaStream_t st) {
    k_prep_beta<<<P * (uint32_t)G, 256, 0, st>>>(pol, P, cum_mass, cnt, sorted, grp_off, prep);
    return cudaGetLastError();
}

}  // namespace disco
