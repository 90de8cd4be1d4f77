// Decode play-out (Sec. 4.3) for requests whose streams never clamp: both endpoints generate every token
// no slower than it is consumed (c_j = tau - x_j >= 0 for all j), so delivery is exactly tau-paced.
//
// Teams of eight lanes play one request each, four requests per warp at a time; a lane owns a contiguous
// run of tokens.  Every token's hash is drawn and mapped to both endpoints' jitter; the lane keeps the sums
// and maxima.  If any c_j is negative the request is put on a list for the general kernel (playout.cu).
// Otherwise:
//  * streams S and D: every TBT equals tau;
//  * hand-off index m (buffer holds B tokens: d_{j-B+1} > g_j) is the first j whose prefix sum of c on the
//    candidate stream exceeds (B-1) tau; the owning lane re-draws its run up to that token;
//  * stream X: token m+1 waits for the hand-off latency M; it is `need` = M - e_m - tau late if that is
//    positive, and each later token of the target stream gains its c_j until the lag is made up.
#include "disco_internal.cuh"

namespace disco {

namespace {

constexpr uint32_t FULL = 0xFFFFFFFFu;
constexpr int kTeam = 8;
constexpr int kFastWarps = 8;

struct LaneGroup {                       // constants of a lane's current request group
    uint32_t mulS, mulD;
    int32_t cS_base, cD_base, kappa, c0;
    int cand;
    const int32_t* K;
};

__device__ __forceinline__ int32_t team_inclusive_sum(int32_t v, int q) {
#pragma unroll
    for (int off = 1; off < kTeam; off <<= 1) {
        const int32_t p = __shfl_up_sync(FULL, v, off, kTeam);
        if (q >= off) v += p;
    }
    return v;
}

__device__ __forceinline__ uint32_t team_sum(uint32_t v, uint32_t tmask) {
#pragma unroll
    for (int off = 1; off < kTeam; off <<= 1) v += __shfl_xor_sync(tmask, v, off, kTeam);
    return v;
}

// Walks the lane's own tokens from run-local index t0, adding c = base - ((h * mul) >> 32) to `run`, and
// stops at the first token where run exceeds `limit` (strict) or reaches it (strict == false).
// Returns the number of tokens passed before that one; `hit` says whether one was found.
__device__ __forceinline__ uint32_t walk(uint32_t key, uint32_t j0, int t0, int cnt, int32_t base, uint32_t mul,
                                         int32_t limit, bool strict, int32_t& run, bool& hit) {
    uint32_t passed = 0;
    uint32_t hin = key + (j0 + (uint32_t)t0) * kHashTok;
    hit = false;
    for (int t = t0; t < cnt; ++t) {
        const int32_t c = base - (int32_t)__umulhi(mix32(hin), mul);
        hin += kHashTok;
        run += c;
        if (strict ? run > limit : run >= limit) { hit = true; break; }
        ++passed;
    }
    return passed;
}

__global__ void __launch_bounds__(kFastWarps * 32)
k_playout_fast(TraceDev tr, const GroupConst* __restrict__ gcs, const ClassConst* __restrict__ ccp,
               const int32_t* __restrict__ knots, uint32_t k0, TimelineRec rec, uint32_t* __restrict__ todo,
               uint32_t* __restrict__ todo_count) {
    const int lane = threadIdx.x & 31, wib = threadIdx.x >> 5;
    const int team = lane >> 3, q = lane & 7;
    const uint32_t tmask = 0xFFu << (team * kTeam);               // the lanes of this team: teams may diverge
    const uint32_t batch0 = (blockIdx.x * kFastWarps + wib) * 32u;
    if (batch0 >= tr.n) return;
    const ClassConst& cc = *ccp;
    const int32_t tau = cc.tau;                                   // pacing is on for every launch of this kernel
    const uint32_t B = (uint32_t)cc.B;
    const long long thr64 = (long long)(B ? B - 1 : 0) * tau;
    const int32_t thr = thr64 > 0x7FFFFFFFLL ? 0x7FFFFFFF : (int32_t)thr64;
    const int W0 = cc.W[0], W1 = cc.W[1], W2 = cc.W[2];
    const bool mig_any = cc.mig_any != 0;

    // ---- one request per lane: inputs
    const uint32_t kk = batch0 + lane;
    const bool live = kk < tr.n;
    uint32_t n_l = 1, l_l = 1, key_l = 0;
    int g_l = 0;
    if (live) {
        n_l = tr.nout[kk]; l_l = tr.l[kk];
        key_l = mix32(k0 + tr.orig[kk] * kHashReq);
        while (g_l + 1 < tr.n_groups && kk >= tr.grp_off[g_l + 1]) ++g_l;
    }
    // ---- one request per lane: results (request team*8 + it is kept by lane q == it of its team)
    uint32_t o_sumX = 0, o_stall = 0, o_m = 0, o_dl = 0;
    bool o_done = false;

    LaneGroup G;
    int cur_g = -1;
    const int n_here = (int)min(32u, tr.n - batch0);

    for (int it = 0; it < kTeam; ++it) {
        const int r = team * kTeam + it;
        const uint32_t n = __shfl_sync(FULL, n_l, r), l = __shfl_sync(FULL, l_l, r);
        const uint32_t key = __shfl_sync(FULL, key_l, r);
        const int g = __shfl_sync(FULL, g_l, r);
        const bool active = r < n_here;
        if (g != cur_g) {
            cur_g = g;
            const GroupConst& gc = gcs[g];
            G.mulS = 2u * (uint32_t)gc.J_srv + 1u; G.mulD = 2u * (uint32_t)gc.J_dev + 1u;
            G.cS_base = tau - (gc.T_srv - gc.J_srv); G.cD_base = tau - (gc.T_dev - gc.J_dev);
            G.kappa = gc.kappa; G.c0 = gc.c0;
            G.cand = mig_any ? gc.candidate : 0;
            G.K = knots + g * kNKnots;
        }
        const uint32_t nI = active ? n - 1 : 0u;                   // inter-token intervals, tokens 2..n
        const uint32_t L = (nI + kTeam - 1) / kTeam;               // tokens per lane
        const uint32_t lo = (uint32_t)q * L;
        const int cnt = lo >= nI ? 0 : (int)min(L, nI - lo);
        const uint32_t j0 = lo + 2;

        // ---- every token: hash draw and both endpoints' jitter, ((h * (2J+1)) >> 32)
        const int Lmax = (int)__reduce_max_sync(FULL, L);
        uint32_t hS = 0, hD = 0, xS = 0, xD = 0;
        uint32_t hin = key + j0 * kHashTok;
#pragma unroll 4
        for (int t = 0; t < Lmax; ++t) {
            uint32_t h = mix32(hin);
            hin += kHashTok;
            h = t < cnt ? h : 0u;
            const uint32_t a = __umulhi(h, G.mulS), b = __umulhi(h, G.mulD);
            hS += a; hD += b; xS = max(xS, a); xD = max(xD, b);
        }
        const int32_t s_S = cnt * G.cS_base - (int32_t)hS, s_D = cnt * G.cD_base - (int32_t)hD;
        const bool neg = cnt != 0 && ((int32_t)xS > G.cS_base || (int32_t)xD > G.cD_base);   // some c_j < 0
        const uint32_t team_neg = (__ballot_sync(FULL, neg) >> (team * kTeam)) & 0xFFu;
        const bool clean = team_neg == 0;
        if (active && !clean) {                                    // leave it to the general kernel
            if (q == 0) todo[atomicAdd(todo_count, 1u)] = batch0 + r;
        }
        const bool go = active && clean && nI != 0;
        // ---- hand-off index on the candidate stream
        const int cand = go ? G.cand : 0;
        const int32_t sC = cand == 1 ? s_S : s_D, sT = cand == 1 ? s_D : s_S;
        const int32_t inC = team_inclusive_sum(sC, q), inT = team_inclusive_sum(sT, q);
        const uint32_t mulC = cand == 1 ? G.mulS : G.mulD, mulT = cand == 1 ? G.mulD : G.mulS;
        const int32_t cC_base = cand == 1 ? G.cS_base : G.cD_base, cT_base = cand == 1 ? G.cD_base : G.cS_base;
        uint32_t m = 0;
        int32_t e_m = 0;
        if (cand && B == 0) m = 1;                                 // nothing to fill: hand off after token 1
        const uint32_t crossers = (__ballot_sync(FULL, cand && B != 0 && inC > thr) >> (team * kTeam)) & 0xFFu;
        if (crossers) {
            const int owner = __ffs(crossers) - 1;
            uint32_t j_found = 0;
            int32_t run = inC - sC;
            if (q == owner) {
                bool hit;
                const uint32_t passed = walk(key, j0, 0, cnt, cC_base, mulC, thr, true, run, hit);
                j_found = j0 + passed;                             // hit is certain: the run's total exceeds thr
            }
            j_found = __shfl_sync(tmask, j_found, owner, kTeam);
            e_m = __shfl_sync(tmask, run, owner, kTeam);            // clean stream: e_m = S_m
            m = j_found + 1 <= n ? j_found : 0u;                   // the hand-off needs a token left to generate
        }
        // ---- stream X
        uint32_t stall = 0, delayed = 0;
        {
            const uint32_t has_m = (__ballot_sync(FULL, m != 0) >> (team * kTeam)) & 0xFFu;   // team-uniform
            if (has_m) {
                uint32_t M;
                if (cand == 1) M = (uint32_t)G.kappa * (l + m) + (uint32_t)G.c0;   // device re-prefills prompt + m tokens
                else {
                    const uint32_t u = mix32(key);                 // a server TTFT drawn from F by its knots
                    const uint32_t ki = u >> 24, fr = (u >> 8) & 0xFFFFu;
                    M = (uint32_t)(G.K[ki] + (int32_t)(((int64_t)(G.K[ki + 1] - G.K[ki]) * (int64_t)fr) >> 16));
                }
                const int32_t v = e_m + (tau - (int32_t)M);        // slot lag of token m+1, negated
                stall = (uint32_t)tau + (uint32_t)max(-v, 0);
                const uint32_t late = __ballot_sync(tmask, v < 0);
                if (late) {
                    // tokens m+2.. stay late while the target's prefix sum of c is below `need`
                    const int32_t need = -v;
                    const uint32_t first_idx = m;                  // run-global index (j - 2) of token m+2
                    const int qs = L ? (int)min((uint32_t)(kTeam - 1), first_idx / L) : 0;
                    int32_t runA = 0;
                    uint32_t contrib = 0;
                    bool hitA = false;
                    if (q == qs && first_idx < nI)
                        contrib = walk(key, j0, (int)(first_idx - lo), cnt, cT_base, mulT, need, false, runA, hitA);
                    runA = __shfl_sync(tmask, runA, qs, kTeam);
                    hitA = __shfl_sync(tmask, (int)hitA, qs, kTeam) != 0;
                    const int32_t inT_qs = __shfl_sync(tmask, inT, qs, kTeam);
                    if (!hitA && q > qs && cnt) {
                        const int32_t through = runA + (inT - inT_qs);           // target's sum up to this run's end
                        int32_t before = through - sT;
                        if (through < need) contrib = (uint32_t)cnt;
                        else if (before < need) { bool hit; contrib = walk(key, j0, 0, cnt, cT_base, mulT, need, false, before, hit); }
                    }
                    delayed = 1u + team_sum(contrib, tmask);
                }
            }
        }
        if (q == it) {
            o_done = go || (active && nI == 0);
            o_m = m; o_stall = m ? stall : 0u; o_dl = m ? delayed : 0u;
            o_sumX = m ? (nI - 1) * (uint32_t)tau + stall : 0u;
        }
    }
    __syncwarp();
    // ---- one request per lane: results out
    if (live && o_done) {
        const uint32_t nI = n_l - 1, ut = (uint32_t)tau;
        rec.sum[0][kk] = nI * ut; rec.max[0][kk] = nI ? ut : 0u;
        rec.sum[1][kk] = nI * ut; rec.max[1][kk] = nI ? ut : 0u;
        rec.sum[2][kk] = o_sumX; rec.max[2][kk] = o_stall;
        rec.stall[kk] = o_stall; rec.m[kk] = (uint16_t)o_m; rec.delayed[kk] = (uint16_t)o_dl;
        const int kt0 = cc.ktau[g_l][0], kt1 = cc.ktau[g_l][1], kt2 = cc.ktau[g_l][2];
        for (int i = 0; i < W0; ++i) rec.win[0][(size_t)kk * W0 + i] = i == kt0 ? nI : 0u;
        for (int i = 0; i < W1; ++i) rec.win[1][(size_t)kk * W1 + i] = i == kt1 ? nI : 0u;
        for (int i = 0; i < W2; ++i) rec.win[2][(size_t)kk * W2 + i] = (i == kt2 && o_m) ? nI - 1 : 0u;
    }
}

}  // namespace

cudaError_t launch_playout_fast(const TraceDev& tr, const GroupConst* gc, const ClassConst* cc, const int32_t* knots,
                                uint64_t seed, TimelineRec rec, uint32_t* todo, uint32_t* todo_count,
                                cudaStream_t st) {
    if (tr.n == 0) return cudaSuccess;
    const uint32_t per_block = kFastWarps * 32;
    k_playout_fast<<<(tr.n + per_block - 1) / per_block, kFastWarps * 32, 0, st>>>(tr, gc, cc, knots, seed_key(seed), rec,
                                                                                    todo, todo_count);
    return cudaGetLastError();
}

}  // namespace disco
