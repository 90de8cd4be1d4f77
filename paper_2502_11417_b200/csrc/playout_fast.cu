// Decode play-out (Sec. 4.3) for requests whose streams never clamp: both endpoints generate every token
// no slower than it is consumed (c_j = tau - x_j >= 0 for all j), so delivery is exactly tau-paced.
//
// A warp plays four or eight requests at a time and shares its 32 lanes among them by their token counts (every
// lane then owns a contiguous run of about the same length, whatever the mix of lengths).
// Every token's hash is drawn and mapped to both endpoints' jitter; the lane keeps the sums and maxima.  If any c_j is negative the request is put on a list for the general kernel (playout.cu).
// Otherwise:
//  * streams S and D: every TBT equals tau;
//  * hand-off index m (buffer holds B tokens: d_{j-B+1} > g_j) is the first j whose prefix sum of c on the
//    candidate stream exceeds (B-1) tau; the owning lane re-draws its run up to that token;
//  * stream X: token m+1 waits for the hand-off latency M; it is `need` = M - e_m - tau late if that is
//    positive, and each later token of the target stream gains its c_j until the lag is made up.
#include <algorithm>

#include "disco_internal.cuh"

namespace disco {

namespace {

constexpr uint32_t FULL = 0xFFFFFFFFu;
constexpr int kFastWarps = 8;

struct LaneGroup {                       // constants of a lane's current request group
    uint32_t mulS, mulD;
    int32_t cS_base, cD_base, kappa, c0;
    int cand;
    const int32_t* K;
};

// Inclusive prefix sum over the lanes of a team (q = lane's position in its team); all 32 lanes call it.
__device__ __forceinline__ int32_t team_inclusive_sum(int32_t v, int q) {
#pragma unroll
    for (int off = 1; off < 32; off <<= 1) {
        const int32_t p = __shfl_up_sync(FULL, v, off);
        if (q >= off) v += p;
    }
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


// rpw = requests per warp (8, 16 or 32): small traces use small batches so that enough warps are in flight.
// LEAN: the host has checked that tau >= T + J for both endpoints of every group, so no interval can exceed
// tau and every request is clamp-free by construction.  Then only the candidate stream's sums are needed to
// find the hand-off index; the target stream is drawn only for the tokens right after a hand-off that stalls.
template <bool LEAN, int PER>
__global__ void __launch_bounds__(kFastWarps * 32)
k_playout_fast(TraceDev tr, const GroupConst* __restrict__ gcs, const ClassConst* __restrict__ ccp,
               const int32_t* __restrict__ knots, uint32_t k0, TimelineRec rec, uint32_t* __restrict__ todo,
               uint32_t* __restrict__ todo_count, uint32_t* __restrict__ tickets, int rpw, uint32_t one) {
    const int lane = threadIdx.x & 31;
    grid_dependency_wait();
    const ClassConst& cc = *ccp;
    const int32_t tau = cc.tau;                                   // pacing is on for every launch of this kernel
    const uint32_t B = (uint32_t)cc.B;
    const long long thr64 = (long long)(B ? B - 1 : 0) * tau;
    const int32_t thr = thr64 > 0x7FFFFFFFLL ? 0x7FFFFFFF : (int32_t)thr64;
    const int W0 = cc.W[0], W1 = cc.W[1], W2 = cc.W[2];
    const bool mig_any = cc.mig_any != 0;

    LaneGroup G;
    int cur_g = -1;
    // Batches of rpw requests are handed out by a ticket counter (zero at launch), so a warp that drew short
    // requests takes more of them and the last batches are spread over the whole GPU.
    for (;;) {
        uint32_t ticket = 0;
        if (lane == 0) ticket = atomicAdd(tickets, 1u);
        const uint32_t batch0 = __shfl_sync(FULL, ticket, 0) * (uint32_t)rpw;
        if (batch0 >= tr.n) break;
        // ---- one request per lane: inputs
        const uint32_t kk = batch0 + lane;
        const bool live = lane < rpw && kk < tr.n;
        uint32_t n_l = 1, l_l = 1, key_l = 0;
        int g_l = 0;
        if (live) {
            n_l = tr.nout[kk]; l_l = tr.l[kk];
            key_l = mix32(k0 + tr.orig[kk] * kHashReq);
            while (g_l + 1 < tr.n_groups && kk >= tr.grp_off[g_l + 1]) ++g_l;
        }
        // ---- one request per lane: results (bit 31 of o_md: played here; bits 0-15 m, 16-30 late tokens)
        uint32_t o_md = 0, o_stall = 0;

        for (int it = 0; it < rpw / PER; ++it) {
            // ---- share the lanes among the PER requests: one lane for each request that has intervals, the
            //      other lanes in proportion to the intervals (n - 1 each).  Any split that gives such a request
            //      a lane is valid; the rounding only moves load.  Every group of PER lanes holds the same
            //      PER values here, lane s of a group standing for request r0 + s.
            const int r0 = it * PER, s8 = lane & (PER - 1);
            const uint32_t nI_s = __shfl_sync(FULL, n_l, r0 + s8) - 1;
            uint32_t inc = nI_s;
#pragma unroll
            for (int off = 1; off < PER; off <<= 1) {
                const uint32_t up = __shfl_up_sync(FULL, inc, off, PER);
                if (s8 >= off) inc += up;
            }
            const uint32_t tot = __shfl_sync(FULL, inc, PER - 1, PER);
            const uint32_t busy = __ballot_sync(FULL, nI_s != 0) & ((1u << PER) - 1u);   // requests with intervals
            const float per = __fdividef((float)(32 - __popc(busy)), (float)max(tot, 1u));
            // first lane of request s: requests with intervals before it, plus its share of the spare lanes
            const int start_s = __popc(busy & ((1u << s8) - 1u)) + __float2int_rn((float)(inc - nI_s) * per);
            const bool owner_s = lane < PER && nI_s != 0;
            const uint32_t starts = __reduce_or_sync(FULL, owner_s ? 1u << start_s : 0u);   // bit 0 is set unless tot == 0
            // request of the k-th team (teams in request order), four bits each
            const uint32_t team_req = __reduce_or_sync(FULL, owner_s ? (uint32_t)s8 << (4 * __popc(busy & ((1u << s8) - 1u))) : 0u);
            const uint32_t upto = starts & (0xFFFFFFFFu >> (31 - lane));           // team starts at or below this lane
            const uint32_t after = starts & ~(0xFFFFFFFFu >> (31 - lane));
            const int a = upto ? 31 - __clz(upto) : 0;
            const int a_next = after ? __ffs(after) - 1 : 32;
            const int lanes = a_next - a, q = lane - a;
            const uint32_t tmask = lanes == 32 ? FULL : (((1u << lanes) - 1u) << a);   // this team's lanes: teams may diverge
            const int r = r0 + (int)((team_req >> (4 * max(__popc(upto) - 1, 0))) & 7u);
            const uint32_t n = __shfl_sync(FULL, n_l, r), l = __shfl_sync(FULL, l_l, r);
            const uint32_t key = __shfl_sync(FULL, key_l, r);
            const int g = __shfl_sync(FULL, g_l, r);
            if (g != cur_g && DBG_OK(g, tr.n_groups, DBG_K_PLAYOUT_FAST, DBG_GROUP)) {
                cur_g = g;
                const GroupConst& gc = gcs[g];
                G.mulS = 2u * (uint32_t)gc.J_srv + 1u; G.mulD = 2u * (uint32_t)gc.J_dev + 1u;
                G.cS_base = tau - (gc.T_srv - gc.J_srv); G.cD_base = tau - (gc.T_dev - gc.J_dev);
                G.kappa = gc.kappa; G.c0 = gc.c0;
                G.cand = mig_any ? gc.candidate : 0;
                G.K = knots + g * kNKnots;
            }
            const uint32_t nI = tot ? n - 1 : 0u;                      // inter-token intervals, tokens 2..n
            // tokens per lane, ceil(nI / lanes) or one more (lanes >= 1 here); all that matters is lanes * L >= nI
            uint32_t L = __float2uint_ru(__fdividef((float)nI, (float)lanes));
            if (L * (uint32_t)lanes < nI) ++L;
            const uint32_t lo = (uint32_t)q * L;
            const int cnt = lo >= nI ? 0 : (int)min(L, nI - lo);
            const uint32_t j0 = lo + 2;

            // ---- every token: hash draw and both endpoints' jitter, ((h * (2J+1)) >> 32)
            const int Lmax = (int)__reduce_max_sync(FULL, L);
            uint32_t hin = key + j0 * kHashTok;
            int32_t s_S = 0, s_D = 0;
            bool clean = true;
            if (LEAN) {
                const uint32_t mul = G.cand == 2 ? G.mulD : G.mulS;    // the stream of the endpoint that may hand over
                uint32_t hC = 0;
    #pragma unroll 4
                for (int t = 0; t < Lmax; ++t) {
                    const uint32_t x = __umulhi(mix32(hin), mul);
                    hin += kHashTok;
                    if (t < cnt) hC = x * one + hC;        // `one` = 1: a multiply-add, off the busy integer pipe
                }
                s_S = s_D = cnt * (G.cand == 2 ? G.cD_base : G.cS_base) - (int32_t)hC;
            } else {
                uint32_t hS = 0, hD = 0, xS = 0, xD = 0;
    #pragma unroll 4
                for (int t = 0; t < Lmax; ++t) {
                    uint32_t h = mix32(hin);
                    hin += kHashTok;
                    h = t < cnt ? h : 0u;
                    const uint32_t x = __umulhi(h, G.mulS), y = __umulhi(h, G.mulD);
                    hS += x; hD += y; xS = max(xS, x); xD = max(xD, y);
                }
                s_S = cnt * G.cS_base - (int32_t)hS; s_D = cnt * G.cD_base - (int32_t)hD;
                const bool neg = cnt != 0 && ((int32_t)xS > G.cS_base || (int32_t)xD > G.cD_base);   // some c_j < 0
                clean = (__ballot_sync(FULL, neg) & tmask) == 0;
                if (nI != 0 && !clean && q == 0) {                     // for the general kernel
                    const uint32_t at = atomicAdd(todo_count, 1u);
                    if (DBG_OK(at, tr.n, DBG_K_PLAYOUT_FAST, DBG_REQUEST)) todo[at] = batch0 + r;
                }
            }
            const bool go = clean && nI != 0;
            // ---- hand-off index on the candidate stream
            const int cand = go ? G.cand : 0;
            const int32_t sC = cand == 1 ? s_S : s_D, sT = cand == 1 ? s_D : s_S;
            const int32_t inC = team_inclusive_sum(sC, q), inT = LEAN ? 0 : team_inclusive_sum(sT, q);
            const uint32_t mulC = cand == 1 ? G.mulS : G.mulD, mulT = cand == 1 ? G.mulD : G.mulS;
            const int32_t cC_base = cand == 1 ? G.cS_base : G.cD_base, cT_base = cand == 1 ? G.cD_base : G.cS_base;
            uint32_t m = 0;
            int32_t e_m = 0;
            if (cand && B == 0) m = 1;                                 // nothing to fill: hand off after token 1
            const uint32_t crossers = __ballot_sync(FULL, cand && B != 0 && inC > thr) & tmask;
            if (crossers) {                                            // team-uniform from here on
                const int owner = __ffs(crossers) - 1;                 // first lane whose run takes the sum past thr
                uint32_t j_found = 0;
                int32_t run = inC - sC;
                if (lane == owner) {
                    bool hit;
                    const uint32_t passed = walk(key, j0, 0, cnt, cC_base, mulC, thr, true, run, hit);
                    j_found = j0 + passed;                             // hit is certain: the run's total exceeds thr
                }
                j_found = __shfl_sync(tmask, j_found, owner);
                e_m = __shfl_sync(tmask, run, owner);                  // clean stream: e_m = S_m
                m = j_found + 1 <= n ? j_found : 0u;                   // the hand-off needs a token left to generate
            }
            // ---- stream X
            uint32_t stall = 0, delayed = 0;
            int32_t need_lean = 0;                                     // LEAN: how late token m+1 is, if it stalls
            if (m) {                                                   // team-uniform
                uint32_t M;
                if (cand == 1) M = (uint32_t)G.kappa * (l + m) + (uint32_t)G.c0;       // device re-prefills prompt + m tokens
                else {
                    const uint32_t u = mix32(key);                     // a server TTFT drawn from F by its knots
                    const uint32_t ki = u >> 24, fr = (u >> 8) & 0xFFFFu;
                    M = 0;
                    if (DBG_OK(ki + 1, kNKnots, DBG_K_PLAYOUT_FAST, DBG_KNOT))
                        M = (uint32_t)(G.K[ki] + (int32_t)(((int64_t)(G.K[ki + 1] - G.K[ki]) * (int64_t)fr) >> 16));
                }
                const int32_t v = e_m + (tau - (int32_t)M);            // slot lag of token m+1, negated
                stall = (uint32_t)tau + (uint32_t)max(-v, 0);
                if (LEAN) need_lean = max(-v, 0);
                if (!LEAN && v < 0) {
                    // tokens m+2.. stay late while the target's prefix sum of c is below `need`
                    const int32_t need = -v;
                    const uint32_t first_idx = m;                      // run-global index (j - 2) of token m+2
                    const int qs = (int)min((uint32_t)(lanes - 1), first_idx / L);
                    int32_t runA = 0;
                    uint32_t contrib = 0;
                    bool hitA = false;
                    if (q == qs && first_idx < nI)
                        contrib = walk(key, j0, (int)(first_idx - lo), cnt, cT_base, mulT, need, false, runA, hitA);
                    runA = __shfl_sync(tmask, runA, a + qs);
                    hitA = __shfl_sync(tmask, (int)hitA, a + qs) != 0;
                    const int32_t inT_qs = __shfl_sync(tmask, inT, a + qs);
                    if (!hitA && q > qs && cnt) {
                        const int32_t through = runA + (inT - inT_qs);               // target's sum up to this run's end
                        int32_t before = through - sT;
                        if (through < need) contrib = (uint32_t)cnt;
                        else if (before < need) { bool hit; contrib = walk(key, j0, 0, cnt, cT_base, mulT, need, false, before, hit); }
                    }
                    delayed = 1u + __reduce_add_sync(tmask, contrib);
                }
            }
            if (LEAN) {
                // tokens m+2.. stay late while the target's prefix sum of c (from token m+2) is below the lag.  The
                // team draws `lanes` tokens of the target stream a round until the sum gets there (c >= 0: the
                // late tokens are a prefix).  All 32 lanes run the rounds; teams that are done draw nothing.
                bool more = need_lean > 0 && m + 2 <= n;
                uint32_t jb = m + 2, late = 0;
                int32_t carry = 0;
                while (__any_sync(FULL, more)) {
                    const uint32_t j = jb + (uint32_t)q;
                    const bool in = more && j <= n;
                    const int32_t c = in ? cT_base - (int32_t)__umulhi(mix32(key + j * kHashTok), mulT) : 0;
                    const int32_t R = carry + team_inclusive_sum(c, q);
                    late += __popc(__ballot_sync(FULL, in && R < need_lean) & tmask);
                    const bool reached = (__ballot_sync(FULL, in && R >= need_lean) & tmask) != 0;
                    carry = __shfl_sync(FULL, R, a + lanes - 1);
                    jb += (uint32_t)lanes;
                    more = more && !reached && jb <= n;
                }
                if (need_lean > 0) delayed = 1u + late;
            }
            // ---- hand the results to the lanes that own the requests' slots
            const uint32_t packed = (nI == 0 || go ? 0x80000000u : 0u) | m | (delayed << 16);
            const uint32_t got_md = __shfl_sync(FULL, packed, start_s & 31), got_stall = __shfl_sync(FULL, stall, start_s & 31);
            if (lane / PER == it) {
                const bool has_lanes = nI_s != 0;                      // no lanes: a single-token request, all zeros
                o_md = has_lanes ? got_md : 0x80000000u;
                o_stall = has_lanes ? got_stall : 0u;
            }
        }
        __syncwarp();
        // ---- one request per lane: results out
        if (live && (o_md >> 31) && DBG_OK(kk, tr.n, DBG_K_PLAYOUT_FAST, DBG_REQUEST) &&
            DBG_OK(g_l, kMaxGroups, DBG_K_PLAYOUT_FAST, DBG_GROUP)) {
            const uint32_t nI = n_l - 1, ut = (uint32_t)tau, m = o_md & 0xFFFFu, dl = (o_md >> 16) & 0x7FFFu;
            rec.sum[0][kk] = nI * ut; rec.max[0][kk] = nI ? ut : 0u;
            rec.sum[1][kk] = nI * ut; rec.max[1][kk] = nI ? ut : 0u;
            rec.sum[2][kk] = m ? (nI - 1) * ut + o_stall : 0u; rec.max[2][kk] = m ? o_stall : 0u;
            rec.stall[kk] = m ? o_stall : 0u; rec.m[kk] = (uint16_t)m; rec.delayed[kk] = (uint16_t)(m ? dl : 0u);
            const int kt0 = cc.ktau[g_l][0], kt1 = cc.ktau[g_l][1], kt2 = cc.ktau[g_l][2];
            for (int i = 0; i < W0; ++i) rec.win[0][(size_t)kk * W0 + i] = i == kt0 ? nI : 0u;
            for (int i = 0; i < W1; ++i) rec.win[1][(size_t)kk * W1 + i] = i == kt1 ? nI : 0u;
            for (int i = 0; i < W2; ++i) rec.win[2][(size_t)kk * W2 + i] = (i == kt2 && m) ? nI - 1 : 0u;
        }
    }
}

}  // namespace

DBG_TRANSLATION_UNIT()

cudaError_t launch_playout_fast(const TraceDev& tr, const GroupConst* gc, const ClassConst* cc, const int32_t* knots,
                                uint32_t k0, TimelineRec rec, uint32_t* todo, uint32_t* todo_count,
                                bool never_clamps, bool long_outputs, int sms, cudaStream_t st) {
    if (tr.n == 0) return cudaSuccess;
    // requests per ticket: small batches spread the end of the launch evenly; large traces amortise the ticket
    int rpw = 8;
    while (rpw < 32 && (uint64_t)tr.n / (2 * rpw) >= (uint64_t)sms * 48u * 4u) rpw *= 2;
    const uint32_t per_block = kFastWarps * (uint32_t)rpw;
    // requests per round: eight halve the cost of a round per request; with long outputs the token loop is
    // what counts, and four requests split the lanes more evenly
    auto* kernel = never_clamps ? (long_outputs ? k_playout_fast<true, 4> : k_playout_fast<true, 8>)
                                : (long_outputs ? k_playout_fast<false, 4> : k_playout_fast<false, 8>);
    // as many blocks as the GPU holds at once (at most six of these per SM); the ticket counter feeds them
    const uint32_t blocks = std::min<uint32_t>((tr.n + per_block - 1) / per_block, (uint32_t)sms * 6u);
    return launch_after(kernel, blocks, kFastWarps * 32, 0, st, tr, gc, cc, knots, k0, rec, todo, todo_count,
                        todo_count + 1, rpw, 1u);
}

}  // namespace disco
