// Decode play-out (Sec. 4.3): warps play requests cooperatively, every token of every stream.
//
// A stream's delivery times follow d_1 = 0, d_j = max(g_j, d_{j-1} + tau) over generation times
// g_j = g_{j-1} + x_j, x_j = T + jitter(hash(seed, request, j)).  With e_j = d_j - g_j (how far delivery lags
// generation) and c_j = tau - x_j this is the recurrence e_j = max(0, e_{j-1} + c_j), and
// TBT_j = tau + (e_j - (e_{j-1} + c_j)).  The map e -> max(r, e + s) is closed under composition, so a warp
// plays a request in rounds of 32 lanes x up to 8 consecutive tokens: every lane hashes its tokens, the
// lanes' maps are combined by a shuffle scan, and each lane replays its tokens from its true state.  When
// no c_j of a round is negative nothing clamps: every TBT equals tau and the round reduces to one sum.
//
// Streams per request: S (server decodes all) and D (device decodes all) share the hash draws and run
// together.  X (the dearer winner, the "candidate", hands off after token m) consists of the candidate's
// tokens up to m, one token that waits for the hand-off latency, and the other endpoint's tokens after
// it; while nothing clamps it follows from the two streams' prefix sums, otherwise it is played out in a
// second pass.
//
// A warp takes 32 consecutive requests at a time: their inputs are loaded and their results stored one
// request per lane, so the per-request memory traffic is coalesced and paid once per 32 requests.
#include <algorithm>
#include <climits>

#include "disco_internal.cuh"

namespace disco {

namespace {

constexpr int kR = 8;                    // tokens per lane and round
constexpr int kRing = 512;               // delivery times kept per warp for the buffer test
constexpr int kWarps = 8;                // warps per block
constexpr uint32_t FULL = 0xFFFFFFFFu;
constexpr uint32_t kNone = 0xFFFFFFFFu;

struct WS {                              // warp-uniform state of one stream
    int32_t e;                           // d_j - g_j after the last token played
    int32_t S;                           // sum of c over the tokens played: g_j = (j-1) tau - S
    uint32_t nt;                         // TBTs equal to tau, counted for whole rounds
    bool clean;                          // nothing has clamped yet: d_j = (j-1) tau for every token played
};

struct Round {                           // what a lane knows about the current round
    int lane, cper, cnt;                 // tokens per lane, valid tokens of this lane
    uint32_t j0, last_j, n;              // lane's first token, round's last valid token, output length
    uint32_t round_valid;                // valid tokens in the round
    int32_t tau_eff;
    bool pacing;
    int32_t* err;
};

struct GroupClass {                      // constants of the request's group under the current class
    uint32_t mulS, mulD;
    int32_t cS_base, cD_base;            // tau_eff - (T - J): c = base - ((h * (2J+1)) >> 32)
    int32_t kappa, c0;
    int cand;                            // 0 none, 1 the server stream may hand off, 2 the device stream
    int lo0, lo1, lo2, kt0, kt1, kt2;
    const int32_t* K;
};

__device__ __forceinline__ void count_slow(uint32_t tbt, uint32_t* win, int lo, int W, int32_t* err) {
    const int b = bin_of_ticks(tbt) - lo;
    if (b >= 0 && b < W && DBG_OK(b, W, DBG_K_PLAYOUT, DBG_WINDOW)) atomicAdd(&win[b], 1u); else atomicExch(&err[2], 1);
}

__device__ __forceinline__ int32_t warp_inclusive_sum(int32_t v, int lane) {
#pragma unroll
    for (int off = 1; off < 32; off <<= 1) {
        const int32_t p = __shfl_up_sync(FULL, v, off);
        if (lane >= off) v += p;
    }
    return v;
}

// State (e, S) in front of each lane's first token: exclusive shuffle scan of the lanes' maps.
__device__ __forceinline__ void lane_state(const WS& st, const int32_t (&c)[kR], const Round& rd, int32_t& e_in,
                                           int32_t& S_in, int32_t& s_total) {
    int32_t r = 0, s = 0;
#pragma unroll
    for (int t = 0; t < kR; ++t)
        if (t < rd.cper) { s += c[t]; r = max(r + c[t], 0); }
    int32_t ri = r, si = s;
#pragma unroll
    for (int off = 1; off < 32; off <<= 1) {
        const int32_t rp = __shfl_up_sync(FULL, ri, off), sp = __shfl_up_sync(FULL, si, off);
        if (rd.lane >= off) { ri = max(ri, rp + si); si += sp; }     // earlier segment first, then this one
    }
    const int32_t rx = __shfl_up_sync(FULL, ri, 1), sx = __shfl_up_sync(FULL, si, 1);
    e_in = rd.lane ? max(rx, st.e + sx) : st.e;
    S_in = st.S + (rd.lane ? sx : 0);
    s_total = __shfl_sync(FULL, si, 31);
}

// Sequential search of the hand-off index by one lane, for buffers deeper than the warp's history ring.
__device__ __noinline__ uint32_t find_handoff_sequential(uint32_t key, int32_t c_base, uint32_t mul, int32_t tau,
                                                         uint32_t B, uint32_t n) {
    int32_t e = 0, e_lag = 0, S = 0, S_lag = 0;
    uint32_t h = key + kHashTok, h_lag = key + kHashTok;
    for (uint32_t j = 2; j + 1 <= n; ++j) {
        h += kHashTok;
        const int32_t c = c_base - (int32_t)__umulhi(mix32(h), mul);
        e = max(e + c, 0); S += c;
        if (j < B) continue;
        if (j > B) {
            h_lag += kHashTok;
            const int32_t cl = c_base - (int32_t)__umulhi(mix32(h_lag), mul);
            e_lag = max(e_lag + cl, 0); S_lag += cl;
        }
        const int32_t q = (int32_t)(j - B + 1);
        if ((q - 1) * tau - S_lag + e_lag > (int32_t)(j - 1) * tau - S) return j;    // d_q > g_j
    }
    return 0;
}

// One round of stream S or D.  s = the lane's sum of c, nonneg = no c of the round is negative.
// `search`: this is the candidate stream and the hand-off index is still unknown; then m_out receives it
// when the buffer first holds B tokens (d_{j-B+1} > g_j) in this round, and, if the stream never clamped
// before, em_out its delivery lag e_m.
__device__ __forceinline__ void play_round(WS& st, uint32_t& mxl, uint32_t& ntl, const int32_t (&c)[kR], int32_t s,
                                           bool nonneg, const Round& rd, uint32_t* win, int lo, int W, bool search,
                                           uint32_t B, int32_t thr, uint32_t& clean_until, uint32_t* ring,
                                           uint32_t& m_out, int32_t& em_out) {
    if (rd.pacing && nonneg && !(search && !st.clean)) {   // no clamp: every TBT of the round equals tau
        const int32_t tot = __reduce_add_sync(FULL, s);
        if (search) {
            // clean stream: d_q = (q-1) tau, so d_{j-B+1} > g_j  <=>  S_j > (B-1) tau, and S is non-decreasing
            if (st.S + tot > thr) {
                int32_t run = st.S + warp_inclusive_sum(s, rd.lane) - s, run_first = 0;
                uint32_t first = kNone;
#pragma unroll
                for (int t = 0; t < kR; ++t)
                    if (t < rd.cnt) {
                        run += c[t];
                        const uint32_t j = rd.j0 + t;
                        if (first == kNone && run > thr && j + 1 <= rd.n) { first = j; run_first = run; }
                    }
                const uint32_t found = __reduce_min_sync(FULL, first);
                if (found != kNone) {
                    m_out = found;
                    em_out = __shfl_sync(FULL, run_first, __ffs(__ballot_sync(FULL, first == found)) - 1);
                }
            }
            clean_until = rd.last_j;
        }
        st.e += tot; st.S += tot; st.nt += rd.round_valid;
        return;
    }
    int32_t e, S_in, tot;
    lane_state(st, c, rd, e, S_in, tot);
    int32_t run = S_in;
#pragma unroll
    for (int t = 0; t < kR; ++t)
        if (t < rd.cnt) {
            const int32_t v = e + c[t];
            e = max(v, 0);
            const uint32_t ex = (uint32_t)(e - v);                                 // TBT - tau
            mxl = max(mxl, ex);
            if (rd.pacing && ex == 0) ++ntl; else count_slow((uint32_t)rd.tau_eff + ex, win, lo, W, rd.err);
            if (search) {
                run += c[t];
                const uint32_t j = rd.j0 + t;
                ring[j & (kRing - 1)] = (uint32_t)((int32_t)(j - 1) * rd.tau_eff - run + e);   // d_j
            }
        }
    st.e = __shfl_sync(FULL, e, 31);
    if (search) {
        __syncwarp();
        run = S_in;
        uint32_t first = kNone;
#pragma unroll
        for (int t = 0; t < kR; ++t)
            if (t < rd.cnt) {
                run += c[t];
                const uint32_t j = rd.j0 + t;
                if (first == kNone && j >= B && j + 1 <= rd.n) {
                    const uint32_t q = j - B + 1;
                    const int32_t dq = q <= clean_until ? (int32_t)(q - 1) * rd.tau_eff : (int32_t)ring[q & (kRing - 1)];
                    if (dq > (int32_t)(j - 1) * rd.tau_eff - run) first = j;
                }
            }
        const uint32_t found = __reduce_min_sync(FULL, first);
        if (found != kNone) m_out = found;
        __syncwarp();
    }
    st.S += tot;
    st.clean = false;
}

struct XResult { uint32_t sum, mx, stall, delayed, nt; };

__device__ __forceinline__ uint32_t handoff_latency(const GroupClass& G, uint32_t key, uint32_t l, uint32_t m) {
    if (G.cand == 1) return (uint32_t)G.kappa * (l + m) + (uint32_t)G.c0;   // device re-prefills prompt + m tokens
    const uint32_t u = mix32(key);                                          // a server TTFT drawn from F by its knots
    const uint32_t kk = u >> 24, fr = (u >> 8) & 0xFFFFu;
    if (!DBG_OK(kk + 1, kNKnots, DBG_K_PLAYOUT, DBG_KNOT)) return 0u;
    return (uint32_t)(G.K[kk] + (int32_t)(((int64_t)(G.K[kk + 1] - G.K[kk]) * (int64_t)fr) >> 16));
}

// Stream X played out token by token: the candidate's tokens up to m, the hand-off latency, then the target.
__device__ __noinline__ void play_x(const GroupClass& G, Round rd, uint32_t key, uint32_t nI, uint32_t m, uint32_t M,
                                    uint32_t* win2, int W2, XResult* out) {
    const int32_t tau_eff = rd.tau_eff;
    const bool pacing = rd.pacing;
    const int32_t cM = tau_eff - (int32_t)M;
    const uint32_t mulC = G.cand == 1 ? G.mulS : G.mulD, mulT = G.cand == 1 ? G.mulD : G.mulS;
    const int32_t cC_base = G.cand == 1 ? G.cS_base : G.cD_base, cT_base = G.cand == 1 ? G.cD_base : G.cS_base;
    WS sX = {0, 0, 0, true};
    uint32_t mxX = 0, ntX = 0, dl = 0, stall = 0;
    int32_t D0 = 0;                                                // e_m - S_m: slot lag of token j is -(D0 + S_j)
    bool D0_known = false;
    uint32_t span = 0;
    for (uint32_t base = 0; base < nI; base += span) {
        rd.cper = (int)min((uint32_t)kR, (nI - base + 31u) / 32u);
        span = 32u * (uint32_t)rd.cper;
        const uint32_t idx0 = base + (uint32_t)rd.lane * rd.cper;
        rd.cnt = idx0 >= nI ? 0 : (int)min((uint32_t)rd.cper, nI - idx0);
        rd.j0 = idx0 + 2;
        rd.round_valid = min(span, nI - base);
        rd.last_j = base + rd.round_valid + 1;
        int32_t cx[kR];
        uint32_t hin = key + rd.j0 * kHashTok;
        int32_t s = 0, neg = 0;
#pragma unroll
        for (int t = 0; t < kR; ++t) {
            cx[t] = 0;
            if (t < rd.cper) {
                const uint32_t h = mix32(hin);
                hin += kHashTok;
                if (t < rd.cnt) {
                    const uint32_t j = rd.j0 + t;
                    const bool src = j <= m;
                    const int32_t v = (src ? cC_base : cT_base) - (int32_t)__umulhi(h, src ? mulC : mulT);
                    cx[t] = j == m + 1 ? cM : v;
                }
                s += cx[t]; neg |= cx[t];
            }
        }
        const bool special = base + 2 <= m + 1 && rd.last_j >= m;        // round holds token m or m+1
        const bool late = pacing && D0_known && D0 + sX.S < 0;           // tokens may still miss their slots
        const bool nonneg = !__any_sync(FULL, neg < 0);
        if (pacing && !special && !late && nonneg) {
            const int32_t tot = __reduce_add_sync(FULL, s);
            sX.e += tot; sX.S += tot; sX.nt += rd.round_valid;
            continue;
        }
        int32_t e, S_in, tot;
        lane_state(sX, cx, rd, e, S_in, tot);
        int32_t run = S_in, em_minus_Sm = 0;
#pragma unroll
        for (int t = 0; t < kR; ++t)
            if (t < rd.cnt) {
                const uint32_t j = rd.j0 + t;
                const int32_t v = e + cx[t];
                e = max(v, 0);
                const uint32_t ex = (uint32_t)(e - v);
                mxX = max(mxX, ex);
                run += cx[t];
                if (j == m + 1) stall = (uint32_t)tau_eff + ex;          // kept apart from the regular TBTs
                else if (pacing && ex == 0) ++ntX;
                else count_slow((uint32_t)tau_eff + ex, win2, G.lo2, W2, rd.err);
                if (j == m) em_minus_Sm = e - run;
            }
        sX.e = __shfl_sync(FULL, e, 31);
        if (m >= base + 2 && m <= rd.last_j) {                           // token m is in this round (m >= 2)
            D0 = __shfl_sync(FULL, em_minus_Sm, (int)((m - 2 - base) / rd.cper));
            D0_known = true;
        } else if (m == 1 && base == 0) {
            D0 = 0; D0_known = true;                                     // e_1 = S_1 = 0
        }
        if (pacing && D0_known) {                                        // generated after d_m + (j-m) tau ?
            run = S_in;
#pragma unroll
            for (int t = 0; t < kR; ++t)
                if (t < rd.cnt) {
                    run += cx[t];
                    if (rd.j0 + t > m && D0 + run < 0) ++dl;
                }
        }
        sX.S += tot;
    }
    out->nt = sX.nt + __reduce_add_sync(FULL, ntX);
    out->mx = (uint32_t)tau_eff + __reduce_max_sync(FULL, mxX);
    out->stall = __reduce_max_sync(FULL, stall);
    out->delayed = __reduce_add_sync(FULL, dl);
    out->sum = (uint32_t)((int32_t)nI * tau_eff - sX.S + sX.e);
}

__global__ void __launch_bounds__(kWarps * 32)
k_playout(TraceDev tr, const GroupConst* __restrict__ gcs, const ClassConst* __restrict__ ccp,
          const int32_t* __restrict__ knots, uint32_t k0, TimelineRec rec, int32_t* err,
          const uint32_t* __restrict__ todo, const uint32_t* __restrict__ todo_count, uint32_t count_imm) {
    // Requests to play: todo[0 .. *todo_count), or 0 .. count_imm when there is no list.
    __shared__ uint32_t ring_s[kWarps][kRing];
    __shared__ XResult xres_s[kWarps];
    const int lane = threadIdx.x & 31, wib = threadIdx.x >> 5;
    grid_dependency_wait();
    const uint32_t count = todo_count ? *todo_count : count_imm;
    for (uint32_t batch0 = (blockIdx.x * kWarps + wib) * 32u; batch0 < count; batch0 += gridDim.x * kWarps * 32u) {
    uint32_t* ring = ring_s[wib];
    const ClassConst& cc = *ccp;
    const int32_t tau_eff = cc.tau_eff, tau = cc.tau;
    const bool pacing = cc.pacing != 0;
    const int W0 = cc.W[0], W1 = cc.W[1], W2 = cc.W[2];
    const uint32_t B = (uint32_t)cc.B;
    const long long thr64 = (long long)(B ? B - 1 : 0) * tau;
    const int32_t thr = thr64 > INT_MAX ? INT_MAX : (int32_t)thr64;

    // ---- one request per lane: inputs
    bool live = batch0 + lane < count;
    const uint32_t kk = !live ? 0u : (todo ? todo[batch0 + lane] : batch0 + lane);
    if (live && !DBG_OK(kk, tr.n, DBG_K_PLAYOUT, DBG_REQUEST)) live = false;
    uint32_t n_l = 1, l_l = 1, key_l = 0;
    int g_l = 0;
    if (live) {
        n_l = tr.nout[kk]; l_l = tr.l[kk];
        key_l = mix32(k0 + tr.orig[kk] * kHashReq);
        while (g_l + 1 < tr.n_groups && kk >= tr.grp_off[g_l + 1]) ++g_l;
        for (int i = 0; i < W0; ++i) rec.win[0][(size_t)kk * W0 + i] = 0;
        for (int i = 0; i < W1; ++i) rec.win[1][(size_t)kk * W1 + i] = 0;
        for (int i = 0; i < W2; ++i) rec.win[2][(size_t)kk * W2 + i] = 0;
    }
    __syncwarp();
    // ---- one request per lane: results
    uint32_t o_sumS = 0, o_maxS = 0, o_sumD = 0, o_maxD = 0, o_sumX = 0, o_maxX = 0, o_stall = 0, o_m = 0, o_dl = 0;
    uint32_t o_ntS = 0, o_ntD = 0, o_ntX = 0;

    GroupClass G;
    int cur_g = -1;
    Round rd;
    rd.lane = lane; rd.tau_eff = tau_eff; rd.pacing = pacing; rd.err = err;
    const int n_here = (int)min(32u, count - batch0);

    for (int r = 0; r < n_here; ++r) {
        const uint32_t n = __shfl_sync(FULL, n_l, r), l = __shfl_sync(FULL, l_l, r);
        const uint32_t key = __shfl_sync(FULL, key_l, r);
        const int g = __shfl_sync(FULL, g_l, r);
        const uint32_t k = __shfl_sync(FULL, kk, r);
        if (g != cur_g && DBG_OK(g, tr.n_groups, DBG_K_PLAYOUT, DBG_GROUP)) {
            cur_g = g;
            const GroupConst& gc = gcs[g];
            G.mulS = 2u * (uint32_t)gc.J_srv + 1u; G.mulD = 2u * (uint32_t)gc.J_dev + 1u;
            G.cS_base = tau_eff - (gc.T_srv - gc.J_srv); G.cD_base = tau_eff - (gc.T_dev - gc.J_dev);
            G.kappa = gc.kappa; G.c0 = gc.c0;
            G.cand = cc.mig_any ? gc.candidate : 0;
            G.lo0 = cc.lo[g][0]; G.lo1 = cc.lo[g][1]; G.lo2 = cc.lo[g][2];
            G.kt0 = cc.ktau[g][0]; G.kt1 = cc.ktau[g][1]; G.kt2 = cc.ktau[g][2];
            G.K = knots + g * kNKnots;
        }
        const uint32_t nI = n - 1;                                     // inter-token intervals, tokens 2..n
        if (nI == 0) continue;                                         // a single token: all results stay 0
        uint32_t* win0 = rec.win[0] + (size_t)k * W0;
        uint32_t* win1 = rec.win[1] + (size_t)k * W1;
        uint32_t* win2 = rec.win[2] + (size_t)k * W2;
        const int cand = G.cand;
        rd.n = n;
        WS sS = {0, 0, 0, true}, sD = {0, 0, 0, true};
        uint32_t mxS = 0, ntS = 0, mxD = 0, ntD = 0;
        uint32_t m = (cand && B == 0) ? 1u : 0u;                       // nothing to fill: hand off after token 1
        int32_t e_m = 0;                                               // candidate's delivery lag at m
        bool m_clean = m != 0;                                         // candidate never clamped up to m
        uint32_t clean_until = 1;
        // Hand-off stream while nothing clamps: token m+1 is generated `need` ticks after its slot and every
        // later token of the target gains its c on the pace; dl_clean counts the tokens still late.
        uint32_t M = 0, dl_clean = 0;
        int32_t v_m1 = 0, need = 0, carry = 0;
        bool counting = false;
        if (m && pacing) {
            M = handoff_latency(G, key, l, m);
            v_m1 = tau_eff - (int32_t)M;
            if (v_m1 < 0) { counting = true; need = -v_m1; dl_clean = 1; }
        }

        uint32_t span = 0;
        for (uint32_t base = 0; base < nI; base += span) {
            rd.cper = (int)min((uint32_t)kR, (nI - base + 31u) / 32u);
            span = 32u * (uint32_t)rd.cper;
            const uint32_t idx0 = base + (uint32_t)lane * rd.cper;
            rd.cnt = idx0 >= nI ? 0 : (int)min((uint32_t)rd.cper, nI - idx0);
            rd.j0 = idx0 + 2;
            rd.round_valid = min(span, nI - base);
            rd.last_j = base + rd.round_valid + 1;
            // every token's hash draw and both endpoints' jitter: sums and maxima of ((h * (2J+1)) >> 32)
            uint32_t hS = 0, hD = 0, xS = 0, xD = 0;
            uint32_t hin = key + rd.j0 * kHashTok;
#pragma unroll
            for (int t = 0; t < kR; ++t)
                if (t < rd.cper) {
                    uint32_t h = mix32(hin);
                    hin += kHashTok;
                    h = t < rd.cnt ? h : 0u;
                    const uint32_t a = __umulhi(h, G.mulS), b = __umulhi(h, G.mulD);
                    hS += a; hD += b; xS = max(xS, a); xD = max(xD, b);
                }
            const int32_t s_S = rd.cnt * G.cS_base - (int32_t)hS, s_D = rd.cnt * G.cD_base - (int32_t)hD;
            const bool posS = __all_sync(FULL, rd.cnt == 0 || (int32_t)xS <= G.cS_base);    // c = tau - x >= 0
            const bool posD = __all_sync(FULL, rd.cnt == 0 || (int32_t)xD <= G.cD_base);
            const int32_t totS = __reduce_add_sync(FULL, s_S), totD = __reduce_add_sync(FULL, s_D);
            const bool searching = cand != 0 && m == 0;
            const bool cand_clean = cand == 1 ? sS.clean : sD.clean;
            const int32_t cand_after = cand == 1 ? sS.S + totS : sD.S + totD;
            if (pacing && posS && posD && !counting && !(searching && (!cand_clean || cand_after > thr))) {
                // nothing clamps, the buffer does not fill in this round: every TBT equals tau
                sS.e += totS; sS.S += totS; sS.nt += rd.round_valid;
                sD.e += totD; sD.S += totD; sD.nt += rd.round_valid;
                if (searching) clean_until = rd.last_j;
                continue;
            }
            // ---- the round needs its tokens one by one
            int32_t cs[kR], cd[kR];
            hin = key + rd.j0 * kHashTok;
#pragma unroll
            for (int t = 0; t < kR; ++t) {
                cs[t] = 0; cd[t] = 0;
                if (t < rd.cper) {
                    const uint32_t h = mix32(hin);
                    hin += kHashTok;
                    if (t < rd.cnt) {
                        cs[t] = G.cS_base - (int32_t)__umulhi(h, G.mulS);     // tau - (T + jitter in [-J, J])
                        cd[t] = G.cD_base - (int32_t)__umulhi(h, G.mulD);
                    }
                }
            }
            bool searchS = cand == 1 && m == 0, searchD = cand == 2 && m == 0;
            // buffers deeper than the ring: once the candidate stream clamps, one lane searches sequentially
            if ((searchS || searchD) && B > kRing / 2 && !(searchS ? posS : posD)) {
                uint32_t mm = 0;
                if (lane == 0)
                    mm = find_handoff_sequential(key, searchS ? G.cS_base : G.cD_base, searchS ? G.mulS : G.mulD, tau,
                                                 B, n);
                mm = __shfl_sync(FULL, mm, 0);
                m = mm ? mm : kNone;                                   // kNone: searched, the buffer never fills
                searchS = searchD = false;
            }
            uint32_t m_new = 0;
            play_round(sS, mxS, ntS, cs, s_S, posS, rd, win0, G.lo0, W0, searchS, B, thr, clean_until, ring, m_new, e_m);
            play_round(sD, mxD, ntD, cd, s_D, posD, rd, win1, G.lo1, W1, searchD, B, thr, clean_until, ring, m_new, e_m);
            if (m_new) {
                m = m_new;
                m_clean = cand_clean && (cand == 1 ? sS.clean : sD.clean);
                if (m_clean) {
                    M = handoff_latency(G, key, l, m);
                    v_m1 = e_m + (tau_eff - (int32_t)M);
                    if (v_m1 < 0) { counting = true; need = -v_m1; dl_clean = 1; }
                }
            }
            if (counting) {                                            // tokens m+2.. of this round on the target stream
                int32_t ct[kR], sc = 0;
#pragma unroll
                for (int t = 0; t < kR; ++t) {
                    ct[t] = (t < rd.cnt && rd.j0 + t >= m + 2) ? (cand == 1 ? cd[t] : cs[t]) : 0;
                    sc += ct[t];
                }
                const int32_t incl = warp_inclusive_sum(sc, lane);
                int32_t run = carry + incl - sc;
                uint32_t here = 0;
#pragma unroll
                for (int t = 0; t < kR; ++t)
                    if (t < rd.cnt && rd.j0 + t >= m + 2) { run += ct[t]; here += run < need; }
                dl_clean += __reduce_add_sync(FULL, here);
                carry += __shfl_sync(FULL, incl, 31);
                if (carry >= need) counting = false;
            }
        }
        if (m == kNone) m = 0;

        // ---- summaries of S and D
        const uint32_t tS = sS.nt + __reduce_add_sync(FULL, ntS), tD = sD.nt + __reduce_add_sync(FULL, ntD);
        const uint32_t r_sumS = (uint32_t)((int32_t)nI * tau_eff - sS.S + sS.e);       // d_n - d_1 = g_n + e_n
        const uint32_t r_sumD = (uint32_t)((int32_t)nI * tau_eff - sD.S + sD.e);
        const uint32_t r_maxS = (uint32_t)tau_eff + __reduce_max_sync(FULL, mxS);
        const uint32_t r_maxD = (uint32_t)tau_eff + __reduce_max_sync(FULL, mxD);

        // ---- stream X
        XResult xr = {0, 0, 0, 0, 0};
        if (m) {
            const bool target_clean = cand == 1 ? sD.clean : sS.clean;
            if (pacing && m_clean && target_clean) {
                // nothing clamps but the hand-off itself: tokens up to m and after m+1 are delivered tau apart
                xr.stall = (uint32_t)tau_eff + (uint32_t)max(-v_m1, 0);
                xr.nt = nI - 1;
                xr.sum = (nI - 1) * (uint32_t)tau_eff + xr.stall;
                xr.mx = xr.stall;
                xr.delayed = v_m1 < 0 ? dl_clean : 0u;
            } else {
                if (!(pacing && m_clean)) M = handoff_latency(G, key, l, m);
                play_x(G, rd, key, nI, m, M, win2, W2, &xres_s[wib]);
                __syncwarp();
                xr = xres_s[wib];
                __syncwarp();
            }
        }
        if (lane == r) {
            o_sumS = r_sumS; o_maxS = r_maxS; o_sumD = r_sumD; o_maxD = r_maxD; o_ntS = tS; o_ntD = tD;
            o_sumX = xr.sum; o_maxX = xr.mx; o_stall = xr.stall; o_m = m; o_dl = xr.delayed; o_ntX = xr.nt;
        }
    }
    __syncwarp();
    // ---- one request per lane: results out
    if (live) {
        rec.sum[0][kk] = o_sumS; rec.max[0][kk] = o_maxS;
        rec.sum[1][kk] = o_sumD; rec.max[1][kk] = o_maxD;
        rec.sum[2][kk] = o_sumX; rec.max[2][kk] = o_maxX;
        rec.stall[kk] = o_stall; rec.m[kk] = (uint16_t)o_m; rec.delayed[kk] = (uint16_t)o_dl;
        const int kt0 = cc.ktau[g_l][0], kt1 = cc.ktau[g_l][1], kt2 = cc.ktau[g_l][2];
        if (kt0 >= 0 && o_ntS) rec.win[0][(size_t)kk * W0 + kt0] += o_ntS;
        if (kt1 >= 0 && o_ntD) rec.win[1][(size_t)kk * W1 + kt1] += o_ntD;
        if (kt2 >= 0 && o_ntX) rec.win[2][(size_t)kk * W2 + kt2] += o_ntX;
    }
    __syncwarp();
    }   // next batch
}

}  // namespace

DBG_TRANSLATION_UNIT()

cudaError_t launch_playout_fast(const TraceDev& tr, const GroupConst* gc, const ClassConst* cc, const int32_t* knots,
                                uint32_t k0, TimelineRec rec, uint32_t* todo, uint32_t* todo_count, bool never_clamps,
                                bool long_outputs, int sms, cudaStream_t st);

// pacing: with the delivery buffer on, the clamp-free kernel plays every request it can and lists the rest
// in todo[0 .. *todo_count) (todo_count must be zero on entry); the general kernel then plays the list.
cudaError_t launch_timeline(const TraceDev& tr, const GroupConst* gc, const ClassConst* cc, bool pacing,
                            const int32_t* knots, uint32_t k0, TimelineRec rec, int32_t* err, uint32_t* todo,
                            uint32_t* todo_count, bool never_clamps, bool long_outputs, cudaEvent_t mid, int sms,
                            cudaStream_t st) {
    if (tr.n == 0) return cudaSuccess;
    const uint32_t per_block = kWarps * 32;
    if (!pacing) {
        if (mid) { cudaError_t e0 = cudaEventRecord(mid, st); if (e0) return e0; }
        const uint32_t blocks = std::min<uint32_t>((tr.n + per_block - 1) / per_block, (uint32_t)sms * 16u);
        return launch_after(k_playout, blocks, kWarps * 32, 0, st, tr, gc, cc, knots, k0, rec, err, nullptr,
                            nullptr, tr.n);
    }
    cudaError_t e = launch_playout_fast(tr, gc, cc, knots, k0, rec, todo, todo_count, never_clamps, long_outputs, sms, st);
    if (e) return e;
    if (mid && (e = cudaEventRecord(mid, st))) return e;
    if (never_clamps) return cudaSuccess;             // no interval can exceed tau: the list stays empty
    const uint32_t blocks = std::min<uint32_t>((tr.n + per_block - 1) / per_block, (uint32_t)sms * 2u);
    return launch_after(k_playout, blocks, kWarps * 32, 0, st, tr, gc, cc, knots, k0, rec, err, todo, todo_count,
                        0u);
}

}  // namespace disco
