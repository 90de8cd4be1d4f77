// Decode play-out (Sec. 4.3): one warp per request, every token of every stream.
//
// A stream's delivery times follow d_1 = 0, d_j = max(g_j, d_{j-1} + tau) over generation times
// g_j = g_{j-1} + x_j, x_j = T + jitter(hash(seed, request, j)).  With e_j = d_j - g_j (how far delivery lags
// generation) and c_j = tau - x_j this is the recurrence e_j = max(0, e_{j-1} + c_j), and
// TBT_j = tau + (e_j - (e_{j-1} + c_j)).  The map e -> max(r, e + s) is closed under composition, so a warp
// plays a request in rounds of 32 lanes x up to 8 consecutive tokens: every lane hashes its tokens, the
// lanes' maps are combined by a shuffle scan, and each lane replays its tokens from its true state.  When
// no c_j of a round is negative nothing clamps: every TBT equals tau and the round reduces to one sum.
//
// Streams per request: S (server decodes all), D (device decodes all) share the hash draws and run
// together; X (the dearer winner hands off after token m) runs as a second pass once m is known.
#include <climits>

#include "disco_internal.cuh"

namespace disco {

namespace {

constexpr int kR = 8;                    // tokens per lane and round
constexpr int kRing = 512;               // delivery times kept per warp for the buffer test
constexpr int kWarps = 8;                // warps (requests) per block
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

__device__ __forceinline__ void count_slow(uint32_t tbt, uint32_t* win, int lo, int W, int32_t* err) {
    const int b = bin_of_ticks(tbt) - lo;
    if (b >= 0 && b < W) atomicAdd(&win[b], 1u); else atomicExch(&err[2], 1);
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
__device__ uint32_t find_handoff_sequential(uint32_t key, int32_t c_base, uint32_t mul, int32_t tau, uint32_t B,
                                            uint32_t n) {
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

// One round of streams S or D.  `search`: this is the candidate stream and the hand-off index is still
// unknown; then m_out receives it when the buffer first holds B tokens (d_{j-B+1} > g_j) in this round.
__device__ __forceinline__ void play_round(WS& st, uint32_t& mxl, uint32_t& ntl, const int32_t (&c)[kR],
                                           const Round& rd, uint32_t* win, int lo, int W, bool search, uint32_t B,
                                           int32_t thr, uint32_t& clean_until, uint32_t* ring, uint32_t& m_out) {
    int32_t s = 0, mn = 0;
#pragma unroll
    for (int t = 0; t < kR; ++t)
        if (t < rd.cper) { s += c[t]; mn = min(mn, c[t]); }
    const bool fast = rd.pacing && __all_sync(FULL, mn >= 0) && !(search && !st.clean);
    if (fast) {                                         // no clamp: every TBT of the round equals tau
        const int32_t tot = __reduce_add_sync(FULL, s);
        if (search) {
            // clean stream: d_q = (q-1) tau, so d_{j-B+1} > g_j  <=>  S_j > (B-1) tau, and S is non-decreasing
            if (st.S + tot > thr) {
                int32_t si = s;
#pragma unroll
                for (int off = 1; off < 32; off <<= 1) {
                    const int32_t sp = __shfl_up_sync(FULL, si, off);
                    if (rd.lane >= off) si += sp;
                }
                int32_t run = st.S + si - s;
                uint32_t first = kNone;
#pragma unroll
                for (int t = 0; t < kR; ++t)
                    if (t < rd.cnt) {
                        run += c[t];
                        const uint32_t j = rd.j0 + t;
                        if (first == kNone && run > thr && j + 1 <= rd.n) first = j;
                    }
                const uint32_t found = __reduce_min_sync(FULL, first);
                if (found != kNone) m_out = found;
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

__global__ void __launch_bounds__(kWarps * 32)
k_playout(TraceDev tr, const GroupConst* __restrict__ gcs, const ClassConst* __restrict__ ccp,
          const int32_t* __restrict__ knots, uint32_t k0, TimelineRec rec, int32_t* err) {
    __shared__ uint32_t ring_s[kWarps][kRing];
    const int lane = threadIdx.x & 31, wib = threadIdx.x >> 5;
    const uint32_t k = blockIdx.x * kWarps + wib;
    if (k >= tr.n) return;
    uint32_t* ring = ring_s[wib];
    int g = 0;
    while (g + 1 < tr.n_groups && k >= tr.grp_off[g + 1]) ++g;
    const GroupConst gc = gcs[g];
    const ClassConst& cc = *ccp;
    const uint32_t n = tr.nout[k], l = tr.l[k];
    const uint32_t nI = n - 1;                                        // inter-token intervals, tokens 2..n
    const uint32_t key = mix32(k0 + tr.orig[k] * kHashReq);
    const int32_t tau_eff = cc.tau_eff, tau = cc.tau;
    const bool pacing = cc.pacing != 0;
    const int W0 = cc.W[0], W1 = cc.W[1], W2 = cc.W[2];
    const int lo0 = cc.lo[g][0], lo1 = cc.lo[g][1], lo2 = cc.lo[g][2];
    uint32_t* win0 = rec.win[0] + (size_t)k * W0;
    uint32_t* win1 = rec.win[1] + (size_t)k * W1;
    uint32_t* win2 = rec.win[2] + (size_t)k * W2;
    for (int i = lane; i < W0; i += 32) win0[i] = 0;
    for (int i = lane; i < W1; i += 32) win1[i] = 0;
    for (int i = lane; i < W2; i += 32) win2[i] = 0;
    __syncwarp();

    const uint32_t mulS = 2u * (uint32_t)gc.J_srv + 1u, mulD = 2u * (uint32_t)gc.J_dev + 1u;
    const int32_t cS_base = tau_eff - (gc.T_srv - gc.J_srv), cD_base = tau_eff - (gc.T_dev - gc.J_dev);
    const int cand = (cc.mig_any && n >= 2) ? gc.candidate : 0;      // 1: server stream may hand off, 2: device stream
    const uint32_t B = (uint32_t)cc.B;
    const long long thr64 = (long long)(B ? B - 1 : 0) * tau;
    const int32_t thr = thr64 > INT_MAX ? INT_MAX : (int32_t)thr64;

    Round rd;
    rd.lane = lane; rd.n = n; rd.tau_eff = tau_eff; rd.pacing = pacing; rd.err = err;
    rd.cper = (int)min((uint32_t)kR, (nI + 31u) / 32u);
    const uint32_t span = 32u * (uint32_t)rd.cper;

    WS sS = {0, 0, 0, true}, sD = {0, 0, 0, true};
    uint32_t mxS = 0, ntS = 0, mxD = 0, ntD = 0;
    uint32_t m = (cand && B == 0) ? 1u : 0u;                           // nothing to fill: hand off after token 1
    uint32_t clean_until = 1;

    for (uint32_t base = 0; base < nI; base += span) {
        const uint32_t idx0 = base + (uint32_t)lane * rd.cper;
        rd.cnt = idx0 >= nI ? 0 : (int)min((uint32_t)rd.cper, nI - idx0);
        rd.j0 = idx0 + 2;
        rd.round_valid = min(span, nI - base);
        rd.last_j = base + rd.round_valid + 1;
        int32_t cs[kR], cd[kR];
        uint32_t hin = key + rd.j0 * kHashTok;
#pragma unroll
        for (int t = 0; t < kR; ++t) {
            cs[t] = 0; cd[t] = 0;
            if (t < rd.cper) {
                const uint32_t h = mix32(hin);
                hin += kHashTok;
                if (t < rd.cnt) {
                    cs[t] = cS_base - (int32_t)__umulhi(h, mulS);     // tau - (T + jitter), jitter in [-J, J]
                    cd[t] = cD_base - (int32_t)__umulhi(h, mulD);
                }
            }
        }
        bool searchS = cand == 1 && m == 0, searchD = cand == 2 && m == 0;
        // buffers deeper than the ring: once the candidate stream clamps, one lane searches sequentially
        if ((searchS || searchD) && B > kRing / 2) {
            const int32_t(&cc_)[kR] = searchS ? cs : cd;
            int32_t mn = 0;
#pragma unroll
            for (int t = 0; t < kR; ++t) mn = min(mn, cc_[t]);
            if (!__all_sync(FULL, mn >= 0)) {
                uint32_t mm = 0;
                if (lane == 0)
                    mm = find_handoff_sequential(key, searchS ? cS_base : cD_base, searchS ? mulS : mulD, tau, B, n);
                mm = __shfl_sync(FULL, mm, 0);
                m = mm ? mm : kNone;                                   // kNone: searched, never fills
                searchS = searchD = false;
            }
        }
        uint32_t m_new = 0;
        play_round(sS, mxS, ntS, cs, rd, win0, lo0, W0, searchS, B, thr, clean_until, ring, m_new);
        play_round(sD, mxD, ntD, cd, rd, win1, lo1, W1, searchD, B, thr, clean_until, ring, m_new);
        if (m_new) m = m_new;
    }
    if (m == kNone) m = 0;

    // ---- summaries of S and D
    {
        const uint32_t tS = sS.nt + __reduce_add_sync(FULL, ntS), tD = sD.nt + __reduce_add_sync(FULL, ntD);
        const uint32_t xS = __reduce_max_sync(FULL, mxS), xD = __reduce_max_sync(FULL, mxD);
        __syncwarp();
        if (lane == 0) {
            const int ktS = cc.ktau[g][0], ktD = cc.ktau[g][1];
            if (ktS >= 0 && tS) atomicAdd(&win0[ktS], tS);
            if (ktD >= 0 && tD) atomicAdd(&win1[ktD], tD);
            rec.sum[0][k] = (uint32_t)((int32_t)nI * tau_eff - sS.S + sS.e);       // d_n - d_1 = g_n + e_n
            rec.sum[1][k] = (uint32_t)((int32_t)nI * tau_eff - sD.S + sD.e);
            rec.max[0][k] = nI ? (uint32_t)tau_eff + xS : 0u;
            rec.max[1][k] = nI ? (uint32_t)tau_eff + xD : 0u;
        }
    }

    // ---- stream X: the candidate's tokens up to m, then the target after the hand-off latency M
    uint32_t stall = 0, delayed = 0, sumX = 0, maxX = 0;
    if (m) {
        uint32_t M;
        if (cand == 1) {
            M = (uint32_t)gc.kappa * (l + m) + (uint32_t)gc.c0;        // device re-prefills prompt + generated tokens
        } else {
            const uint32_t u = mix32(key);                             // a server TTFT drawn from F by its knots
            const int32_t* K = knots + g * kNKnots;
            const uint32_t kk = u >> 24, fr = (u >> 8) & 0xFFFFu;
            M = (uint32_t)(K[kk] + (int32_t)(((int64_t)(K[kk + 1] - K[kk]) * (int64_t)fr) >> 16));
        }
        const int32_t cM = tau_eff - (int32_t)M;
        const uint32_t mulC = cand == 1 ? mulS : mulD, mulT = cand == 1 ? mulD : mulS;
        const int32_t cC_base = cand == 1 ? cS_base : cD_base, cT_base = cand == 1 ? cD_base : cS_base;
        WS sX = {0, 0, 0, true};
        uint32_t mxX = 0, ntX = 0, dl = 0;
        int32_t D0 = 0;                                                // e_m - S_m: slot lag of token j is -(D0 + S_j)
        bool D0_known = false;
        for (uint32_t base = 0; base < nI; base += span) {
            const uint32_t idx0 = base + (uint32_t)lane * rd.cper;
            rd.cnt = idx0 >= nI ? 0 : (int)min((uint32_t)rd.cper, nI - idx0);
            rd.j0 = idx0 + 2;
            rd.round_valid = min(span, nI - base);
            rd.last_j = base + rd.round_valid + 1;
            int32_t cx[kR];
            uint32_t hin = key + rd.j0 * kHashTok;
            int32_t s = 0, mn = 0;
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
                    s += cx[t]; mn = min(mn, cx[t]);
                }
            }
            const bool special = base + 2 <= m + 1 && rd.last_j >= m;        // round holds token m or m+1
            const bool late = pacing && D0_known && D0 + sX.S < 0;           // tokens may still miss their slots
            const bool fast = pacing && !special && !late && __all_sync(FULL, mn >= 0);
            if (fast) {
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
                    else count_slow((uint32_t)tau_eff + ex, win2, lo2, W2, err);
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
        const uint32_t tX = sX.nt + __reduce_add_sync(FULL, ntX);
        maxX = (uint32_t)tau_eff + __reduce_max_sync(FULL, mxX);
        stall = __reduce_max_sync(FULL, stall);
        delayed = __reduce_add_sync(FULL, dl);
        sumX = (uint32_t)((int32_t)nI * tau_eff - sX.S + sX.e);
        __syncwarp();
        const int ktX = cc.ktau[g][2];
        if (lane == 0 && ktX >= 0 && tX) atomicAdd(&win2[ktX], tX);
    }
    if (lane == 0) {
        rec.sum[2][k] = sumX; rec.max[2][k] = maxX; rec.stall[k] = stall;
        rec.m[k] = (uint16_t)m; rec.delayed[k] = (uint16_t)delayed;
    }
}

}  // namespace

cudaError_t launch_timeline(const TraceDev& tr, const GroupConst* gc, const ClassConst* cc, const int32_t* knots,
                            uint64_t seed, TimelineRec rec, int32_t* err, cudaStream_t st) {
    if (tr.n == 0) return cudaSuccess;
    k_playout<<<(tr.n + kWarps - 1) / kWarps, kWarps * 32, 0, st>>>(tr, gc, cc, knots, seed_key(seed), rec, err);
    return cudaGetLastError();
}

}  // namespace disco
