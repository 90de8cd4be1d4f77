// Per-pair evaluation: dispatch decision (Algorithms 2-3, wait-then-race), TTFT, which decode stream
// applies (migration trigger, Eq. 4), tokens per endpoint and cost (Eq. 8), for every (request, policy).
//
// Two kernels share the decision logic:
//  * k_pairs_acc  -- reductions.  A lane owns a policy and walks the requests, so every per-policy sum
//    lives in registers and needs no cross-lane traffic; the TTFT histogram and the histogram of hand-off
//    stalls are block-private in shared memory (16-bit counters, two per word).
//  * k_pairs_rows -- the optional per-pair arrays.  A lane owns a request and walks the policies, so each
//    store instruction writes 32 consecutive requests of one policy row.
#include <type_traits>

#include "tile.cuh"

namespace disco {

namespace {

struct PairIn {                 // one request and its play-out summaries
    uint32_t l, n, S, m;
    float saving;               // delta_c * (n - m): Eq. 4's projected saving on the true remainder
    uint32_t u;                 // the request's routing draw (stochastic baselines only)
    float delta_c;
};

struct PairOut {
    bool dev_only, started, dev_wins, race, migr;
    uint32_t ttft;
};

// The request's draw for the stochastic baselines: the jitter hash at the reserved token index 2^32 - 1.
__device__ __forceinline__ uint32_t routing_draw(uint32_t k0, uint32_t orig) {
    return mix32(mix32(k0 + orig * kHashReq) + 0xFFFFFFFFu * kHashTok);
}

// Dispatch and race for one (request, policy); candidate = which winner may migrate in this group.
// EXT: the policy may be a Stoch-S / Stoch-D baseline or trigger migration on an expected length.
template <bool EXT>
__device__ __forceinline__ PairOut decide(const PairIn& q, const Prep& pr, uint32_t Td, int candidate) {
    PairOut o;
    o.dev_only = !pr.device_constrained && (int32_t)q.l < pr.l_th;                 // Algorithm 3
    uint32_t w = 0;                                                                // Algorithm 2's wait map
    if (pr.device_constrained)
        w = (int32_t)q.l < pr.l_star ? 0u : ((int32_t)q.l == pr.l_star ? (uint32_t)pr.w_star : (uint32_t)pr.w_tail);
    float saving = q.saving;
    if (EXT) {
        if (pr.stochastic) {                                                       // constrained endpoint with probability b
            const bool constrained = pr.route_all || q.u < pr.route_thr;
            o.dev_only = pr.device_constrained ? constrained : !constrained;
            w = 0xFFFFFFFFu;                                                       // otherwise the device never starts
        }
        else if (pr.beta_rule)                                                     // Eq. 1: min(beta l, w_tail) above l_immediate
            w = (int32_t)q.l <= pr.l_star ? 0u : (uint32_t)min((unsigned long long)(uint32_t)pr.w_star * q.l,
                                                               (unsigned long long)(uint32_t)pr.w_tail);
        if (pr.expected_len) saving = q.delta_c * (float)max((int32_t)pr.expected_len - (int32_t)q.m, 0);
    }
    o.started = o.dev_only || q.S > w;                                             // the device starts after the wait
    const uint32_t wTd = w + Td;
    o.dev_wins = o.dev_only || (o.started && q.S > wTd);                           // a tie goes to the server
    o.ttft = o.dev_only ? Td : (EXT && !o.started ? q.S : min(q.S, wTd));
    o.race = o.started && !o.dev_only;
    o.migr = pr.mig_on && o.race && q.m != 0 && candidate == (o.dev_wins ? 2 : 1) && saving > pr.theta;
    return o;
}

// ------------------------------------------------------------------------------------------------------
// Reductions: lane = policy.
//
// A pair ends in one of six outcomes, and everything it adds to the sums depends on the request and the
// outcome only.  The lane that loads a request therefore writes, once, one row of addends per outcome into
// shared memory; a policy lane decides the outcome and adds the row it selects.
//
// Tiles whose policies can be evaluated zone by zone (tile.cuh, zones.cu) have been through that kernel first:
// this one then takes only the requests it flagged for the tile in the bit mask, packed to the front of the
// staging area, and returns at once where nothing was flagged.
// ------------------------------------------------------------------------------------------------------
constexpr int kAccThreads = 512;         // one block per SM: histograms and staging fill its shared memory
constexpr int kAccWarps = kAccThreads / 32;
constexpr int kStageReq = 32;           // requests a warp stages at a time
constexpr int kIlp = 4;                 // requests a lane works on at a time
constexpr int kStageVec = 7;            // uint4 per request in each of the two staging blocks (odd: no bank conflicts)

// words in front of the staging area: two histograms and the sums, rounded up to 16 bytes
__host__ __device__ constexpr int acc_stage_offset_words(int PL) { return (2 * PL * kHWords + 2 * PL * kNAcc + 3) / 4 * 4; }

enum TileKind { K_NOWAIT = 0, K_WAIT = 1, K_ANY = 2 };

// WIDE: some stream's regular TBTs span several histogram bins (pacing off, or generation slower than
// consumption), so a pair also adds its stream's window of bins.
template <bool EXT, bool WIDE>
__global__ void __launch_bounds__(kAccThreads, 1)
k_pairs_acc(TraceDev tr, const GroupConst* __restrict__ gcs, const ClassConst* __restrict__ ccp,
            const Prep* __restrict__ prep, uint32_t P, const uint32_t* __restrict__ pol_list, uint32_t n_list,
            int PL, const Chunk* __restrict__ chunks, uint32_t n_tiles, TimelineRec rec, uint32_t k0,
            unsigned long long* __restrict__ acc, unsigned long long* __restrict__ hist_ttft,
            unsigned long long* __restrict__ hist_tbt, const uint32_t* __restrict__ left_mask,
            const uint32_t* __restrict__ left_count, const uint32_t* __restrict__ left_lists,
            unsigned long long* __restrict__ work) {
    extern __shared__ uint32_t smem[];
    uint32_t* h_ttft = smem;                                  // [PL][kHWords]
    uint32_t* h_stall = smem + PL * kHWords;                  // [PL][kHWords]
    unsigned long long* s_acc = (unsigned long long*)(smem + 2 * PL * kHWords);   // [PL][kNAcc]; 866 words per policy keep it 8-byte aligned
    grid_dependency_wait();

    // consecutive blocks take the policy tiles of one request chunk, so that the chunk is read from HBM once and
    // from L2 by the other tiles
    const uint32_t tile = blockIdx.x % n_tiles, chunk_id = blockIdx.x / n_tiles;
    const Chunk ch = chunks[chunk_id];
    const int g = ch.g;
    const int lane = threadIdx.x & 31, wib = threadIdx.x >> 5;
    const int pol_in_tile = lane % PL, slot = lane / PL, slots = 32 / PL;
    const uint32_t pol_idx = tile * PL + pol_in_tile;
    const bool act = pol_idx < n_list;
    const uint32_t p = pol_list[act ? pol_idx : 0];
    if (!DBG_OK(p, P, DBG_K_PAIRS_ACC, DBG_POLICY) || !DBG_OK(g, tr.n_groups, DBG_K_PAIRS_ACC, DBG_GROUP) ||
        (ch.len && !DBG_OK((unsigned long long)ch.start + ch.len - 1, tr.n, DBG_K_PAIRS_ACC, DBG_REQUEST)))
        return;
    const Prep pr = prep[(size_t)g * P + p];
    const int pols_here = (int)min((uint32_t)PL, n_list - tile * PL);
    // a tile that went through the zone kernel: only the requests it flagged are left (block-uniform)
    const bool flagged_only = left_mask != nullptr && left_count[(size_t)chunk_id * n_tiles + tile] != kNotByZones;
    if (flagged_only && left_count[(size_t)chunk_id * n_tiles + tile] == 0u) return;
    const uint32_t mask_words = left_words_per_request(n_tiles), mask_bit = 1u << (tile & 31u);
    const GroupConst& gc = gcs[g];
    const ClassConst& cc = *ccp;
    const uint32_t kappa = (uint32_t)gc.kappa, c0 = (uint32_t)gc.c0;
    const int candidate = gc.candidate;
    const float delta_c = gc.delta_c;
    const int W0 = cc.W[0], W1 = cc.W[1], W2 = cc.W[2];
    const int kt0 = cc.ktau[g][0], kt1 = cc.ktau[g][1], kt2 = cc.ktau[g][2];
    const uint32_t tau = (uint32_t)cc.tau;

    // With no waits in the tile (Algorithm 3, random routing) a TTFT is the request's S or its T_d, whose
    // histogram increments are staged; otherwise the bin is worked out per pair.
    const bool waits = __syncthreads_or(act && pr.device_constrained && !pr.stochastic) != 0;
    // a tile of Algorithm 2 policies alone has no device-only prompts either
    const bool all_wait = !EXT && __syncthreads_or(act && !pr.device_constrained) == 0;
    const int kind = EXT ? K_ANY : (!waits ? K_NOWAIT : (all_wait ? K_WAIT : K_ANY));
    uint32_t* my_ttft = h_ttft + pol_in_tile * kHWords;
    uint32_t* my_stall = h_stall + pol_in_tile * kHWords;

    // The block-private histogram counters are 16 bits wide: at most 65,280 requests are evaluated between two
    // flushes.  A longer chunk (one that the zone kernel left more than that of, or took nothing of) goes in passes.
    const uint32_t to_do = flagged_only ? left_count[(size_t)chunk_id * n_tiles + tile] : ch.len;
    const uint32_t pass_len = to_do <= 65280u ? ch.len : 65280u;
    for (uint32_t r_lo = 0; r_lo < ch.len; r_lo += pass_len) {
    const uint32_t r_hi = min(ch.len, r_lo + pass_len);
    for (int i = threadIdx.x; i < 2 * PL * kHWords + 2 * PL * kNAcc; i += kAccThreads) smem[i] = 0;   // (staging needs no clearing)
    __syncthreads();

    uint32_t a_td = 0, a_ps = 0, a_pd = 0, a_dl = 0, a_tau = 0;
    uint32_t cnt_a = 0, cnt_b = 0;                              // device-only | race << 16,  device won | migrated << 16
    uint32_t cnt8 = 0;                                          // the same four counts, a byte each, within a batch
    uint32_t staged = 0;                                        // requests this warp evaluated pair by pair
    unsigned long long a_tt = 0;

    // [warp][32 requests][kStageVec]: block A = the request, then the first half of each outcome's row;
    // block B = the second halves, then the stall increment and what only the extended policies read.
    uint4* stA = (uint4*)(smem + acc_stage_offset_words(PL)) + wib * kStageReq * kStageVec;
    uint4* stB = stA + kAccWarps * kStageReq * kStageVec;
    // The wait map without mode tests: Algorithm 3 has no waits (l_star beyond every length), Algorithm 2 no
    // device-only prompts (l_th = 0, as the preparation kernel leaves it).
    const int32_t l_th = pr.l_th, l_star = pr.device_constrained ? pr.l_star : 0x7FFFFFFF;
    const uint32_t w_star = (uint32_t)pr.w_star, w_tail = (uint32_t)pr.w_tail;
    // Which race winner may migrate is a property of the group; a policy without migration never passes.
    const float theta = (pr.mig_on && candidate != 0) ? pr.theta : __int_as_float(0x7F800000);
    const bool dev_migrates = candidate == 2;
    const uint32_t lth16 = (uint32_t)max(l_th, 0) << 4;      // against a staged (l << 4 | outcome at w = 0)

    // One request per lane, fetched a batch ahead so that the loads fly while the previous batch is evaluated.
    struct Raw { uint32_t l, n, S, m, dly, stall, nt0, nt1, nt2, orig; };   // as loaded: nothing may consume a load early
    auto fetch = [&](uint32_t at) {                              // the request at position `at` of the chunk
        const uint32_t kk = ch.start + min(at, r_hi - 1);
        Raw q;
        q.l = tr.l[kk]; q.n = tr.nout[kk]; q.S = (uint32_t)tr.S[kk];
        q.m = rec.m[kk]; q.dly = rec.delayed[kk]; q.stall = rec.stall[kk];
        q.nt0 = kt0 >= 0 ? rec.win[0][(size_t)kk * W0 + kt0] : 0u;
        q.nt1 = kt1 >= 0 ? rec.win[1][(size_t)kk * W1 + kt1] : 0u;
        q.nt2 = kt2 >= 0 ? rec.win[2][(size_t)kk * W2 + kt2] : 0u;
        q.orig = EXT ? tr.orig[kk] : 0u;
        return q;
    };
    // Stages the requests of the lanes in `taken`, packed to the front of the staging area, and evaluates them under
    // the tile's policies.  b0: chunk position of lane 0's request when the lanes hold a batch in order.
    auto run_batch = [&](const Raw& cur, uint32_t taken, uint32_t b0) {
        const int n_here = __popc(taken);
        staged += (uint32_t)n_here;
        if (((taken >> lane) & 1u) && DBG_OK(__popc(taken & ((1u << lane) - 1u)), kStageReq, DBG_K_PAIRS_ACC, DBG_SLOT)) {
            const int at = __popc(taken & ((1u << lane) - 1u));
            const uint32_t l = cur.l, n = cur.n, S = cur.S, m = cur.m;
            const uint32_t stall = cur.stall, dly = cur.dly;
            const uint32_t nt0 = cur.nt0, nt1 = cur.nt1;
            uint32_t nt2 = cur.nt2;
            uint32_t stall_code = 0u;                          // the token after a hand-off: counted with tau's bin,
            if (stall == tau) ++nt2; else stall_code = hist16_code(bin_of_ticks(stall));   // else an increment of its own
            // a request may only migrate if its buffer filled (m != 0); fold that into the saving (Eq. 4)
            const float saving = m ? delta_c * (float)(n - m) : -1.0f;
            const uint32_t Td = kappa * l + c0, lm = l + m;
            const uint32_t hS = hist16_code(bin_of_ticks(S)), hT = hist16_code(bin_of_ticks(Td));
            uint4* a = stA + at * kStageVec;
            uint4* b = stB + at * kStageVec;
            if (EXT || waits) {
                a[0] = make_uint4(l, S, Td, __float_as_uint(saving));
            } else {
                // no policy of the tile waits: the race at w = 0 is the request's own, and so is whether its
                // winner is the endpoint that may hand over
                const int oc0 = S > 0u ? (S > Td ? O_RACE_DEV : O_RACE_SRV) : O_SERVER_ONLY;
                const bool can = oc0 == (dev_migrates ? O_RACE_DEV : O_RACE_SRV);
                a[0] = make_uint4(l << 4 | (uint32_t)oc0, __float_as_uint(can ? saving : -1.0f), min(S, Td), Td);
            }
            //                      tokens on device, server prefill, device prefill, TBTs in tau's bin
            a[1 + O_SERVER_ONLY] = make_uint4(0u, l, 0u, nt0);
            a[1 + O_DEVICE_ONLY] = make_uint4(n, 0u, l, nt1);
            a[1 + O_RACE_SRV] = make_uint4(0u, l, l, nt0);
            a[1 + O_RACE_DEV] = make_uint4(n, l, l, nt1);
            a[1 + O_MIGR_TO_DEV] = make_uint4(n - m, l, l + lm, nt2);
            a[1 + O_MIGR_TO_SRV] = make_uint4(m, l + lm, l, nt2);
            //                      delayed tokens << 17 | stall increment, counts (a byte each: device only, race,
            //                      device won, migrated), TTFT counter pair's byte offset, TTFT increment
            const uint32_t oS = hS & 0xFFCu, iS = hS & 0x10001u, oT = hT & 0xFFCu, iT = hT & 0x10001u;
            b[O_SERVER_ONLY] = make_uint4(0u, 0x00000000u, oS, iS);
            b[O_DEVICE_ONLY] = make_uint4(0u, 0x00000001u, oT, iT);
            b[O_RACE_SRV] = make_uint4(0u, 0x00000100u, oS, iS);
            b[O_RACE_DEV] = make_uint4(0u, 0x00010100u, oT, iT);
            b[O_MIGR_TO_DEV] = make_uint4(dly << 17 | stall_code, 0x01000100u, oS, iS);
            b[O_MIGR_TO_SRV] = make_uint4(dly << 17 | stall_code, 0x01010100u, oT, iT);
            b[6] = make_uint4(0u, EXT ? routing_draw(k0, cur.orig) : 0u, m, n);
        }
        __syncwarp();
        // kIlp requests at a time per lane, phase by phase, so that the shared-memory loads of one do not
        // queue behind the histogram atomics of another
        auto pairs_of = [&](auto tile_kind, auto all_ok, const int (&rr)[kIlp], const bool (&ok)[kIlp]) {
            constexpr int kKind = decltype(tile_kind)::value;
            constexpr bool kNoWaits = kKind == K_NOWAIT, kAllOk = decltype(all_ok)::value;
            uint4 Q[kIlp];
            bool dev_wins[kIlp], migr[kIlp];
            int oc[kIlp];
            uint32_t ttft[kIlp];
#pragma unroll
            for (int k = 0; k < kIlp; ++k) Q[k] = stA[rr[k] * kStageVec];
#pragma unroll
            for (int k = 0; k < kIlp; ++k) {
                if (kNoWaits) {
                    // ---- Algorithm 3's threshold; the race and the hand-over candidate were settled at staging
                    const bool dev_only = Q[k].x < lth16;
                    const int oc0 = (int)(Q[k].x & 15u);
                    migr[k] = !dev_only && __uint_as_float(Q[k].y) > theta;
                    dev_wins[k] = dev_only || oc0 == O_RACE_DEV;
                    ttft[k] = dev_only ? Q[k].w : Q[k].z;
                    oc[k] = dev_only ? O_DEVICE_ONLY : oc0 + (migr[k] ? 2 : 0);
                    continue;
                }
                const uint32_t l = Q[k].x, S = Q[k].y, Td = Q[k].z;
                if (kKind == K_WAIT) {
                    // ---- Algorithm 2's wait map and the race
                    const uint32_t w = (int32_t)l < l_star ? 0u : ((int32_t)l == l_star ? w_star : w_tail);
                    const bool started = S > w;                        // the device starts after the wait
                    const uint32_t wTd = w + Td;
                    dev_wins[k] = S > wTd;                             // a tie goes to the server
                    ttft[k] = min(S, wTd);
                    migr[k] = started && dev_wins[k] == dev_migrates && __uint_as_float(Q[k].w) > theta;
                    oc[k] = !started ? O_SERVER_ONLY : (dev_wins[k] ? O_RACE_DEV : O_RACE_SRV) + (migr[k] ? 2 : 0);
                    continue;
                }
                bool dev_only, started;
                if (EXT) {
                    const uint4 X = stB[rr[k] * kStageVec + 6];
                    PairIn q;
                    q.l = l; q.n = X.w; q.S = S; q.m = X.z; q.saving = __uint_as_float(Q[k].w); q.u = X.y; q.delta_c = delta_c;
                    const PairOut o = decide<true>(q, pr, Td, candidate);
                    dev_only = o.dev_only; started = o.started; dev_wins[k] = o.dev_wins; migr[k] = o.migr; ttft[k] = o.ttft;
                } else {
                    // ---- dispatch (Algorithm 2's wait map / Algorithm 3's threshold) and the race
                    dev_only = (int32_t)l < l_th;
                    const uint32_t w = (int32_t)l < l_star ? 0u : ((int32_t)l == l_star ? w_star : w_tail);
                    started = dev_only || S > w;                       // the device starts after the wait
                    const uint32_t wTd = w + Td;
                    dev_wins[k] = dev_only || (started && S > wTd);    // a tie goes to the server
                    ttft[k] = dev_only ? Td : min(S, wTd);
                    migr[k] = started && !dev_only && dev_wins[k] == dev_migrates && __uint_as_float(Q[k].w) > theta;
                }
                oc[k] = dev_only ? O_DEVICE_ONLY
                                 : (!started ? O_SERVER_ONLY : (dev_wins[k] ? O_RACE_DEV : O_RACE_SRV) + (migr[k] ? 2 : 0));
            }
            uint4 h1[kIlp], h2[kIlp];
#pragma unroll
            for (int k = 0; k < kIlp; ++k) {
                h1[k] = stA[rr[k] * kStageVec + 1 + oc[k]];
                h2[k] = stB[rr[k] * kStageVec + oc[k]];
            }
#pragma unroll
            for (int k = 0; k < kIlp; ++k) {
                if (!kAllOk && !ok[k]) continue;
                a_td += h1[k].x; a_ps += h1[k].y; a_pd += h1[k].z; a_tau += h1[k].w;
                a_dl += h2[k].x >> 17; cnt8 += h2[k].y;
                a_tt += ttft[k];
                if (EXT ? !waits : kNoWaits) atomicAdd((uint32_t*)((char*)my_ttft + h2[k].z), h2[k].w);
                else if (DBG_OK(bin_of_ticks(ttft[k]), kNBins, DBG_K_PAIRS_ACC, DBG_BIN)) hist16_add_ticks(my_ttft, ttft[k]);
            }
            // only the row of a pair whose hand-off stalled carries an increment for the stall histogram: one test
            // for the four pairs, then each
            uint32_t any_stall = 0;
#pragma unroll
            for (int k = 0; k < kIlp; ++k) any_stall |= (kAllOk || ok[k]) ? h2[k].x : 0u;
            if (any_stall & 0x10001u) {
#pragma unroll
                for (int k = 0; k < kIlp; ++k)
                    if ((kAllOk || ok[k]) && (h2[k].x & 0x10001u)) hist16_apply(my_stall, h2[k].x);
            }
            if (WIDE && act) {                                 // regular TBTs outside the bin of tau
                for (int k = 0; k < kIlp; ++k) {
                    if (!kAllOk && !ok[k]) continue;
                    const int c = migr[k] ? 2 : (dev_wins[k] ? 1 : 0);
                    const int W = c == 2 ? W2 : (c == 1 ? W1 : W0), kt = c == 2 ? kt2 : (c == 1 ? kt1 : kt0);
                    // (no bit mask with wide windows: the staged requests are the batch's first ones, in order)
                    const uint32_t* wp = rec.win[c] + (size_t)(ch.start + b0 + rr[k]) * W;
                    unsigned long long* hp = hist_tbt + (size_t)p * kNBins + cc.lo[g][c];
                    for (int j = 0; j < W; ++j) {
                        const uint32_t v = j == kt ? 0u : wp[j];
                        if (v && DBG_OK(cc.lo[g][c] + j, kNBins, DBG_K_PAIRS_ACC, DBG_BIN)) atomicAdd(&hp[j], (unsigned long long)v);
                    }
                }
            }
        };
        int r_done = 0;
        if (PL == 32) {                                         // 32 policies: the staged request is warp-uniform
#pragma unroll 2
            for (; r_done + kIlp <= n_here; r_done += kIlp) {   // whole groups of kIlp requests
                int rr[kIlp];
                bool ok[kIlp];
#pragma unroll
                for (int k = 0; k < kIlp; ++k) { rr[k] = r_done + k; ok[k] = true; }
                if (kind == K_NOWAIT) pairs_of(std::integral_constant<int, K_NOWAIT>{}, std::true_type{}, rr, ok);
                else if (kind == K_WAIT) pairs_of(std::integral_constant<int, K_WAIT>{}, std::true_type{}, rr, ok);
                else pairs_of(std::integral_constant<int, K_ANY>{}, std::true_type{}, rr, ok);
            }
        }
        for (int r0 = r_done; r0 < n_here; r0 += kIlp * slots) {
            int rr[kIlp];
            bool ok[kIlp];
#pragma unroll
            for (int k = 0; k < kIlp; ++k) {
                const int r = r0 + k * slots + slot;
                ok[k] = r < n_here;
                rr[k] = min(r, n_here - 1);                     // a slot that was staged in this batch
                if (!DBG_OK(rr[k], kStageReq, DBG_K_PAIRS_ACC, DBG_SLOT)) { rr[k] = 0; ok[k] = false; }
            }
            if (kind == K_NOWAIT) pairs_of(std::integral_constant<int, K_NOWAIT>{}, std::false_type{}, rr, ok);
            else if (kind == K_WAIT) pairs_of(std::integral_constant<int, K_WAIT>{}, std::false_type{}, rr, ok);
            else pairs_of(std::integral_constant<int, K_ANY>{}, std::false_type{}, rr, ok);
        }
        cnt_a += __byte_perm(cnt8, 0u, 0x4140); cnt_b += __byte_perm(cnt8, 0u, 0x4342); cnt8 = 0;
    };
    if (!flagged_only) {
        // ---- every request of the range: one per lane, fetched a batch ahead so that the loads fly while the
        //      previous batch is evaluated
        Raw nx = fetch(r_lo + wib * kStageReq + lane);
        for (uint32_t b0 = r_lo + wib * kStageReq; b0 < r_hi; b0 += kAccWarps * kStageReq) {
            const Raw cur = nx;
            if (b0 + kAccWarps * kStageReq < r_hi) nx = fetch(b0 + kAccWarps * kStageReq + lane);
            __syncwarp();
            run_batch(cur, __ballot_sync(0xFFFFFFFFu, b0 + lane < r_hi), b0);
        }
    } else {
        // ---- only the requests the zone kernel flagged for this tile: the warp reads the flags of 32 requests at a
        //      time and collects the flagged ones, one per lane, until it holds (nearly) a full batch
        uint32_t held = 0;                                       // chunk position of the request this lane holds
        int n_held = 0;                                          // warp-uniform
        auto work_off = [&]() {
            const Raw d = fetch(held);                           // (lanes beyond n_held fetch a valid request and drop it)
            __syncwarp();
            run_batch(d, n_held == 32 ? 0xFFFFFFFFu : (1u << n_held) - 1u, 0u);
            n_held = 0;
        };
        if (left_lists && to_do <= kLeftList) {
            // few enough to be listed by position: no scan
            const uint32_t* list = left_lists + ((size_t)chunk_id * n_tiles + tile) * kLeftList;
            for (uint32_t k0l = wib * 32u; k0l < to_do; k0l += kAccWarps * 32u) {
                n_held = (int)min(32u, to_do - k0l);
                if (lane < n_held) held = list[k0l + lane];
                work_off();
            }
        } else {
        constexpr int kScan = 4;                                 // flag words a lane has in flight
        constexpr uint32_t kStride = kAccWarps * kStageReq;
        auto flags_at = [&](uint32_t at) {
            return at < r_hi ? left_mask[(size_t)(ch.start + at) * mask_words + (tile >> 5)] & mask_bit : 0u;
        };
        for (uint32_t c0 = r_lo + wib * kStageReq; c0 < r_hi; c0 += kScan * kStride) {
            const uint32_t f0 = flags_at(c0 + lane), f1 = flags_at(c0 + kStride + lane);
            const uint32_t f2 = flags_at(c0 + 2 * kStride + lane), f3 = flags_at(c0 + 3 * kStride + lane);
            static_assert(kScan == 4, "four flag words are loaded by name");
#pragma unroll 1
            for (int j = 0; j < kScan; ++j) {                    // (not unrolled: the batch evaluation is long code)
                const uint32_t b0 = c0 + j * kStride;
                const uint32_t taken = __ballot_sync(0xFFFFFFFFu, (j == 0 ? f0 : j == 1 ? f1 : j == 2 ? f2 : f3) != 0u);
                if (taken == 0u) continue;
                const int n_new = __popc(taken);
                if (n_held + n_new > 32) work_off();
                const int want = lane - n_held;                  // lane n_held + j takes the j-th flagged request
                if (want >= 0 && want < n_new) held = b0 + __fns(taken, 0, want + 1);
                n_held += n_new;
                if (n_held >= 28) work_off();
            }
        }
        if (n_held > 0) work_off();
        }
    }
    // ---- block totals, then one flush per block.  With fewer than 32 policies in the tile several lanes of a warp
    //      hold sums of the same policy: they are added up by shuffles first, so that one lane per policy and warp
    //      touches the shared totals (with one policy, 512 threads would otherwise queue on ten addresses).
    for (int off = 16; off >= PL; off >>= 1) {
        a_td += __shfl_xor_sync(0xFFFFFFFFu, a_td, off); a_ps += __shfl_xor_sync(0xFFFFFFFFu, a_ps, off);
        a_pd += __shfl_xor_sync(0xFFFFFFFFu, a_pd, off); a_dl += __shfl_xor_sync(0xFFFFFFFFu, a_dl, off);
        a_tau += __shfl_xor_sync(0xFFFFFFFFu, a_tau, off);
        cnt_a += __shfl_xor_sync(0xFFFFFFFFu, cnt_a, off); cnt_b += __shfl_xor_sync(0xFFFFFFFFu, cnt_b, off);
        a_tt += __shfl_xor_sync(0xFFFFFFFFu, a_tt, off);
    }
    if (act && lane < PL) {
        // 32-bit adds on the low words (shared memory has no native 64-bit add): every total but the TTFT sum
        // stays below 2^32 within a block (at most 65,280 requests of at most 12,288 tokens each); the TTFT
        // sum carries into its high word
        uint32_t* a = (uint32_t*)(s_acc + pol_in_tile * kNAcc);
        atomicAdd(&a[2 * A_DEVICE_ONLY], cnt_a & 0xFFFFu); atomicAdd(&a[2 * A_RACE], cnt_a >> 16);
        atomicAdd(&a[2 * A_DEVICE_WON], cnt_b & 0xFFFFu); atomicAdd(&a[2 * A_MIGR], cnt_b >> 16);
        atomicAdd(&a[2 * A_TOK_DEVICE], a_td); atomicAdd(&a[2 * A_PRE_SERVER], a_ps);
        atomicAdd(&a[2 * A_PRE_DEVICE], a_pd); atomicAdd(&a[2 * A_DELAYED], a_dl);
        atomicAdd(&a[2 * A_TAU_CNT], a_tau);
        const uint32_t lo = (uint32_t)a_tt, before = atomicAdd(&a[2 * A_TTFT_SUM], lo);
        const uint32_t hi = (uint32_t)(a_tt >> 32) + (before + lo < before ? 1u : 0u);
        if (hi) atomicAdd(&a[2 * A_TTFT_SUM + 1], hi);
    }
    if (work && lane == 0 && staged) atomicAdd(&work[1], (unsigned long long)staged * pols_here);   // pairs evaluated one by one
    __syncthreads();
    const int bin_tau = bin_of_ticks(tau);
    for (int i = threadIdx.x; i < pols_here * kHWords; i += kAccThreads) {
        const int pi = i / kHWords, wd = i - pi * kHWords;
        const size_t o = (size_t)pol_list[tile * PL + pi] * kNBins + 2 * wd;
        const uint32_t a = h_ttft[pi * kHWords + wd], b = h_stall[pi * kHWords + wd];
        if (a & 0xFFFFu) atomicAdd(&hist_ttft[o], (unsigned long long)(a & 0xFFFFu));
        if (a >> 16) atomicAdd(&hist_ttft[o + 1], (unsigned long long)(a >> 16));
        if (b & 0xFFFFu) atomicAdd(&hist_tbt[o], (unsigned long long)(b & 0xFFFFu));
        if (b >> 16) atomicAdd(&hist_tbt[o + 1], (unsigned long long)(b >> 16));
    }
    for (int i = threadIdx.x; i < pols_here * kNAcc; i += kAccThreads) {
        const int pi = i / kNAcc, s = i - pi * kNAcc;
        const unsigned long long v = s_acc[pi * kNAcc + s];
        if (!v) continue;
        const uint32_t pp = pol_list[tile * PL + pi];
        if (s == A_TAU_CNT) atomicAdd(&hist_tbt[(size_t)pp * kNBins + bin_tau], v);   // TBTs equal to tau
        else atomicAdd(&acc[((size_t)pp * tr.n_groups + g) * kNAcc + s], v);
    }
    __syncthreads();
    }   // next pass
}

size_t acc_smem_bytes(int PL) {
    return sizeof(uint32_t) * acc_stage_offset_words(PL) + (size_t)kAccWarps * kStageReq * 2 * kStageVec * sizeof(uint4);
}

// ------------------------------------------------------------------------------------------------------
// Per-pair arrays: lane = request, up to 16 policies per block row.
//
// What a pair writes besides its TTFT depends on the request and on which of the six outcomes it ends in.
// Each thread therefore prices its request once per outcome (Eq. 8, token split, TBT mean and maximum of
// the stream that applies) into a row of shared memory that only it reads; a pair then costs the decision,
// one 16-byte row load and the nine stores.  A store instruction writes 32 consecutive requests of one
// policy row.
// ------------------------------------------------------------------------------------------------------
constexpr int kRowThreads = 256;
constexpr int kRowPols = 16;
constexpr int kRowVec = 7;              // uint4 per request: six outcome rows and one of padding (odd stride)

// What the dispatch of one (group, policy) needs, with the mode tests folded into the thresholds: Algorithm 3
// has no waits (l_star beyond every length), Algorithm 2 no device-only prompts (l_th = 0, as the preparation
// kernel leaves it), and a policy or group without migration never passes the trigger (theta = +inf).
struct __align__(8) RowPol {
    int32_t l_th, l_star;
    uint32_t w_star, w_tail;
    float theta;
    uint32_t pol;
};

__device__ __forceinline__ RowPol row_pol(const Prep& pr, int candidate, uint32_t p) {
    RowPol r;
    r.l_th = pr.l_th; r.l_star = pr.device_constrained ? pr.l_star : 0x7FFFFFFF;
    r.w_star = (uint32_t)pr.w_star; r.w_tail = (uint32_t)pr.w_tail;
    r.theta = (pr.mig_on && candidate != 0) ? pr.theta : __int_as_float(0x7F800000);
    r.pol = p;
    return r;
}

// IDX32: every element index p * N + i fits 32 bits, so a store address is one widening multiply-add.
template <bool EXT, bool IDX32>
__global__ void __launch_bounds__(kRowThreads)
k_pairs_rows(TraceDev tr, const GroupConst* __restrict__ gcs, const Prep* __restrict__ prep, uint32_t P,
             const uint32_t* __restrict__ pol_list, uint32_t n_list, TimelineRec rec, uint32_t k0,
             disco_pair_out_t out) {
    using idx_t = typename std::conditional<IDX32, uint32_t, size_t>::type;
    __shared__ Prep s_prep[EXT ? kRowPols : 1];
    __shared__ RowPol s_rp[kRowPols];
    __shared__ uint4 s_rows[kRowThreads * kRowVec];
    grid_dependency_wait();
    const uint32_t first = blockIdx.y * kRowPols;
    const int npol = (int)min((uint32_t)kRowPols, n_list - first);
    // the block's requests are consecutive in the internal order; most blocks lie inside one group
    const uint32_t k_lo = blockIdx.x * kRowThreads, k_hi = min(tr.n, k_lo + kRowThreads) - 1;
    int g_lo = 0, g_hi = 0;
    while (g_lo + 1 < tr.n_groups && k_lo >= tr.grp_off[g_lo + 1]) ++g_lo;
    g_hi = g_lo;
    while (g_hi + 1 < tr.n_groups && k_hi >= tr.grp_off[g_hi + 1]) ++g_hi;
    const bool one_group = g_lo == g_hi;
    if ((int)threadIdx.x < npol) {
        const uint32_t p = pol_list[first + threadIdx.x];
        const Prep pr = prep[(size_t)g_lo * P + p];
        if (EXT) s_prep[threadIdx.x] = pr;
        s_rp[threadIdx.x] = row_pol(pr, gcs[g_lo].candidate, p);
    }
    __syncthreads();
    uint32_t k = k_lo + threadIdx.x;
    if (k >= tr.n) return;
    // one group: a thread per request in the caller's order, so that the rows are written side by side (the reads
    // are scattered instead, once per request); several groups: the block's policies depend on the group, a thread
    // per request in the internal order
    uint32_t orig = k;
    if (tr.n_groups == 1) k = tr.inv[k]; else orig = tr.orig[k];
    if (!DBG_OK(k, tr.n, DBG_K_PAIRS_ROWS, DBG_REQUEST)) return;
    int g = g_lo;
    while (g < g_hi && k >= tr.grp_off[g + 1]) ++g;
    const GroupConst& gc = gcs[g];
    const int candidate = gc.candidate;
    const bool dev_migrates = candidate == 2;
    const float delta_c = gc.delta_c, cps = gc.cps, cds = gc.cds, lcpd = gc.lcpd, lcdd = gc.lcdd;
    const idx_t N = (idx_t)tr.n;

    PairIn q;
    q.l = tr.l[k]; q.n = tr.nout[k]; q.S = (uint32_t)tr.S[k]; q.m = rec.m[k];
    q.saving = delta_c * (float)(q.n - q.m);
    q.delta_c = delta_c;
    q.u = EXT ? routing_draw(k0, orig) : 0u;
    const uint32_t Td = (uint32_t)gc.kappa * q.l + (uint32_t)gc.c0, dly = rec.delayed[k];
    const float saving_m = q.m ? q.saving : -1.0f;        // a request migrates only if its buffer filled (m != 0)
    const uint4* row = s_rows + threadIdx.x * kRowVec;
    {
        uint4* wrow = s_rows + threadIdx.x * kRowVec;
        const float inv_cnt = q.n > 1 ? 1e-6f / (float)(q.n - 1) : 0.0f;
        float mean[3], mx[3];
#pragma unroll
        for (int c = 0; c < 3; ++c) { mean[c] = (float)rec.sum[c][k] * inv_cnt; mx[c] = (float)rec.max[c][k] * 1e-6f; }
        const uint32_t l = q.l, n = q.n, m = q.m, lm = l + m;
        auto put = [&](int oc, uint32_t pre_srv, uint32_t pre_dev, uint32_t tok_dev, int stream) {
            const uint32_t tok_srv = n - tok_dev;
            const float cost = cps * (float)pre_srv + cds * (float)tok_srv + lcpd * (float)pre_dev + lcdd * (float)tok_dev;   // Eq. 8
            wrow[oc] = make_uint4(__float_as_uint(cost), tok_srv | tok_dev << 16, __float_as_uint(mean[stream]),
                                  __float_as_uint(mx[stream]));
        };
        put(O_SERVER_ONLY, l, 0u, 0u, 0);
        put(O_DEVICE_ONLY, 0u, l, n, 1);
        put(O_RACE_SRV, l, l, 0u, 0);
        put(O_RACE_DEV, l, l, n, 1);
        put(O_MIGR_TO_DEV, l, l + lm, n - m, 2);          // the server decoded m tokens, the device re-prefills l + m
        put(O_MIGR_TO_SRV, l + lm, l, m, 2);
    }
    auto emit = [&](idx_t at, bool dev_only, bool started, bool dev_wins, bool migr, uint32_t ttft) {
        const int oc = dev_only ? O_DEVICE_ONLY
                                : (!started ? O_SERVER_ONLY : (dev_wins ? O_RACE_DEV : O_RACE_SRV) + (migr ? 2 : 0));
        const uint4 r = row[oc];
        if (out.ttft_s) out.ttft_s[at] = (float)ttft * 1e-6f;
        if (out.tbt_mean_s) out.tbt_mean_s[at] = __uint_as_float(r.z);
        if (out.tbt_max_s) out.tbt_max_s[at] = __uint_as_float(r.w);
        if (out.cost) out.cost[at] = __uint_as_float(r.x);
        if (out.tok_server) out.tok_server[at] = r.y & 0xFFFFu;
        if (out.tok_device) out.tok_device[at] = r.y >> 16;
        if (out.mig_at) out.mig_at[at] = migr ? q.m : 0u;
        if (out.delayed) out.delayed[at] = (uint16_t)(migr ? dly : 0u);
        if (out.decision) out.decision[at] = (uint8_t)(dev_only ? DISCO_DEVICE_ONLY : (started ? DISCO_RACE : DISCO_SERVER_ONLY));
    };
    auto pair = [&](const RowPol& rp, const Prep* full) {
        const idx_t at = (idx_t)rp.pol * N + (idx_t)orig;
        if (!DBG_OK(rp.pol, P, DBG_K_PAIRS_ROWS, DBG_POLICY) || !DBG_OK(orig, tr.n, DBG_K_PAIRS_ROWS, DBG_REQUEST)) return;
        if (EXT) {
            const PairOut o = decide<true>(q, *full, Td, candidate);
            emit(at, o.dev_only, o.started, o.dev_wins, o.migr, o.ttft);
            return;
        }
        // ---- dispatch (Algorithm 2's wait map / Algorithm 3's threshold) and the race
        const bool dev_only = (int32_t)q.l < rp.l_th;
        const uint32_t w = (int32_t)q.l < rp.l_star ? 0u : ((int32_t)q.l == rp.l_star ? rp.w_star : rp.w_tail);
        const bool started = dev_only || q.S > w;               // the device starts after the wait
        const uint32_t wTd = w + Td;
        const bool dev_wins = dev_only || (started && q.S > wTd);   // a tie goes to the server
        const uint32_t ttft = dev_only ? Td : min(q.S, wTd);
        const bool migr = started && !dev_only && dev_wins == dev_migrates && saving_m > rp.theta;
        emit(at, dev_only, started, dev_wins, migr, ttft);
    };
    if (one_group) {
#pragma unroll 4
        for (int pi = 0; pi < npol; ++pi) pair(s_rp[pi], EXT ? &s_prep[pi] : nullptr);
    } else {
        for (int pi = 0; pi < npol; ++pi) {
            const Prep pr = prep[(size_t)g * P + s_rp[pi].pol];
            const RowPol rp = row_pol(pr, candidate, s_rp[pi].pol);
            pair(rp, &pr);
        }
    }
}

}  // namespace

DBG_TRANSLATION_UNIT()

cudaError_t launch_pairs(const TraceDev& tr, const GroupConst* gc, const ClassConst* cc, const Prep* prep, uint32_t P,
                         const uint32_t* pol_list, uint32_t n_list, const Chunk* chunks, uint32_t n_chunks,
                         TimelineRec rec, disco_pair_out_t out, uint64_t* acc, uint64_t* hist_ttft,
                         uint64_t* hist_tbt, uint32_t* left_mask, uint32_t* left_count, uint32_t* left_lists,
                         uint32_t zone_blocks, uint32_t* zone_ticket, uint64_t* work, uint32_t k0,
                         bool extras, bool wide, cudaEvent_t mid, cudaStream_t st) {
    if (n_chunks == 0 || n_list == 0) return mid ? cudaEventRecord(mid, st) : cudaSuccess;
    int PL = 1;
    while (PL < 32 && (uint32_t)PL < n_list) PL <<= 1;
    auto* acc_kernel = extras ? (wide ? k_pairs_acc<true, true> : k_pairs_acc<true, false>)
                              : (wide ? k_pairs_acc<false, true> : k_pairs_acc<false, false>);
    cudaError_t e = cudaFuncSetAttribute(acc_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                         (int)acc_smem_bytes(32));
    if (e) return e;
    const uint32_t n_tiles = (n_list + PL - 1) / PL;
    if ((uint64_t)n_chunks * n_tiles > 0x7FFFFFFFull) return cudaErrorInvalidConfiguration;
    // zone by zone first (tiles it cannot take return at once), then pair by pair what is left
    const bool zones = !wide && left_mask != nullptr;
    if (zones) {
        const size_t mask_bytes = (size_t)tr.n * left_words_per_request(n_tiles) * 4;
        if ((e = cudaMemsetAsync(left_mask, 0, mask_bytes, st))) return e;
        if ((e = launch_pairs_zones(tr, gc, cc, prep, P, pol_list, n_list, PL, chunks, n_chunks, rec, acc, hist_ttft,
                                    hist_tbt, left_mask, left_count, left_lists, zone_blocks, zone_ticket, work, st)))
            return e;
    }
    if ((e = launch_after(acc_kernel, dim3(n_chunks * n_tiles), kAccThreads, acc_smem_bytes(PL), st, tr, gc, cc, prep, P,
                          pol_list, n_list, PL, chunks, n_tiles, rec, k0, (unsigned long long*)acc,
                          (unsigned long long*)hist_ttft, (unsigned long long*)hist_tbt,
                          (const uint32_t*)(zones ? left_mask : nullptr), (const uint32_t*)left_count,
                          (const uint32_t*)left_lists, (unsigned long long*)work)))
        return e;
    if (mid && (e = cudaEventRecord(mid, st))) return e;
    const bool rows = out.ttft_s || out.tbt_mean_s || out.tbt_max_s || out.cost || out.tok_server || out.tok_device ||
                      out.mig_at || out.delayed || out.decision;
    if (rows) {
        const bool idx32 = (uint64_t)P * tr.n <= 0xFFFFFFFFull;
        auto* row_kernel = extras ? (idx32 ? k_pairs_rows<true, true> : k_pairs_rows<true, false>)
                                  : (idx32 ? k_pairs_rows<false, true> : k_pairs_rows<false, false>);
        dim3 grid_r((tr.n + kRowThreads - 1) / kRowThreads, (n_list + kRowPols - 1) / kRowPols);
        e = launch_after(row_kernel, grid_r, kRowThreads, 0, st, tr, gc, prep, P, pol_list, n_list, rec, k0, out);
    }
    return e;
}

}  // namespace disco
