// Per-policy reductions over (request, policy) pairs, zone by zone: dispatch decision (Algorithms 2-3,
// wait-then-race), TTFT, which decode stream applies (migration trigger, Eq. 4), tokens per endpoint.
//
// Along an ascending budget axis the policies of a tile differ in thresholds that are ordered: Algorithm 3's
// l_th does not increase, Algorithm 2's l* does not decrease.  For one request the tile therefore falls into at
// most three runs of neighbouring policies that dispatch it alike:
//   Algorithm 3:  policies [0, k) have l_th > l  -> device only;   [k, npol) race at once (wait 0);
//   Algorithm 2:  policies [0, k1) have l* < l   -> wait w_tail;   [k1, k2) have l* = l -> wait their own w*;
//                 [k2, npol) have l* > l         -> wait 0.
// k, k1, k2 come from tables over the prompt lengths built once per block.  If the policies of a run also agree
// on the race and on the migration trigger, the run ends in ONE outcome, and the sums over policies become
// range updates.  A lane owns a request and
//   1. adds the outcome of the last run (wait 0) for EVERY policy of the tile, into sums and a histogram that
//      the whole tile shares;
//   2. if the request also has a first run, or policies with l* = l, queues it; the warp later takes 32 queued
//      requests at a time and enters their corrections (run outcome minus the common one) at row k1 of a
//      difference table, to be carried to the policies below k1 when the block flushes -- and, for each policy
//      with l* = l, a correction for that policy alone (plus at row p + 1, minus at row p).
// Nothing is done per pair.  What the runs cannot express -- waits that straddle the server's TTFT, a saving
// between the tile's smallest and largest migration overhead -- is flagged in a bit mask and left to the
// pair-by-pair kernel (pairs.cu).
#include <cstddef>

#include "tile.cuh"

namespace disco {

namespace {

constexpr int kZThreads = 1024;
static_assert(kZThreads == 1024, "the flush assigns its work to threads 0 .. 1023 by index");
constexpr int kZWarps = kZThreads / 32;
constexpr int kZRows = 33;              // difference rows: row q is carried to the policies below q, q = 1 .. 32
// Requests a block may queue for corrections between two flushes.  A signed 16-bit count of the difference rows
// moves by at most one per queued request under Algorithm 3 (one boundary) and by at most two under Algorithm 2 (a
// boundary and a policy of its own at the same row).
constexpr uint32_t kZItems = 32640, kZItemsWaits = 16320;
constexpr uint32_t kZStretch = 8160;     // requests between two looks at that budget
constexpr int kZQueue = 64;             // queue slots per warp
enum ZSum { Z_TD = 0, Z_PS, Z_PD, Z_TAU, Z_DL, Z_CNT_A, Z_CNT_B, Z_TT_LO, Z_TT_HI, kZSums };
constexpr int kZSumStride = 12;
constexpr int kLenTab = kMaxPrompt + 8; // bytes per table over the prompt lengths 0 .. 4096

struct ZoneSmem {
    uint32_t e_ttft[kZRows][kHWords];   // difference rows of the TTFT histogram: two signed 16-bit counts a word
    uint32_t e_stall[kZRows][kHWords];  // ... of the histogram of hand-off stalls
    uint32_t c_ttft[2 * kHWords];       // what every policy of the tile gets: 32-bit counts
    uint32_t c_stall[2 * kHWords];
    uint32_t e_sum[kZRows][kZSumStride];   // difference rows of the sums (wrap-around 32-bit words)
    unsigned long long c_sum[kZSums];
    uint32_t n_left, n_items;
    // ---- not cleared between flushes
    uint32_t n_listed;                  // requests left to the pair kernel so far (their list positions)
    uint32_t queue[kZWarps][kZQueue];   // requests (chunk-relative) that await their corrections
    int32_t key[32];                    // the policies' length thresholds, in tile order
    uint32_t w_star[32];                // Algorithm 2: the wait of the length class l*
    uint32_t w_tail[32];                // ... and of the longer prompts
    float theta[32];                    // Eq. 4's overhead (+inf: the policy never hands over)
    uint32_t pol[32];                   // the policies' indices in the caller's list
    uint8_t tab1[kLenTab], tab2[kLenTab];
};

// What one request adds to the sums of a policy under which it ends in outcome oc.
struct Addends { uint32_t td, ps, pd, tau, dl, cnt; };

struct Req { uint32_t l, n, S, m, dly, stall, nt0, nt1, nt2; };

__device__ __forceinline__ Addends addends_of(int oc, const Req& r) {
    const bool migr = oc >= O_MIGR_TO_DEV, dev_wins = (oc & 1) != 0;
    const uint32_t lm = r.l + r.m;
    Addends a;
    a.td = migr ? (dev_wins ? r.m : r.n - r.m) : (dev_wins ? r.n : 0u);         // tokens the device generated
    a.ps = oc == O_DEVICE_ONLY ? 0u : r.l + ((migr && dev_wins) ? lm : 0u);     // prompt tokens billed by the server
    a.pd = oc == O_SERVER_ONLY ? 0u : r.l + ((migr && !dev_wins) ? lm : 0u);    // ... by the device
    a.tau = migr ? r.nt2 : (dev_wins ? r.nt1 : r.nt0);                          // TBTs in the bin of tau
    a.dl = migr ? r.dly : 0u;
    // a byte each: device only, race, device won, migrated
    a.cnt = oc == O_DEVICE_ONLY ? 0x00000001u
          : oc == O_RACE_SRV ? 0x00000100u : oc == O_RACE_DEV ? 0x00010100u
          : oc == O_MIGR_TO_DEV ? 0x01000100u : oc == O_MIGR_TO_SRV ? 0x01010100u : 0u;
    return a;
}

// A byte-packed count word as two words of two 16-bit counts: (device only | race << 16), (device won | migrated << 16).
__device__ __forceinline__ uint32_t cnt_pair_a(uint32_t c) { return (c & 0xFFu) | ((c & 0xFF00u) << 8); }
__device__ __forceinline__ uint32_t cnt_pair_b(uint32_t c) { return ((c >> 16) & 0xFFu) | ((c >> 24) << 16); }

// Everything a lane needs to evaluate requests of one (chunk, tile).
struct TileCtx {
    const TraceDev* tr; const TimelineRec* rec; const Chunk* ch;
    uint32_t tau, kappa, c0, E0, wt_min, wt_max;
    float delta_c, th_min, th_max;
    int npol, race_that_migrates, W0, W1, W2, kt0, kt1, kt2;
    bool may_migrate;
    bool wt_ordered;                    // the policies' w_tail do not increase along the tile
};

template <bool LEAN>
__device__ __forceinline__ Req load_request(const TileCtx& c, uint32_t i) {
    const uint32_t kk = c.ch->start + min(i, c.ch->len - 1);
    Req q;
    q.l = c.tr->l[kk]; q.n = c.tr->nout[kk]; q.S = (uint32_t)c.tr->S[kk];
    q.m = 0; q.dly = 0; q.stall = c.tau;
    if (c.may_migrate) { q.m = c.rec->m[kk]; q.dly = c.rec->delayed[kk]; q.stall = c.rec->stall[kk]; }
    q.nt0 = q.nt1 = q.nt2 = 0;
    if (!LEAN) {
        q.nt0 = c.kt0 >= 0 ? c.rec->win[0][(size_t)kk * c.W0 + c.kt0] : 0u;
        q.nt1 = c.kt1 >= 0 ? c.rec->win[1][(size_t)kk * c.W1 + c.kt1] : 0u;
        q.nt2 = c.kt2 >= 0 ? c.rec->win[2][(size_t)kk * c.W2 + c.kt2] : 0u;
    }
    return q;
}

// With every stream delivered at the pace tau the TBTs in tau's bin are all n - 1 intervals (n - 2 beside a
// hand-off); a hand-off stall of exactly tau counts with them, any other gets a histogram increment of its own.
template <bool LEAN>
__device__ __forceinline__ uint32_t finish_request(const TileCtx& c, Req& q) {
    if (LEAN) { const uint32_t nI = q.n - 1; q.nt0 = nI; q.nt1 = nI; q.nt2 = nI ? nI - 1 : 0u; }
    if (q.stall == c.tau) { ++q.nt2; return 0u; }
    return hist16_code(bin_of_ticks(q.stall));
}

// Eq. 4's projected saving, on the true remainder or on what is left of the expected length; a request may only
// hand over if its buffer filled (m != 0).
__device__ __forceinline__ float saving_of(const TileCtx& c, const Req& q) {
    if (!c.may_migrate || q.m == 0) return -1.0f;
    return c.delta_c * (float)(c.E0 ? (uint32_t)max((int32_t)c.E0 - (int32_t)q.m, 0) : q.n - q.m);
}

// The migration trigger over the whole tile for a race outcome: 0 no policy hands over, 1 every policy does,
// -1 they differ.
__device__ __forceinline__ int trigger_all(const TileCtx& c, int base, float saving) {
    if (base != c.race_that_migrates || !(saving > c.th_min)) return 0;
    return saving > c.th_max ? 1 : -1;
}

// The run of policies that wait 0: the race is the request's own.  Returns false if the policies disagree.
__device__ __forceinline__ bool tail_outcome(const TileCtx& c, const Req& q, uint32_t Td, float saving, int& oc, uint32_t& tt) {
    const int base = q.S > 0u ? (q.S > Td ? O_RACE_DEV : O_RACE_SRV) : O_SERVER_ONLY;
    tt = min(q.S, Td);
    const int t = trigger_all(c, base, saving);
    oc = base + 2 * t;
    return t >= 0;
}

// The run of Algorithm 2 policies [0, k1) that wait their w_tail.  On success the policies [j, k1) end in
// (oc, tt) and the policies [0, j), whose longer waits cover the server's TTFT, in O_SERVER_ONLY with the same
// TTFT (j = 0: none).  Returns false if the run cannot be expressed that way.
__device__ __forceinline__ bool head_outcome_waits(const TileCtx& c, const ZoneSmem& sm, const Req& q, uint32_t Td,
                                                   float saving, int k1, int& oc, uint32_t& tt, int& j) {
    int base;
    tt = q.S;
    j = 0;
    if (q.S <= c.wt_min) base = O_SERVER_ONLY;                                 // the server answers within every wait
    else if (q.S <= c.wt_min + Td) {                                           // whoever starts the device loses the race
        base = O_RACE_SRV;
        if (q.S <= c.wt_max) {                                                 // some waits cover S: those policies first
            if (!c.wt_ordered) return false;
            int lo = 0, hi = k1;
            while (lo < hi) { const int mid = (lo + hi) >> 1; if (sm.w_tail[mid] >= q.S) lo = mid + 1; else hi = mid; }
            j = lo;
            if (j == k1) { base = O_SERVER_ONLY; j = 0; }                      // every wait of the run covers S
        }
    } else if (c.wt_min == c.wt_max) { base = O_RACE_DEV; tt = c.wt_min + Td; }   // the device wins under every policy
    else return false;
    const int t = trigger_all(c, base, saving);
    oc = base + 2 * t;
    return t >= 0;
}

// Enters (outcome oc, TTFT tt) minus (outcome oc_b, TTFT tt_b) of request q at difference row `row`, times sign.
__device__ __forceinline__ void enter_difference(ZoneSmem& sm, int row, uint32_t sign, const Req& q, uint32_t stall_code,
                                                 int oc, uint32_t tt, int oc_b, uint32_t tt_b) {
    if (!DBG_OK(row, kZRows, DBG_K_PAIRS_ZONES, DBG_SLOT)) return;
    const Addends h = addends_of(oc, q), a = addends_of(oc_b, q);
    uint32_t* r = sm.e_sum[row];
    atomicAdd(&r[Z_TD], sign * (h.td - a.td));
    atomicAdd(&r[Z_PS], sign * (h.ps - a.ps));
    atomicAdd(&r[Z_PD], sign * (h.pd - a.pd));
    atomicAdd(&r[Z_TAU], sign * (h.tau - a.tau));
    atomicAdd(&r[Z_DL], sign * (h.dl - a.dl));
    atomicAdd(&r[Z_CNT_A], sign * (cnt_pair_a(h.cnt) - cnt_pair_a(a.cnt)));
    atomicAdd(&r[Z_CNT_B], sign * (cnt_pair_b(h.cnt) - cnt_pair_b(a.cnt)));
    if (tt != tt_b) {
        atomicAdd(&r[Z_TT_LO], sign * ((tt & 0xFFFFu) - (tt_b & 0xFFFFu)));
        atomicAdd(&r[Z_TT_HI], sign * ((tt >> 16) - (tt_b >> 16)));
        const uint32_t up = hist16_code(bin_of_ticks(tt)), down = hist16_code(bin_of_ticks(tt_b));
        if (sign == 1u) { hist16_apply(sm.e_ttft[row], up); hist16_retract(sm.e_ttft[row], down); }
        else { hist16_retract(sm.e_ttft[row], up); hist16_apply(sm.e_ttft[row], down); }
    }
    const bool st = oc >= O_MIGR_TO_DEV && stall_code != 0u, st_b = oc_b >= O_MIGR_TO_DEV && stall_code != 0u;
    if (st != st_b) {
        if (st == (sign == 1u)) hist16_apply(sm.e_stall[row], stall_code); else hist16_retract(sm.e_stall[row], stall_code);
    }
}

// The corrections of up to 32 queued requests, one per lane.
template <bool WAITS, bool LEAN>
__device__ __forceinline__ void drain_queue(ZoneSmem& sm, const TileCtx& c, const uint32_t* queue, int count) {
    const int lane = threadIdx.x & 31;
    if (lane < count && DBG_OK(lane, kZQueue, DBG_K_PAIRS_ZONES, DBG_SLOT)) {
        Req q = load_request<LEAN>(c, queue[lane]);
        if (!DBG_OK(q.l, kMaxPrompt + 1, DBG_K_PAIRS_ZONES, DBG_TABLE)) q.l = 0;
        const uint32_t stall_code = finish_request<LEAN>(c, q);
        const uint32_t Td = c.kappa * q.l + c.c0;
        const float saving = saving_of(c, q);
        const int k1 = sm.tab1[q.l], k2 = WAITS ? sm.tab2[q.l] : k1;
        int oc_b, oc_h = O_DEVICE_ONLY, j = 0;
        uint32_t tt_b, tt_h = Td;
        tail_outcome(c, q, Td, saving, oc_b, tt_b);              // (every run was settled when the request was queued)
        if (WAITS && k1 > 0) head_outcome_waits(c, sm, q, Td, saving, k1, oc_h, tt_h, j);
        if (k2 >= c.npol) { oc_b = oc_h; tt_b = tt_h; }          // every policy is in the first run: it is the common part
        else if (k1 > 0) enter_difference(sm, k1, 1u, q, stall_code, oc_h, tt_h, oc_b, tt_b);
        if (j > 0) enter_difference(sm, j, 1u, q, stall_code, O_SERVER_ONLY, q.S, oc_h, tt_h);
        if (WAITS && k2 < c.npol) {
            for (int p = k1; p < k2; ++p) {                      // policies whose l* is this length: their own wait
                const uint32_t w = sm.w_star[p];
                int oc = O_SERVER_ONLY;
                uint32_t tt = q.S;
                if (q.S > w) {                                   // the device starts after the wait
                    tt = min(q.S, w + Td);
                    oc = q.S > w + Td ? O_RACE_DEV : O_RACE_SRV; // a tie goes to the server
                    if (oc == c.race_that_migrates && saving > sm.theta[p]) oc += 2;
                }
                // for policy p alone: plus at the row above it, minus at its own row
                enter_difference(sm, p + 1, 1u, q, stall_code, oc, tt, oc_b, tt_b);
                enter_difference(sm, p, 0u - 1u, q, stall_code, oc, tt, oc_b, tt_b);
            }
        }
    }
    __syncwarp();
}

// Where a block's results go.
struct FlushTo {
    unsigned long long *acc, *hist_ttft, *hist_tbt;
    int n_groups, g, bin_tau;
};

// Adds what the block holds to the policies' global sums and histograms.  All threads call; the shared tables must
// be complete (barrier before) and may be cleared after the next barrier.
__device__ __forceinline__ void flush_tile(ZoneSmem& sm, int npol, const FlushTo& to) {
    unsigned long long* acc = to.acc; unsigned long long* hist_ttft = to.hist_ttft; unsigned long long* hist_tbt = to.hist_tbt;
    const int g = to.g, bin_tau = to.bin_tau;
    // policy p gets the common part plus the difference rows above it (rows q > p); two threads a histogram word:
    // one for the upper half of the policies, one for the lower half
    if ((threadIdx.x & 511) < kHWords) {
        const int wd = threadIdx.x & 511;
        const int half = npol > 16 ? 16 : 0;                                        // policies [half, npol) | [0, half)
        const bool upper = threadIdx.x < 512;
        int32_t t0 = (int32_t)sm.c_ttft[2 * wd], t1 = (int32_t)sm.c_ttft[2 * wd + 1];
        int32_t s0 = (int32_t)sm.c_stall[2 * wd], s1 = (int32_t)sm.c_stall[2 * wd + 1];
        for (int p = npol - 1; p >= (upper ? half : 0); --p) {
            const uint32_t et = sm.e_ttft[p + 1][wd], es = sm.e_stall[p + 1][wd];   // row p + 1: for policies up to p
            t0 += packed_lo(et); t1 += packed_hi(et); s0 += packed_lo(es); s1 += packed_hi(es);
            if (!upper && p >= half) continue;                                      // (the other thread's policies)
            const size_t o = (size_t)sm.pol[p] * kNBins + 2 * wd;
            if (t0) atomicAdd(&hist_ttft[o], (unsigned long long)t0);
            if (t1) atomicAdd(&hist_ttft[o + 1], (unsigned long long)t1);
            if (s0) atomicAdd(&hist_tbt[o], (unsigned long long)s0);
            if (s1) atomicAdd(&hist_tbt[o + 1], (unsigned long long)s1);
        }
    }
    if (threadIdx.x >= 512 && threadIdx.x < 512 + 32 * kZSums) {                 // a thread per (field, policy)
        const int f = (threadIdx.x - 512) >> 5, p = threadIdx.x & 31;
        const bool is_packed = f == Z_CNT_A || f == Z_CNT_B;                    // two counts in the word
        long long lo = is_packed ? (long long)(sm.c_sum[f] & 0xFFFFFFFFull) : (long long)sm.c_sum[f];
        long long hi = is_packed ? (long long)(sm.c_sum[f] >> 32) : 0;
        for (int q = p + 1; q <= npol; ++q) {                                   // the rows above the policy
            const uint32_t e = sm.e_sum[q][f];
            if (is_packed) { lo += packed_lo(e); hi += packed_hi(e); } else lo += (int32_t)e;
        }
        if (p < npol) {
            const uint32_t pp = sm.pol[p];
            unsigned long long* a = acc + ((size_t)pp * to.n_groups + g) * kNAcc;
            // (the two halves of the TTFT sum may be negative on their own: the 64-bit adds wrap to the right total)
            switch (f) {
                case Z_TD: if (lo) atomicAdd(&a[A_TOK_DEVICE], (unsigned long long)lo); break;
                case Z_PS: if (lo) atomicAdd(&a[A_PRE_SERVER], (unsigned long long)lo); break;
                case Z_PD: if (lo) atomicAdd(&a[A_PRE_DEVICE], (unsigned long long)lo); break;
                case Z_TAU: if (lo) atomicAdd(&hist_tbt[(size_t)pp * kNBins + bin_tau], (unsigned long long)lo); break;
                case Z_DL: if (lo) atomicAdd(&a[A_DELAYED], (unsigned long long)lo); break;
                case Z_CNT_A: if (lo) atomicAdd(&a[A_DEVICE_ONLY], (unsigned long long)lo);
                              if (hi) atomicAdd(&a[A_RACE], (unsigned long long)hi); break;
                case Z_CNT_B: if (lo) atomicAdd(&a[A_DEVICE_WON], (unsigned long long)lo);
                              if (hi) atomicAdd(&a[A_MIGR], (unsigned long long)hi); break;
                case Z_TT_LO: if (lo) atomicAdd(&a[A_TTFT_SUM], (unsigned long long)lo); break;
                default: if (lo) atomicAdd(&a[A_TTFT_SUM], (unsigned long long)lo << 16); break;   // Z_TT_HI
            }
        }
    }
}

// WAITS: the tile's policies are Algorithm 2's (wait map); otherwise Algorithm 3's (length threshold).
// LEAN: pacing is on and each stream's regular intervals fall in one histogram bin (tau's).
//
// The chunk is worked through in stretches of kZStretch requests.  The shared tables are flushed (and cleared) when
// the requests queued for corrections since the last flush, plus a stretch that could all be queued, would no longer
// fit the signed 16-bit counts of the difference rows -- and at the end of the chunk.
template <bool WAITS, bool LEAN>
__device__ __forceinline__ void zone_chunk(ZoneSmem& sm, const TileCtx& c, uint32_t tile, uint32_t n_tiles,
                                           uint32_t* __restrict__ left_mask, uint32_t* __restrict__ left_list,
                                           const FlushTo& out, uint32_t& left_total, uint32_t& items_total) {
    const int lane = threadIdx.x & 31, wib = threadIdx.x >> 5;
    const int npol = c.npol;
    uint32_t* queue = sm.queue[wib];
    int queued = 0;                                              // warp-uniform, below 32 between iterations
    // what every policy of the tile gets from this lane's requests since the last flush (a lane sees at most 128 of
    // a chunk's requests: its byte counts cannot overflow)
    uint32_t c_td = 0, c_ps = 0, c_pd = 0, c_tau = 0, c_dl = 0, c_cnt = 0;
    unsigned long long c_tt = 0;
    uint32_t n_left = 0, n_queued = 0;
    const uint32_t words = left_words_per_request(n_tiles);
    const uint32_t left_bit = 1u << (tile & 31u);
    const uint32_t budget = WAITS ? kZItemsWaits : kZItems;
    const uint32_t len = c.ch->len;

    for (int i = threadIdx.x; i < (int)(offsetof(ZoneSmem, queue) / 4); i += kZThreads) ((uint32_t*)&sm)[i] = 0;
    __syncthreads();
    for (uint32_t r_lo = 0; r_lo < len; r_lo += kZStretch) {
    const uint32_t r_hi = min(len, r_lo + kZStretch);
    Req nx = load_request<LEAN>(c, r_lo + threadIdx.x);
    for (uint32_t i0 = r_lo + wib * 32u; i0 < r_hi; i0 += kZThreads) {      // a warp's lanes iterate together
        const uint32_t i = i0 + lane;
        Req q = nx;
        if (i0 + kZThreads < r_hi) nx = load_request<LEAN>(c, i + kZThreads);
        bool valid = i < r_hi;
        if (!DBG_OK(q.l, kMaxPrompt + 1, DBG_K_PAIRS_ZONES, DBG_TABLE)) { q.l = 0; valid = false; }
        const uint32_t Td = c.kappa * q.l + c.c0;
        const int k1 = sm.tab1[q.l], k2 = WAITS ? sm.tab2[q.l] : k1;
        const float saving = saving_of(c, q);
        // ---- can the runs express the request?  oc_all: what every policy gets; later: corrections to queue
        int oc_all = O_DEVICE_ONLY;
        uint32_t tt_all = Td;
        bool ok = true, later = false;
        if (k2 < npol) {
            ok = tail_outcome(c, q, Td, saving, oc_all, tt_all);
            later = k2 > 0;                                      // a first run, or policies with l* = l
            if (WAITS && k1 > 0) { int oc, j; uint32_t tt; ok = head_outcome_waits(c, sm, q, Td, saving, k1, oc, tt, j) && ok; }
        } else if (k1 < npol) {
            ok = false;                                          // l* = l for the last policies and nobody waits 0
        } else if (WAITS) {
            int j;                                               // every policy waits its w_tail
            ok = head_outcome_waits(c, sm, q, Td, saving, k1, oc_all, tt_all, j);
            later = j > 0;
        }
        ok = ok && valid;
        if (valid && !ok) {
            atomicOr(&left_mask[(size_t)(c.ch->start + i) * words + (tile >> 5)], left_bit);
            ++n_left;
            if (left_list) { const uint32_t at = atomicAdd(&sm.n_listed, 1u); if (at < kLeftList) left_list[at] = i; }
        }
        // ---- every policy of the tile gets the outcome of the last run
        if (ok) {
            const uint32_t stall_code = finish_request<LEAN>(c, q);
            const Addends a = addends_of(oc_all, q);
            c_td += a.td; c_ps += a.ps; c_pd += a.pd; c_tau += a.tau; c_dl += a.dl; c_cnt += a.cnt; c_tt += tt_all;
            if (DBG_OK(bin_of_ticks(tt_all), kNBins, DBG_K_PAIRS_ZONES, DBG_BIN)) atomicAdd(&sm.c_ttft[bin_of_ticks(tt_all)], 1u);
            if (oc_all >= O_MIGR_TO_DEV && stall_code != 0u) atomicAdd(&sm.c_stall[bin_of_ticks(q.stall)], 1u);
        }
        // ---- queue the requests that need corrections; a full warp of them is worked off at once
        const uint32_t enq = __ballot_sync(0xFFFFFFFFu, ok && later);
        if (enq) {
            if (ok && later && DBG_OK(queued + __popc(enq & ((1u << lane) - 1u)), kZQueue, DBG_K_PAIRS_ZONES, DBG_SLOT))
                queue[queued + __popc(enq & ((1u << lane) - 1u))] = i;
            queued += __popc(enq);
            n_queued += (uint32_t)__popc(enq);
            __syncwarp();
            if (queued >= 32) {
                drain_queue<WAITS, LEAN>(sm, c, queue, 32);
                queued -= 32;
                const uint32_t moved = lane < queued ? queue[lane + 32] : 0u;
                __syncwarp();
                if (lane < queued) queue[lane] = moved;
                __syncwarp();
            }
        }
    }
    // ---- end of a stretch: flush now, or go on with the tables as they are?
    if (lane == 0 && n_queued) { atomicAdd(&sm.n_items, n_queued); }
    n_queued = 0;
    __syncthreads();
    const bool flush_now = r_hi == len || sm.n_items + kZStretch > budget;      // block-uniform
    if (flush_now) {
        if (queued > 0) { drain_queue<WAITS, LEAN>(sm, c, queue, queued); queued = 0; }
        // block totals of what every policy gets
        uint32_t c_ca = cnt_pair_a(c_cnt), c_cb = cnt_pair_b(c_cnt);   // a lane's byte counts stay below 256
#pragma unroll
        for (int off = 16; off > 0; off >>= 1) {
            c_td += __shfl_xor_sync(0xFFFFFFFFu, c_td, off); c_ps += __shfl_xor_sync(0xFFFFFFFFu, c_ps, off);
            c_pd += __shfl_xor_sync(0xFFFFFFFFu, c_pd, off); c_tau += __shfl_xor_sync(0xFFFFFFFFu, c_tau, off);
            c_dl += __shfl_xor_sync(0xFFFFFFFFu, c_dl, off); c_ca += __shfl_xor_sync(0xFFFFFFFFu, c_ca, off);
            c_cb += __shfl_xor_sync(0xFFFFFFFFu, c_cb, off); c_tt += __shfl_xor_sync(0xFFFFFFFFu, c_tt, off);
            n_left += __shfl_xor_sync(0xFFFFFFFFu, n_left, off);
        }
        if (lane == 0) {
            // a warp adds once per flush: the 64-bit adds (compare-and-swap loops in shared memory) do not queue up
            atomicAdd(&sm.c_sum[Z_TD], (unsigned long long)c_td); atomicAdd(&sm.c_sum[Z_PS], (unsigned long long)c_ps);
            atomicAdd(&sm.c_sum[Z_PD], (unsigned long long)c_pd); atomicAdd(&sm.c_sum[Z_TAU], (unsigned long long)c_tau);
            atomicAdd(&sm.c_sum[Z_DL], (unsigned long long)c_dl);
            atomicAdd(&sm.c_sum[Z_CNT_A], (unsigned long long)(c_ca & 0xFFFFu) | ((unsigned long long)(c_ca >> 16) << 32));
            atomicAdd(&sm.c_sum[Z_CNT_B], (unsigned long long)(c_cb & 0xFFFFu) | ((unsigned long long)(c_cb >> 16) << 32));
            atomicAdd(&sm.c_sum[Z_TT_LO], c_tt);
            atomicAdd(&sm.n_left, n_left);
        }
        c_td = c_ps = c_pd = c_tau = c_dl = c_cnt = 0; c_tt = 0; n_left = 0;
        __syncthreads();
        left_total += sm.n_left;
        items_total += sm.n_items;
        flush_tile(sm, npol, out);
        __syncthreads();
        for (int i = threadIdx.x; i < (int)(offsetof(ZoneSmem, queue) / 4); i += kZThreads) ((uint32_t*)&sm)[i] = 0;
        __syncthreads();
    }
    }   // next stretch
}

__global__ void __launch_bounds__(kZThreads, 1)
k_pairs_zones(TraceDev tr, const GroupConst* __restrict__ gcs, const ClassConst* __restrict__ ccp,
              const Prep* __restrict__ prep, uint32_t P, const uint32_t* __restrict__ pol_list, uint32_t n_list,
              int PL, const Chunk* __restrict__ chunks, uint32_t n_tiles, TimelineRec rec,
              unsigned long long* __restrict__ acc, unsigned long long* __restrict__ hist_ttft,
              unsigned long long* __restrict__ hist_tbt, uint32_t* __restrict__ left_mask,
              uint32_t* __restrict__ left_count, uint32_t* __restrict__ left_lists,
              unsigned long long* __restrict__ work) {
    extern __shared__ __align__(16) unsigned char zsmem_raw[];
    ZoneSmem& sm = *reinterpret_cast<ZoneSmem*>(zsmem_raw);
    grid_dependency_wait();
    const uint32_t tile = blockIdx.x % n_tiles, chunk_id = blockIdx.x / n_tiles;
    const Chunk ch = chunks[chunk_id];
    const int g = ch.g;
    const int lane = threadIdx.x & 31, wib = threadIdx.x >> 5;
    const int npol = (int)min((uint32_t)PL, n_list - tile * PL);

    // ---- the tile's policies, one per lane
    const uint32_t pol_idx = tile * PL + lane % PL;
    const bool act = pol_idx < n_list;
    const Prep pr = prep[(size_t)g * P + pol_list[act ? pol_idx : 0]];
    if (!tile_by_zones(pr, act, lane, npol)) return;              // block-uniform: the pair kernel takes the tile
    if (!DBG_OK(g, tr.n_groups, DBG_K_PAIRS_ZONES, DBG_GROUP) ||
        (ch.len && !DBG_OK((unsigned long long)ch.start + ch.len - 1, tr.n, DBG_K_PAIRS_ZONES, DBG_REQUEST)))
        return;
    const GroupConst& gc = gcs[g];
    const ClassConst& cc = *ccp;
    const bool waits = pr.device_constrained != 0;                // Algorithm 2 (true) or Algorithm 3 (every lane alike)
    const float theta = (pr.mig_on && gc.candidate != 0) ? pr.theta : __int_as_float(0x7F800000);
    TileCtx c;
    c.tr = &tr; c.rec = &rec; c.ch = &ch;
    c.tau = (uint32_t)cc.tau; c.kappa = (uint32_t)gc.kappa; c.c0 = (uint32_t)gc.c0;
    c.E0 = pr.expected_len;                                       // the same for every policy of the tile
    c.delta_c = gc.delta_c;
    c.npol = npol; c.race_that_migrates = gc.candidate == 2 ? O_RACE_DEV : O_RACE_SRV;
    c.W0 = cc.W[0]; c.W1 = cc.W[1]; c.W2 = cc.W[2];
    c.kt0 = cc.ktau[g][0]; c.kt1 = cc.ktau[g][1]; c.kt2 = cc.ktau[g][2];
    // thresholds are non-negative floats or +inf: their bit patterns order like the values
    c.th_min = __uint_as_float(__reduce_min_sync(0xFFFFFFFFu, act ? __float_as_uint(theta) : 0x7F800000u));
    c.th_max = __uint_as_float(__reduce_max_sync(0xFFFFFFFFu, act ? __float_as_uint(theta) : 0u));
    c.wt_min = __reduce_min_sync(0xFFFFFFFFu, act ? (uint32_t)pr.w_tail : 0xFFFFFFFFu);
    c.wt_max = __reduce_max_sync(0xFFFFFFFFu, act ? (uint32_t)pr.w_tail : 0u);
    c.may_migrate = c.th_min != __int_as_float(0x7F800000);      // some policy of the tile can hand over
    {
        const uint32_t next = __shfl_down_sync(0xFFFFFFFFu, (uint32_t)pr.w_tail, 1);
        c.wt_ordered = __all_sync(0xFFFFFFFFu, lane + 1 >= npol || (uint32_t)pr.w_tail >= next) != 0;
    }

    if (threadIdx.x == 0) sm.n_listed = 0;
    uint32_t* left_list = left_lists ? left_lists + ((size_t)chunk_id * n_tiles + tile) * kLeftList : nullptr;
    if (wib == 0 && lane < npol) {
        sm.key[lane] = waits ? pr.l_star : pr.l_th;
        sm.w_star[lane] = (uint32_t)pr.w_star;
        sm.w_tail[lane] = (uint32_t)pr.w_tail;
        sm.theta[lane] = theta;
        sm.pol[lane] = DBG_OK(pol_list[pol_idx], P, DBG_K_PAIRS_ZONES, DBG_POLICY) ? pol_list[pol_idx] : 0u;
    }
    __syncthreads();
    // tables over the prompt length: how many of the tile's (ordered) thresholds lie on which side of it
    for (int l = threadIdx.x; l <= kMaxPrompt; l += kZThreads) {
        int lo = 0, hi = npol;                                    // first position whose threshold fails the test
        if (waits) {
            while (lo < hi) { const int mid = (lo + hi) >> 1; if (sm.key[mid] < l) lo = mid + 1; else hi = mid; }
            const int k1 = lo;                                    // thresholds below l (ascending order)
            hi = npol;
            while (lo < hi) { const int mid = (lo + hi) >> 1; if (sm.key[mid] <= l) lo = mid + 1; else hi = mid; }
            sm.tab1[l] = (uint8_t)k1; sm.tab2[l] = (uint8_t)lo;   // k1, k2
        } else {
            while (lo < hi) { const int mid = (lo + hi) >> 1; if (sm.key[mid] > l) lo = mid + 1; else hi = mid; }
            sm.tab1[l] = (uint8_t)lo; sm.tab2[l] = (uint8_t)lo;   // thresholds above l (descending order)
        }
    }
    // with pacing on and one histogram bin per stream, every regular interval of a stream lies in that bin (tau's)
    const bool lean = cc.pacing != 0 && cc.W[0] == 1 && cc.W[1] == 1 && cc.W[2] == 1;
    uint32_t left_total = 0, items_total = 0;

    FlushTo out;
    out.acc = acc; out.hist_ttft = hist_ttft; out.hist_tbt = hist_tbt; out.n_groups = tr.n_groups; out.g = g;
    out.bin_tau = bin_of_ticks(c.tau);
    if (waits) {
        if (lean) zone_chunk<true, true>(sm, c, tile, n_tiles, left_mask, left_list, out, left_total, items_total);
        else zone_chunk<true, false>(sm, c, tile, n_tiles, left_mask, left_list, out, left_total, items_total);
    } else {
        if (lean) zone_chunk<false, true>(sm, c, tile, n_tiles, left_mask, left_list, out, left_total, items_total);
        else zone_chunk<false, false>(sm, c, tile, n_tiles, left_mask, left_list, out, left_total, items_total);
    }
    if (threadIdx.x == 0) {
        left_count[(size_t)chunk_id * n_tiles + tile] = left_total;
        if (work) {
            atomicAdd(&work[0], (unsigned long long)(ch.len - left_total) * npol);   // pairs settled zone by zone
            atomicAdd(&work[2], (unsigned long long)(ch.len - left_total));          // requests settled, per tile
            atomicAdd(&work[3], (unsigned long long)items_total);                    // ... of which with corrections
        }
    }
}

}  // namespace

DBG_TRANSLATION_UNIT()

cudaError_t launch_pairs_zones(const TraceDev& tr, const GroupConst* gc, const ClassConst* cc, const Prep* prep,
                               uint32_t P, const uint32_t* pol_list, uint32_t n_list, int PL, const Chunk* chunks,
                               uint32_t n_chunks, TimelineRec rec, uint64_t* acc, uint64_t* hist_ttft,
                               uint64_t* hist_tbt, uint32_t* left_mask, uint32_t* left_count, uint32_t* left_lists,
                               uint64_t* work, cudaStream_t st) {
    const uint32_t n_tiles = (n_list + PL - 1) / PL;
    if ((uint64_t)n_chunks * n_tiles > 0x7FFFFFFFull) return cudaErrorInvalidConfiguration;
    cudaError_t e = cudaFuncSetAttribute(k_pairs_zones, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)sizeof(ZoneSmem));
    if (e) return e;
    return launch_after(k_pairs_zones, dim3(n_chunks * n_tiles), kZThreads, sizeof(ZoneSmem), st, tr, gc, cc, prep, P,
                        pol_list, n_list, PL, chunks, n_tiles, rec, (unsigned long long*)acc,
                        (unsigned long long*)hist_ttft, (unsigned long long*)hist_tbt, left_mask, left_count, left_lists,
                        (unsigned long long*)work);
}

}  // namespace disco
