// Per-policy reductions over (request, policy) pairs, zone by zone: dispatch decision (Algorithms 2-3,
// wait-then-race), TTFT, which decode stream applies (migration trigger, Eq. 4), tokens per endpoint.
//
// Along an ascending budget axis the policies differ in thresholds that are ordered: Algorithm 3's l_th does not
// increase, Algorithm 2's l* does not decrease.  For one request a family of up to 128 such policies (four tiles
// of 32) therefore falls into at most three runs of neighbours that dispatch it alike:
//   Algorithm 3:  policies [0, k) have l_th > l  -> device only;   [k, npol) race at once (wait 0);
//   Algorithm 2:  policies [0, k1) have l* < l   -> wait w_tail;   [k1, k2) have l* = l -> wait their own w*;
//                 [k2, npol) have l* > l         -> wait 0.
// k, k1, k2 depend on the prompt length alone, and the requests of a group are stored by prompt length.  A chunk of
// requests therefore splits into a few SEGMENTS of consecutive requests that share (k1, k2); the block that owns a
// (chunk, family) works through them one after another.  Within a segment a lane takes a request and works out
//   the outcome of the last run, which goes to what EVERY policy of the family gets (sums in the lane's
//   registers, a histogram in shared memory), and
//   the outcome of the first run, whose difference to the former is summed up for the segment.
// When the segment is done the block enters that difference ONCE: into row k1 of a table of sums, carried to the
// policies below k1 when the chunk is done; its histogram into a row per whole tile below k1 and, for the
// policies below k1 inside k1's own tile, straight into their global histograms.  A segment whose prompt length is
// some policies' l* is swept once more per such policy, for that policy alone.  If a run's policies also agree on the
// race and on the migration trigger, nothing is done per pair.  What the runs cannot express -- waits that straddle
// the server's TTFT, a saving between the family's smallest and largest migration overhead -- is flagged in a bit
// mask and left to the pair-by-pair kernel (pairs.cu).
#include <cstddef>

#include "tile.cuh"

namespace disco {

namespace {

#ifndef DISCO_ZONE_THREADS
#define DISCO_ZONE_THREADS 1024
#endif
#ifndef DISCO_ZONE_BLOCKS_PER_SM
#define DISCO_ZONE_BLOCKS_PER_SM 1
#endif
constexpr int kZThreads = DISCO_ZONE_THREADS;
constexpr int kZBlocksPerSm = DISCO_ZONE_BLOCKS_PER_SM;
constexpr int kZWarps = kZThreads / 32;
constexpr int kFamTiles = 4;            // tiles of 32 policies a family may span
constexpr int kFamPol = 32 * kFamTiles;
constexpr int kSumRows = kFamPol + 1;   // difference rows of the sums: row q is carried to the policies below q
constexpr int kCoarseRows = kFamTiles + 1;   // ... of the histograms: row t is carried to every policy of the tiles below t
constexpr int kMaxSeg = 2 * kFamPol + 2;
constexpr int kJRows = 33;              // rows a single request may enter a difference at: within the first tile
enum ZSum { Z_TD = 0, Z_PS, Z_PD, Z_TAU, Z_DL, Z_DO, Z_RACE, Z_DW, Z_MIGR, Z_TT, kZSums };
constexpr int kLenTab = kMaxPrompt + 8; // bytes per table over the prompt lengths 0 .. 4096
static_assert(kZWarps >= kZSums, "the sums go out one warp per field");

struct Seg { uint32_t pa, pb; int32_t k1, k2; };       // requests [pa, pb) of the chunk share (k1, k2)

struct ZoneSmem {
    uint32_t g_ttft[kNBins], g_stall[kNBins];           // the segment in work: what every policy gets
    uint32_t h_ttft[kNBins], h_stall[kNBins];           // ... the first run (or a policy with l* = l)
    int32_t c_ttft[kNBins], c_stall[kNBins];            // the chunk: what every policy gets
    int32_t k_ttft[kCoarseRows][kNBins], k_stall[kCoarseRows][kNBins];   // coarse difference rows
    long long e_sum[kSumRows][kZSums];                  // difference rows of the sums
    long long c_sum[kZSums];                            // what every policy gets
    long long part[kZWarps][kZSums];                    // the warps' shares of a segment's difference
    int32_t j_sum[kJRows][kZSums];                      // differences entered request by request during a sweep, rows 1 .. 32
    uint32_t n_left, n_apart, n_listed, n_listed0, n_seg, ticket;
    uint32_t red[4];                                    // smallest / largest overhead (float bits), smallest / largest w_tail
    Seg seg[kMaxSeg];
    int32_t key[kFamPol];                               // the policies' length thresholds, in list order
    uint32_t w_star[kFamPol];                           // Algorithm 2: the wait of the length class l*
    uint32_t w_tail[kFamPol];                           // ... and of the longer prompts
    float theta[kFamPol];                               // Eq. 4's overhead (+inf: the policy never hands over)
    uint32_t pol[kFamPol];                              // the policies' indices in the caller's list
    uint32_t e_len[kFamPol];                            // expected length for Eq. 4
    uint8_t kind[kFamPol];                              // 0 Algorithm 3, 1 Algorithm 2, 2 neither (not a plain policy)
    uint8_t tab1[kLenTab], tab2[kLenTab];
};

struct Req { uint32_t l, n, S, m, dly, stall, nt0, nt1, nt2; };

// What a lane has summed up: the sums of one outcome per request, or of differences between two.
struct Sums {
    int32_t td, ps, pd, tau, dl, c_do, c_race, c_dw, c_migr;
    long long tt;
};

__device__ __forceinline__ void clear(Sums& s) { s.td = s.ps = s.pd = s.tau = s.dl = s.c_do = s.c_race = s.c_dw = s.c_migr = 0; s.tt = 0; }

// Adds sign times what a request that ends in outcome oc with TTFT tt contributes.
__device__ __forceinline__ void add_outcome(Sums& s, int sign, int oc, const Req& r, uint32_t tt) {
    const bool migr = oc >= O_MIGR_TO_DEV, dev_wins = (oc & 1) != 0;
    const uint32_t lm = r.l + r.m;
    const uint32_t td = migr ? (dev_wins ? r.m : r.n - r.m) : (dev_wins ? r.n : 0u);         // tokens the device generated
    const uint32_t ps = oc == O_DEVICE_ONLY ? 0u : r.l + ((migr && dev_wins) ? lm : 0u);     // prompt tokens billed by the server
    const uint32_t pd = oc == O_SERVER_ONLY ? 0u : r.l + ((migr && !dev_wins) ? lm : 0u);    // ... by the device
    const uint32_t tau = migr ? r.nt2 : (dev_wins ? r.nt1 : r.nt0);                          // TBTs in the bin of tau
    s.td += sign * (int32_t)td; s.ps += sign * (int32_t)ps; s.pd += sign * (int32_t)pd; s.tau += sign * (int32_t)tau;
    s.dl += migr ? sign * (int32_t)r.dly : 0;
    s.c_do += oc == O_DEVICE_ONLY ? sign : 0;
    s.c_race += oc >= O_RACE_SRV ? sign : 0;
    s.c_dw += (oc == O_RACE_DEV || oc == O_MIGR_TO_SRV) ? sign : 0;
    s.c_migr += migr ? sign : 0;
    s.tt += sign * (long long)tt;
}

__device__ __forceinline__ long long field_of(const Sums& s, int f) {
    switch (f) {
        case Z_TD: return s.td; case Z_PS: return s.ps; case Z_PD: return s.pd; case Z_TAU: return s.tau;
        case Z_DL: return s.dl; case Z_DO: return s.c_do; case Z_RACE: return s.c_race; case Z_DW: return s.c_dw;
        case Z_MIGR: return s.c_migr; default: return s.tt;
    }
}

// Everything a lane needs to evaluate requests of one (chunk, family).
struct TileCtx {
    const TraceDev* tr; const TimelineRec* rec; const Chunk* ch;
    uint32_t tau, kappa, c0, E0, wt_min, wt_max;
    float delta_c, th_min, th_max;
    int npol, race_that_migrates;
    bool may_migrate;
    bool wt_ordered;                    // the policies' w_tail do not increase along the family
    bool tile0_apart;                   // more than one tile, and only the first tile's w_tail differ from wt_min
};

// With every stream delivered at the pace tau the TBTs in tau's bin are all n - 1 intervals (n - 2 beside a
// hand-off); a hand-off stall of exactly tau counts with them, any other gets a histogram increment of its own
// (stall_bin).
__device__ __forceinline__ Req load_request(const TileCtx& c, uint32_t i, bool& stall_bin) {
    const uint32_t kk = c.ch->start + min(i, c.ch->len - 1);
    Req q;
    q.l = c.tr->l[kk]; q.n = c.tr->nout[kk]; q.S = (uint32_t)c.tr->S[kk];
    q.m = 0; q.dly = 0; q.stall = c.tau;
    if (c.may_migrate) { q.m = c.rec->m[kk]; q.dly = c.rec->delayed[kk]; q.stall = c.rec->stall[kk]; }
    const uint32_t nI = q.n - 1;
    q.nt0 = nI; q.nt1 = nI; q.nt2 = nI ? nI - 1 : 0u;
    stall_bin = q.stall != c.tau;
    if (!stall_bin) ++q.nt2;
    return q;
}

// Eq. 4's projected saving, on the true remainder or on what is left of the expected length; a request may only
// hand over if its buffer filled (m != 0).
__device__ __forceinline__ float saving_of(const TileCtx& c, const Req& q) {
    if (!c.may_migrate || q.m == 0) return -1.0f;
    return c.delta_c * (float)(c.E0 ? (uint32_t)max((int32_t)c.E0 - (int32_t)q.m, 0) : q.n - q.m);
}

// The migration trigger over the whole family for a race outcome: 0 no policy hands over, 1 every policy does,
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
//
// apart: in a family of several tiles whose first tile alone has waits above wt_min, the device wins under the
// policies of the other tiles at wt_min + T_d while the first tile's policies each end their own way: the outcome
// then holds for the tiles after the first, and the request is left to the pair kernel for the first tile only.
__device__ __forceinline__ bool head_outcome_waits(const TileCtx& c, const ZoneSmem& sm, const Req& q, uint32_t Td,
                                                   float saving, int k1, int& oc, uint32_t& tt, int& j, bool& apart) {
    int base;
    tt = q.S;
    j = 0;
    apart = false;
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
    } else if (c.wt_min == c.wt_max || c.tile0_apart) {                        // the device wins under every policy
        base = O_RACE_DEV; tt = c.wt_min + Td;                                 // (of the tiles after the first)
        apart = c.wt_min != c.wt_max;
    } else return false;
    const int t = trigger_all(c, base, saving);
    oc = base + 2 * t;
    return t >= 0;
}

// One more count in a block-private histogram, for counts that tend to meet in one bin (requests of one prompt
// length share the device's TTFT): if all the warp's counts fall in one bin, one lane adds them.
__device__ __forceinline__ void hist_add(uint32_t* hist, bool on, int bin) {
    on = on && DBG_OK(bin, kNBins, DBG_K_PAIRS_ZONES, DBG_BIN);
    const uint32_t live = __ballot_sync(0xFFFFFFFFu, on);
    if (live == 0u) return;
    const int leader = __ffs(live) - 1;
    const int bin0 = __shfl_sync(0xFFFFFFFFu, bin, leader);
    if (__all_sync(0xFFFFFFFFu, !on || bin == bin0)) {
        if ((int)(threadIdx.x & 31) == leader) atomicAdd(&hist[bin0], (uint32_t)__popc(live));
    } else if (on) {
        atomicAdd(&hist[bin], 1u);
    }
}

// The same for counts that are rare or spread over many bins: every lane adds for itself.
__device__ __forceinline__ void hist_add_each(uint32_t* hist, bool on, int bin) {
    if (on && DBG_OK(bin, kNBins, DBG_K_PAIRS_ZONES, DBG_BIN)) atomicAdd(&hist[bin], 1u);
}

// One request's difference into a row of 32-bit sums (the TTFT sum is not entered: the caller sees to it).  A
// segment's rows are added to the 64-bit ones when the segment is entered; a sum stays below 2^31 over a chunk.
__device__ __forceinline__ void enter_small(int32_t* row, const Sums& e) {
#pragma unroll
    for (int f = 0; f < kZSums; ++f) {
        if (f == Z_TT) continue;
        const int v = (int)field_of(e, f);
        if (v) atomicAdd(&row[f], v);
    }
}

// What a request comes to under the policies of its segment.
struct Fate {
    bool ok;                            // the runs express it
    bool apart;                         // ... except for the policies of the family's first tile
    int oc_c, oc_h, j;                  // outcome every policy gets; outcome of the first run [j, k1); covered waits [0, j)
    uint32_t tt_c, tt_h;
};

// k1, k2: the segment's.  With k2 < npol what every policy gets is the last run's outcome and the first run (if
// any) differs from it; with k1 = k2 = npol every policy is in the first run, whose outcome then is what every
// policy gets.
template <bool WAITS>
__device__ __forceinline__ Fate fate_of(const TileCtx& c, const ZoneSmem& sm, const Req& q, uint32_t Td, float saving,
                                         int k1, int k2) {
    Fate v;
    v.oc_c = O_DEVICE_ONLY; v.oc_h = O_DEVICE_ONLY; v.j = 0; v.tt_c = Td; v.tt_h = Td; v.ok = true; v.apart = false;
    if (k2 < c.npol) {
        v.ok = tail_outcome(c, q, Td, saving, v.oc_c, v.tt_c);
        if (WAITS && k1 > 0) v.ok = head_outcome_waits(c, sm, q, Td, saving, k1, v.oc_h, v.tt_h, v.j, v.apart) && v.ok;
    } else if (WAITS) {
        v.ok = head_outcome_waits(c, sm, q, Td, saving, k1, v.oc_c, v.tt_c, v.j, v.apart);
        v.oc_h = v.oc_c; v.tt_h = v.tt_c;
    }
    v.apart = v.apart && v.ok;
    return v;
}

// Where a block's results go.
struct FlushTo {
    unsigned long long *acc, *hist_ttft, *hist_tbt;
    int n_groups, g, bin_tau;
};

// One sweep over the requests [s.pa, s.pb) of the chunk.  point < 0: the segment's main sweep -- what every policy
// gets (into `every` and g_*), the first run's difference to it (returned, and h_*), covered waits, requests the
// runs cannot express.  point >= 0: the sweep for that policy alone, one with l* = l: its difference to what every
// policy gets is returned, its histograms go to h_*.
template <bool WAITS>
__device__ __forceinline__ Sums sweep(ZoneSmem& sm, const TileCtx& c, const Seg& s, int point, Sums& every, uint32_t& n_left,
                                      uint32_t& n_apart, uint32_t tile0, int n_fam, uint32_t n_tiles,
                                      uint32_t* __restrict__ left_mask, uint32_t* __restrict__ left_list, const FlushTo& out) {
    const int lane = threadIdx.x & 31;
    const int k1 = s.k1, k2 = s.k2;
    const bool first_run = k2 < c.npol && k1 > 0;                // a first run that differs from what every policy gets
    const uint32_t words = left_words_per_request(n_tiles);
    const uint32_t left_bits = ((1u << n_fam) - 1u) << (tile0 & 31u);       // (a family does not straddle a mask word)
    Sums d;
    clear(d);
    long long tt_back = 0;                                       // TTFTs taken back at row 32 (requests left for the first tile alone)
    for (uint32_t i0 = s.pa + (threadIdx.x & ~31u); i0 < s.pb; i0 += kZThreads) {      // a warp's lanes iterate together
        const uint32_t i = i0 + lane;
        bool stall_bin;
        const Req q = load_request(c, i, stall_bin);
        const bool valid = i < s.pb;
        const uint32_t Td = c.kappa * q.l + c.c0;
        const float saving = saving_of(c, q);
        const Fate v = fate_of<WAITS>(c, sm, q, Td, saving, k1, k2);
        const bool ok = v.ok && valid;
        const bool apart = v.apart && valid;                     // left to the pair kernel for the first tile alone
        if (point < 0) {
            if (valid && (!ok || apart)) {
                // left to the pair kernel: for every tile of the family, or for the first one alone
                atomicOr(&left_mask[(size_t)(c.ch->start + i) * words + (tile0 >> 5)], ok ? 1u << (tile0 & 31u) : left_bits);
                if (ok) ++n_apart; else ++n_left;
                if (left_list) {
                    const uint32_t at0 = atomicAdd(&sm.n_listed0, 1u);
                    if (at0 < kLeftList) left_list[at0] = i;
                    if (!ok && n_fam > 1) {
                        const uint32_t at = atomicAdd(&sm.n_listed, 1u);
                        if (at < kLeftList) for (int t = 1; t < n_fam; ++t) left_list[(size_t)t * kLeftList + at] = i;
                    }
                }
            }
            if (ok) add_outcome(every, 1, v.oc_c, q, v.tt_c);
            hist_add_each(sm.g_ttft, ok, bin_of_ticks(v.tt_c));
            if (c.may_migrate) hist_add_each(sm.g_stall, ok && v.oc_c >= O_MIGR_TO_DEV && stall_bin, bin_of_ticks(q.stall));
            // (a request left for the first tile alone, whose first run lies inside that tile: no first run to enter)
            const bool runs = ok && !(WAITS && apart && k1 < 32);
            if (first_run) {
                if (runs) { add_outcome(d, 1, v.oc_h, q, v.tt_h); add_outcome(d, -1, v.oc_c, q, v.tt_c); }
                // (h_* minus g_* is entered for the segment: a request without a first run joins both)
                // (Algorithm 3: the first run's TTFT is the device's, one bin for a prompt length; Algorithm 2: mostly
                // the server's own, spread over the bins)
                if (WAITS) hist_add_each(sm.h_ttft, ok, bin_of_ticks(runs ? v.tt_h : v.tt_c));
                else hist_add(sm.h_ttft, ok, bin_of_ticks(runs ? v.tt_h : v.tt_c));
                if (c.may_migrate) hist_add_each(sm.h_stall, ok && (runs ? v.oc_h : v.oc_c) >= O_MIGR_TO_DEV && stall_bin, bin_of_ticks(q.stall));
            }
            if (WAITS && c.tile0_apart) {
                // ---- the first tile gets nothing from the family for such a request (the pair kernel evaluates it there):
                //      what its policies would get is taken back at row 32, the row carried to the first tile
                if (__ballot_sync(0xFFFFFFFFu, apart)) {
                    const bool head = first_run && k1 >= 32;             // they would get the first run's outcome, else the common one
                    const int oc_x = head ? v.oc_h : v.oc_c;
                    const uint32_t tt_x = head ? v.tt_h : v.tt_c;
                    if (apart) {
                        Sums e;
                        clear(e);
                        add_outcome(e, -1, oc_x, q, tt_x);
                        enter_small(sm.j_sum[32], e);
                        tt_back += e.tt;                                 // (entered once, when the sweep is over)
                        if (DBG_OK(bin_of_ticks(tt_x), kNBins, DBG_K_PAIRS_ZONES, DBG_BIN)) atomicSub(&sm.k_ttft[1][bin_of_ticks(tt_x)], 1);
                        if (oc_x >= O_MIGR_TO_DEV && stall_bin) atomicSub(&sm.k_stall[1][bin_of_ticks(q.stall)], 1);
                    }
                }
            }
            if (WAITS && c.wt_min != c.wt_max) {
                // ---- waits that cover the server's TTFT: the policies [0, j) end in O_SERVER_ONLY instead of the first
                //      run's outcome (a race the server wins, with the same TTFT).  The lanes that share j add up.
                const bool has_j = ok && v.j > 0 && DBG_OK(v.j, kJRows, DBG_K_PAIRS_ZONES, DBG_SLOT);
                if (has_j) {
                    Sums e;
                    clear(e);
                    add_outcome(e, 1, O_SERVER_ONLY, q, q.S); add_outcome(e, -1, v.oc_h, q, v.tt_h);   // (the two TTFTs are equal)
                    enter_small(sm.j_sum[v.j], e);
                    // a hand-off stall the first run would have had: those policies lose it
                    if (v.oc_h >= O_MIGR_TO_DEV && stall_bin)
                        for (int p = 0; p < v.j; ++p)
                            atomicAdd(&out.hist_tbt[(size_t)sm.pol[p] * kNBins + bin_of_ticks(q.stall)], ~0ull);
                }
            }
        } else {
            // the policy's own wait w*
            const uint32_t w = sm.w_star[point];
            int oc = O_SERVER_ONLY;
            uint32_t tt = q.S;
            if (q.S > w) {                                       // the device starts after the wait
                tt = min(q.S, w + Td);
                oc = q.S > w + Td ? O_RACE_DEV : O_RACE_SRV;     // a tie goes to the server
                if (oc == c.race_that_migrates && saving > sm.theta[point]) oc += 2;
            }
            const bool mine = ok && !(apart && point < 32);    // (the pair kernel has the first tile of such a request)
            if (mine) { add_outcome(d, 1, oc, q, tt); add_outcome(d, -1, v.oc_c, q, v.tt_c); }
            // (h_* minus g_* is entered for the policy: a request that is not its own joins both)
            hist_add_each(sm.h_ttft, ok, bin_of_ticks(mine ? tt : v.tt_c));
            if (c.may_migrate) hist_add_each(sm.h_stall, ok && (mine ? oc : v.oc_c) >= O_MIGR_TO_DEV && stall_bin, bin_of_ticks(q.stall));
        }
    }
    if (WAITS && c.tile0_apart && point < 0) {
#pragma unroll
        for (int off = 16; off > 0; off >>= 1) tt_back += __shfl_xor_sync(0xFFFFFFFFu, tt_back, off);
        if (lane == 0 && tt_back) atomicAdd((unsigned long long*)&sm.e_sum[32][Z_TT], (unsigned long long)tt_back);
    }
    return d;
}

// The warps' shares of a lane-wise sum go to sm.part (to be added up by one thread per field after a barrier).
__device__ __forceinline__ void share_out(ZoneSmem& sm, const Sums& s) {
    const int lane = threadIdx.x & 31, w = threadIdx.x >> 5;
#pragma unroll
    for (int f = 0; f < kZSums; ++f) {
        long long v = field_of(s, f);
        if (f == Z_TT) {
#pragma unroll
            for (int off = 16; off > 0; off >>= 1) v += __shfl_xor_sync(0xFFFFFFFFu, v, off);
        } else {
            v = __reduce_add_sync(0xFFFFFFFFu, (int)v);
        }
        if (lane == 0) sm.part[w][f] = v;
    }
}

// After a sweep (barrier before): enters the difference the sweep returned (shared out to sm.part) and its
// histograms h_* minus g_*.  row > 0: for the policies below `row` -- sums row, coarse histogram rows, and global
// histograms of the policies of row's own tile.  alone >= 0: for that policy alone.  With add_every, g_* joins what
// every policy gets.  Clears h_* and, with clear_g, g_*.  All threads call; barrier after.
__device__ __forceinline__ void enter_segment(ZoneSmem& sm, int row, int alone, bool add_every, bool clear_g, const FlushTo& out) {
    for (int b = threadIdx.x; b < kNBins + kZSums + kJRows * kZSums; b += kZThreads) {
    if (b < kNBins) {
        const int32_t gt = (int32_t)sm.g_ttft[b], gs = (int32_t)sm.g_stall[b];
        const int32_t dt = (int32_t)sm.h_ttft[b] - gt, ds = (int32_t)sm.h_stall[b] - gs;
        if (add_every) { sm.c_ttft[b] += gt; sm.c_stall[b] += gs; }
        if (row > 0) {
            const int t = row >> 5, r = row & 31;
            if (t) { sm.k_ttft[t][b] += dt; sm.k_stall[t][b] += ds; }
            if (dt | ds) {
                for (int p = 32 * t; p < 32 * t + r; ++p) {
                    const size_t o = (size_t)sm.pol[p] * kNBins + b;
                    if (dt) atomicAdd(&out.hist_ttft[o], (unsigned long long)(long long)dt);
                    if (ds) atomicAdd(&out.hist_tbt[o], (unsigned long long)(long long)ds);
                }
            }
        } else if (alone >= 0) {
            const size_t o = (size_t)sm.pol[alone] * kNBins + b;
            if (dt) atomicAdd(&out.hist_ttft[o], (unsigned long long)(long long)dt);
            if (ds) atomicAdd(&out.hist_tbt[o], (unsigned long long)(long long)ds);
        }
        sm.h_ttft[b] = 0; sm.h_stall[b] = 0;
        if (clear_g) { sm.g_ttft[b] = 0; sm.g_stall[b] = 0; }
    } else if (b < kNBins + kZSums) {
        if (row > 0 || alone >= 0) {
            const int f = b - kNBins;
            long long v = 0;
            for (int w = 0; w < kZWarps; ++w) v += sm.part[w][f];
            // (atomic: the threads below may add to the same row)
            unsigned long long* e = (unsigned long long*)&sm.e_sum[row > 0 ? row : alone + 1][f];
            atomicAdd(e, (unsigned long long)v);
            if (row <= 0 && alone > 0) atomicAdd((unsigned long long*)&sm.e_sum[alone][f], 0ull - (unsigned long long)v);   // (row 0 is carried to nobody)
        }
    } else {
        // what single requests entered during the sweep
        const int k = b - kNBins - kZSums, r = k / kZSums, f = k % kZSums;
        const int32_t v = sm.j_sum[r][f];
        if (v) { atomicAdd((unsigned long long*)&sm.e_sum[r][f], (unsigned long long)(long long)v); sm.j_sum[r][f] = 0; }
    }
    }
}

// Adds the sums rows and what every policy gets to the policies' global sums.  All threads call (barrier before).
__device__ __forceinline__ void flush_sums(const ZoneSmem& sm, int npol, const FlushTo& to) {
    const int lane = threadIdx.x & 31, f = threadIdx.x >> 5;                    // a warp per field
    if (f >= kZSums) return;
    long long above = sm.c_sum[f];                                              // what every policy gets + the rows above the segment
    for (int seg = (npol - 1) >> 5; seg >= 0; --seg) {                          // 32 policies at a time, last first
        const int p = seg * 32 + lane;
        long long v = p < npol ? sm.e_sum[p + 1][f] : 0;                        // policy p gets the rows above it: p + 1 ..
#pragma unroll
        for (int off = 1; off < 32; off <<= 1) {                                // sums over the lanes from this one on
            const long long a = __shfl_down_sync(0xFFFFFFFFu, v, off);
            if (lane + off < 32) v += a;
        }
        v += above;
        above = __shfl_sync(0xFFFFFFFFu, v, 0);
        if (p >= npol || v == 0) continue;
        const uint32_t pp = sm.pol[p];
        unsigned long long* a = to.acc + ((size_t)pp * to.n_groups + to.g) * kNAcc;
        const unsigned long long u = (unsigned long long)v;
        switch (f) {
            case Z_TD: atomicAdd(&a[A_TOK_DEVICE], u); break;
            case Z_PS: atomicAdd(&a[A_PRE_SERVER], u); break;
            case Z_PD: atomicAdd(&a[A_PRE_DEVICE], u); break;
            case Z_TAU: atomicAdd(&to.hist_tbt[(size_t)pp * kNBins + to.bin_tau], u); break;
            case Z_DL: atomicAdd(&a[A_DELAYED], u); break;
            case Z_DO: atomicAdd(&a[A_DEVICE_ONLY], u); break;
            case Z_RACE: atomicAdd(&a[A_RACE], u); break;
            case Z_DW: atomicAdd(&a[A_DEVICE_WON], u); break;
            case Z_MIGR: atomicAdd(&a[A_MIGR], u); break;
            default: atomicAdd(&a[A_TTFT_SUM], u); break;                       // Z_TT
        }
    }
}

// Adds to the global histograms of every policy what the chunk gave all of them plus the coarse rows above the
// policy's tile.  All threads call (barrier before).
__device__ __forceinline__ void flush_hist(const ZoneSmem& sm, int n_fam, int npol, const FlushTo& to) {
    for (int b = threadIdx.x; b < kNBins; b += kZThreads) {
        int32_t t = sm.c_ttft[b], s = sm.c_stall[b];
        for (int tile = n_fam - 1; tile >= 0; --tile) {
            if (tile + 1 < kCoarseRows) { t += sm.k_ttft[tile + 1][b]; s += sm.k_stall[tile + 1][b]; }
            if ((t | s) == 0) continue;
            for (int p = 32 * tile; p < min(npol, 32 * tile + 32); ++p) {
                const size_t o = (size_t)sm.pol[p] * kNBins + b;
                if (t) atomicAdd(&to.hist_ttft[o], (unsigned long long)(long long)t);
                if (s) atomicAdd(&to.hist_tbt[o], (unsigned long long)(long long)s);
            }
        }
    }
}

// What a family's evaluation of a chunk reports.
struct FamTotals { uint32_t left, apart, passes; };   // apart: left for the first tile alone

// One chunk under one family of n_fam tiles starting at tile0 (the shared tables of the family are set up).
// WAITS: the policies are Algorithm 2's (wait map); otherwise Algorithm 3's (length threshold).
template <bool WAITS>
__device__ __forceinline__ FamTotals zone_family(ZoneSmem& sm, const TileCtx& c, uint32_t tile0, int n_fam, uint32_t n_tiles,
                                                 uint32_t chunk_id, const uint32_t* __restrict__ len_end,
                                                 uint32_t* __restrict__ left_mask, uint32_t* __restrict__ left_lists,
                                                 const FlushTo& out) {
    const int npol = c.npol;
    const uint32_t len = c.ch->len;
    uint32_t* left_list = left_lists ? left_lists + ((size_t)chunk_id * n_tiles + tile0) * kLeftList : nullptr;
    for (int i = threadIdx.x; i < (int)(offsetof(ZoneSmem, red) / 4); i += kZThreads) ((uint32_t*)&sm)[i] = 0;
    __syncthreads();

    // ---- the segments: stretches of prompt lengths between two thresholds, and (Algorithm 2) the thresholds
    //      themselves; a thread per candidate looks up where its lengths lie in the chunk
    {
        const int n_cand = len ? (WAITS ? 2 * npol + 1 : npol + 1) : 0;
        for (int q = threadIdx.x; q < n_cand; q += kZThreads) {
            auto cl = [](int x) { return min(max(x, 0), kMaxPrompt + 1); };
            int la, lb;
            bool any = true;
            if (WAITS) {                                             // thresholds ascend
                const int p = q >> 1;
                if (q == 2 * npol) { la = cl(sm.key[npol - 1] + 1); lb = kMaxPrompt + 1; }
                else if (q & 1) { la = cl(sm.key[p]); lb = cl(sm.key[p] + 1); any = p == 0 || sm.key[p] != sm.key[p - 1]; }
                else { la = p ? cl(sm.key[p - 1] + 1) : 0; lb = cl(sm.key[p]); }
            } else {                                                 // thresholds descend
                la = q ? cl(sm.key[npol - q]) : 0;
                lb = q < npol ? cl(sm.key[npol - 1 - q]) : kMaxPrompt + 1;
            }
            if (any && la < lb) {
                // first request of the group with a prompt of at least L tokens: where the shorter ones end
                const uint32_t* ends = len_end + (size_t)c.ch->g * (kMaxPrompt + 1);
                const uint32_t g0 = c.tr->grp_off[c.ch->g];
                const uint32_t at_a = la ? ends[la - 1] : g0, at_b = ends[lb - 1];
                const uint32_t lo = c.ch->start, hi = c.ch->start + len;
                const uint32_t pa = min(max(at_a, lo), hi) - lo, pb = min(max(at_b, lo), hi) - lo;
                if (pa < pb) {
                    const uint32_t at = atomicAdd(&sm.n_seg, 1u);
                    if (DBG_OK(at, kMaxSeg, DBG_K_PAIRS_ZONES, DBG_SLOT)) {
                        Seg s;
                        s.pa = pa; s.pb = pb; s.k1 = sm.tab1[la]; s.k2 = WAITS ? sm.tab2[la] : s.k1;
                        sm.seg[at] = s;
                    }
                }
            }
        }
    }
    __syncthreads();

    Sums every;
    clear(every);
    uint32_t n_left = 0, n_apart = 0, passes = 0;
    const int n_seg = (int)min(sm.n_seg, (uint32_t)kMaxSeg);
    for (int si = 0; si < n_seg; ++si) {
        const Seg s = sm.seg[si];
        const bool points = s.k2 < npol && s.k2 > s.k1;
        const bool no_run = s.k2 >= npol && s.k1 < npol;              // l* = l for the last policies and nobody waits 0
        if (no_run) {
            // the pair kernel takes these requests
            for (uint32_t i = s.pa + threadIdx.x; i < s.pb; i += kZThreads) {
                atomicOr(&left_mask[(size_t)(c.ch->start + i) * left_words_per_request(n_tiles) + (tile0 >> 5)],
                         ((1u << n_fam) - 1u) << (tile0 & 31u));
                ++n_left;
                if (left_list) {
                    const uint32_t at0 = atomicAdd(&sm.n_listed0, 1u), at = n_fam > 1 ? atomicAdd(&sm.n_listed, 1u) : 0u;
                    if (at0 < kLeftList) left_list[at0] = i;
                    if (at < kLeftList) for (int t = 1; t < n_fam; ++t) left_list[(size_t)t * kLeftList + at] = i;
                }
            }
            continue;
        }
        const Sums d = sweep<WAITS>(sm, c, s, -1, every, n_left, n_apart, tile0, n_fam, n_tiles, left_mask, left_list, out);
        const bool first_run = s.k2 < npol && s.k1 > 0;
        if (first_run) share_out(sm, d);
        __syncthreads();
        enter_segment(sm, first_run ? s.k1 : 0, -1, true, !points, out);
        __syncthreads();
        ++passes;
        if (WAITS && points) {
            for (int p = s.k1; p < s.k2; ++p) {
                const Sums dp = sweep<WAITS>(sm, c, s, p, every, n_left, n_apart, tile0, n_fam, n_tiles, left_mask, left_list, out);
                share_out(sm, dp);
                __syncthreads();
                enter_segment(sm, 0, p, false, p + 1 == s.k2, out);
                __syncthreads();
                ++passes;
            }
        }
    }
    // ---- the chunk is done: what every policy gets, then everything goes out
    share_out(sm, every);
    n_left = __reduce_add_sync(0xFFFFFFFFu, n_left);
    n_apart = __reduce_add_sync(0xFFFFFFFFu, n_apart);
    if ((threadIdx.x & 31) == 0 && (n_left | n_apart)) { atomicAdd(&sm.n_left, n_left); atomicAdd(&sm.n_apart, n_apart); }
    __syncthreads();
    if (threadIdx.x < kZSums) {
        long long v = 0;
        for (int w = 0; w < kZWarps; ++w) v += sm.part[w][threadIdx.x];
        sm.c_sum[threadIdx.x] = v;
    }
    __syncthreads();
    flush_sums(sm, npol, out);
    flush_hist(sm, n_fam, npol, out);
    FamTotals tot;
    tot.left = sm.n_left;
    tot.apart = sm.n_apart;
    tot.passes = passes;
    __syncthreads();
    return tot;
}

// Loads the policies [first, first + npol) of the list into the shared tables and tells whether they can be
// evaluated as one family: plain Algorithm 2 or plain Algorithm 3 policies of one kind (no random routing, no
// Eq. 1-2 wait rule, one expected length for Eq. 4) whose length thresholds are ordered along the list --
// Algorithm 3's l_th not increasing, Algorithm 2's l* not decreasing, as they are along an ascending budget axis.
// In a family of more than one tile of Algorithm 2 policies, only the first tile's waits w_tail may differ from the
// smallest one (as they do along a budget axis: the lowest budgets wait longest).  All threads call.
__device__ __forceinline__ bool family_setup(ZoneSmem& sm, TileCtx& c, const Prep* __restrict__ prep, uint32_t P, int g,
                                             const GroupConst& gc, const uint32_t* __restrict__ pol_list, uint32_t first,
                                             int npol, bool& waits) {
    const int p = threadIdx.x;
    __syncthreads();                                                  // (earlier readers of the tables are done)
    if (p == 0) { sm.red[0] = 0x7F800000u; sm.red[1] = 0u; sm.red[2] = 0xFFFFFFFFu; sm.red[3] = 0u; }
    __syncthreads();
    if (p < npol) {
        const uint32_t pp = DBG_OK(pol_list[first + p], P, DBG_K_PAIRS_ZONES, DBG_POLICY) ? pol_list[first + p] : 0u;
        const Prep pr = prep[(size_t)g * P + pp];
        const float theta = (pr.mig_on && gc.candidate != 0) ? pr.theta : __int_as_float(0x7F800000);
        sm.key[p] = pr.device_constrained ? pr.l_star : pr.l_th;
        sm.w_star[p] = (uint32_t)pr.w_star;
        sm.w_tail[p] = (uint32_t)pr.w_tail;
        sm.theta[p] = theta;
        sm.pol[p] = pp;
        sm.e_len[p] = pr.expected_len;
        sm.kind[p] = (pr.stochastic || pr.beta_rule) ? 2 : (pr.device_constrained ? 1 : 0);
        // thresholds are non-negative floats or +inf: their bit patterns order like the values
        atomicMin(&sm.red[0], __float_as_uint(theta)); atomicMax(&sm.red[1], __float_as_uint(theta));
        atomicMin(&sm.red[2], (uint32_t)pr.w_tail); atomicMax(&sm.red[3], (uint32_t)pr.w_tail);
    }
    __syncthreads();
    waits = sm.kind[0] == 1;
    bool ok = true, wt_ok = true;
    if (p < npol) {
        ok = sm.kind[p] != 2 && sm.kind[p] == sm.kind[0] && sm.e_len[p] == sm.e_len[0];
        if (p + 1 < npol) {
            ok = ok && (waits ? sm.key[p] <= sm.key[p + 1] : sm.key[p] >= sm.key[p + 1]);
            wt_ok = sm.w_tail[p] >= sm.w_tail[p + 1];
        }
    }
    ok = __syncthreads_and(ok) != 0;
    c.wt_ordered = __syncthreads_and(wt_ok) != 0;
    c.npol = npol;
    c.E0 = sm.e_len[0];
    c.th_min = __uint_as_float(sm.red[0]); c.th_max = __uint_as_float(sm.red[1]);
    c.wt_min = sm.red[2]; c.wt_max = sm.red[3];
    c.may_migrate = c.th_min != __int_as_float(0x7F800000);          // some policy of the family can hand over
    // several tiles of Algorithm 2 policies: beyond the first tile the waits w_tail must all be the smallest one
    const bool rest_alike = __syncthreads_and(p < 32 || p >= npol || sm.w_tail[p] == c.wt_min) != 0;
    c.tile0_apart = npol > 32 && waits && c.wt_min != c.wt_max;
    if (c.tile0_apart && !(rest_alike && c.wt_ordered)) ok = false;
    return ok;
}

__global__ void __launch_bounds__(kZThreads, kZBlocksPerSm)
k_pairs_zones(TraceDev tr, const GroupConst* __restrict__ gcs, const ClassConst* __restrict__ ccp,
              const Prep* __restrict__ prep, uint32_t P, const uint32_t* __restrict__ pol_list, uint32_t n_list,
              int PL, const Chunk* __restrict__ chunks, uint32_t n_chunks, uint32_t n_tiles, TimelineRec rec,
              unsigned long long* __restrict__ acc, unsigned long long* __restrict__ hist_ttft,
              unsigned long long* __restrict__ hist_tbt, uint32_t* __restrict__ left_mask,
              uint32_t* __restrict__ left_count, uint32_t* __restrict__ left_lists,
              uint32_t* __restrict__ ticket, unsigned long long* __restrict__ work) {
    extern __shared__ __align__(16) unsigned char zsmem_raw[];
    ZoneSmem& sm = *reinterpret_cast<ZoneSmem*>(zsmem_raw);
    grid_dependency_wait();
    const ClassConst& cc = *ccp;
    // the kernel counts on pacing with one histogram bin per stream: every regular interval of a stream lies in tau's
    const bool lean = cc.pacing != 0 && cc.W[0] == 1 && cc.W[1] == 1 && cc.W[2] == 1;
    const uint32_t n_fams = (n_tiles + kFamTiles - 1) / kFamTiles;

    // the blocks draw (chunk, family) items from a counter (zero at launch): items differ in cost
    for (;;) {
        __syncthreads();
        if (threadIdx.x == 0) sm.ticket = atomicAdd(ticket, 1u);
        __syncthreads();
        const uint32_t item = sm.ticket;
        if (item >= n_chunks * n_fams) break;
        const uint32_t fam = item % n_fams, chunk_id = item / n_fams;
        const Chunk ch = chunks[chunk_id];
        const int g = ch.g;
        if (!DBG_OK(g, tr.n_groups, DBG_K_PAIRS_ZONES, DBG_GROUP) ||
            (ch.len && !DBG_OK((unsigned long long)ch.start + ch.len - 1, tr.n, DBG_K_PAIRS_ZONES, DBG_REQUEST)))
            continue;
        const GroupConst& gc = gcs[g];
        TileCtx c;
        c.tr = &tr; c.rec = &rec; c.ch = &ch;
        c.tau = (uint32_t)cc.tau; c.kappa = (uint32_t)gc.kappa; c.c0 = (uint32_t)gc.c0;
        c.delta_c = gc.delta_c;
        c.race_that_migrates = gc.candidate == 2 ? O_RACE_DEV : O_RACE_SRV;
        FlushTo out;
        out.acc = acc; out.hist_ttft = hist_ttft; out.hist_tbt = hist_tbt; out.n_groups = tr.n_groups; out.g = g;
        out.bin_tau = bin_of_ticks(c.tau);

        // the widest families the item's tiles form, first to last
        const uint32_t t_end = min(n_tiles, (fam + 1) * kFamTiles);
        for (uint32_t tile0 = fam * kFamTiles; tile0 < t_end;) {
            int n_fam = PL == 32 ? (int)(t_end - tile0) : 1;
            bool waits = false, ok = false;
            for (; lean && n_fam >= 1; --n_fam) {
                const int npol = (int)min((uint32_t)(n_fam * PL), n_list - tile0 * PL);
                ok = family_setup(sm, c, prep, P, g, gc, pol_list, tile0 * PL, npol, waits);
                if (ok) break;
            }
            if (!ok) {                                               // the pair kernel takes the tile whole
                if (threadIdx.x == 0) left_count[(size_t)chunk_id * n_tiles + tile0] = kNotByZones;
                ++tile0;
                continue;
            }
            const int npol = c.npol;
            // tables over the prompt length: how many of the family's (ordered) thresholds lie on which side of it
            for (int l = threadIdx.x; l <= kMaxPrompt; l += kZThreads) {
                int lo = 0, hi = npol;                                // first position whose threshold fails the test
                if (waits) {
                    while (lo < hi) { const int mid = (lo + hi) >> 1; if (sm.key[mid] < l) lo = mid + 1; else hi = mid; }
                    const int k1 = lo;                                // thresholds below l (ascending order)
                    hi = npol;
                    while (lo < hi) { const int mid = (lo + hi) >> 1; if (sm.key[mid] <= l) lo = mid + 1; else hi = mid; }
                    sm.tab1[l] = (uint8_t)k1; sm.tab2[l] = (uint8_t)lo;   // k1, k2
                } else {
                    while (lo < hi) { const int mid = (lo + hi) >> 1; if (sm.key[mid] > l) lo = mid + 1; else hi = mid; }
                    sm.tab1[l] = (uint8_t)lo; sm.tab2[l] = (uint8_t)lo;   // thresholds above l (descending order)
                }
            }
            const FamTotals tot = waits ? zone_family<true>(sm, c, tile0, n_fam, n_tiles, chunk_id, tr.len_end, left_mask, left_lists, out)
                                        : zone_family<false>(sm, c, tile0, n_fam, n_tiles, chunk_id, tr.len_end, left_mask, left_lists, out);
            if (threadIdx.x == 0) {
                for (int t = 0; t < n_fam; ++t) left_count[(size_t)chunk_id * n_tiles + tile0 + t] = tot.left + (t ? 0u : tot.apart);
                if (work) {
                    atomicAdd(&work[0], (unsigned long long)(ch.len - tot.left) * npol - (unsigned long long)tot.apart * 32u);   // pairs settled zone by zone
                    atomicAdd(&work[2], (unsigned long long)(ch.len - tot.left));          // requests settled, per family
                    atomicAdd(&work[3], (unsigned long long)tot.passes);                   // sweeps over segments
                }
            }
            tile0 += n_fam;
        }
    }
}

}  // namespace

DBG_TRANSLATION_UNIT()

cudaError_t launch_pairs_zones(const TraceDev& tr, const GroupConst* gc, const ClassConst* cc, const Prep* prep,
                               uint32_t P, const uint32_t* pol_list, uint32_t n_list, int PL, const Chunk* chunks,
                               uint32_t n_chunks, TimelineRec rec, uint64_t* acc, uint64_t* hist_ttft,
                               uint64_t* hist_tbt, uint32_t* left_mask, uint32_t* left_count, uint32_t* left_lists,
                               uint32_t max_blocks, uint32_t* ticket, uint64_t* work, cudaStream_t st) {
    const uint32_t n_tiles = (n_list + PL - 1) / PL;
    const uint32_t n_fams = (n_tiles + kFamTiles - 1) / kFamTiles;
    if ((uint64_t)n_chunks * n_tiles > 0x7FFFFFFFull) return cudaErrorInvalidConfiguration;
    cudaError_t e = cudaFuncSetAttribute(k_pairs_zones, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)sizeof(ZoneSmem));
    if (e) return e;
    const uint32_t blocks = (uint32_t)std::min<uint64_t>((uint64_t)n_chunks * n_fams, (uint64_t)max_blocks * kZBlocksPerSm);
    return launch_after(k_pairs_zones, dim3(blocks), kZThreads, sizeof(ZoneSmem), st, tr, gc, cc, prep, P,
                        pol_list, n_list, PL, chunks, n_chunks, n_tiles, rec, (unsigned long long*)acc,
                        (unsigned long long*)hist_ttft, (unsigned long long*)hist_tbt, left_mask, left_count, left_lists,
                        ticket, (unsigned long long*)work);
}

}  // namespace disco
