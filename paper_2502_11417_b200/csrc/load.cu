// Trace ingestion on the device: tick conversion and validation, per-group prompt-length histogram,
// internal request order (by group, then by prompt length), radix sort of the server-TTFT ticks (the empirical F of
// Algorithm 1), cumulative input-token mass (Eq. 3) and the quantile knots of F.
#include "load.cuh"

#include <algorithm>
#include <mutex>

namespace disco {

namespace {

constexpr int kIngestThreads = 1024;

__global__ void k_ingest(uint32_t n, const int32_t* __restrict__ prompt, const int32_t* __restrict__ outlen,
                         const float* __restrict__ ttft, const uint8_t* __restrict__ sp,
                         const uint8_t* __restrict__ dp, uint32_t ns, uint32_t nd, uint64_t* __restrict__ keys,
                         uint32_t* __restrict__ cnt, unsigned long long* __restrict__ grp_sum_n,
                         uint32_t* __restrict__ grp_n, uint32_t* __restrict__ max_n, int32_t* __restrict__ err,
                         uint16_t* __restrict__ l_out, uint16_t* __restrict__ n_out,
                         uint32_t* __restrict__ counts0, uint32_t per_block0,
                         uint32_t blocks0, int hist_groups) {
    // l_out, n_out: packed copies of the lengths in the caller's order, for the scatter into the internal order;
    // counts0: first radix digit counted per sort block (small traces; large ones use the histogram kernel)
    __shared__ unsigned long long s_sum[kMaxGroups];
    __shared__ uint32_t s_cnt[kMaxGroups];
    __shared__ uint32_t s_max, s_max_ticks;         // longest output, largest TTFT ticks (max_n[0], max_n[1])
    // hist_groups: groups whose length histograms this block keeps in shared memory (all of them, or none when they
    // do not fit: then the counts go to global memory one by one)
    extern __shared__ uint32_t s_len[];              // [hist_groups][kMaxPrompt + 1]
    const int G = (int)(ns * nd);
    const bool one = G == 1;
    for (int g = threadIdx.x; g < G; g += blockDim.x) { s_sum[g] = 0; s_cnt[g] = 0; }
    for (int i = threadIdx.x; i < hist_groups * (kMaxPrompt + 1); i += blockDim.x) s_len[i] = 0;
    if (threadIdx.x == 0) { s_max = 0; s_max_ticks = 0; }
    __syncthreads();
    const uint32_t stride = gridDim.x * blockDim.x;
    for (uint32_t i0 = blockIdx.x * blockDim.x; i0 < n; i0 += stride) {       // whole warps iterate together
        const uint32_t i = i0 + threadIdx.x;
        const bool in = i < n;
        const int32_t l = in ? prompt[i] : 1, o = in ? outlen[i] : 1;
        const float t = in ? ttft[i] : 1.0f;
        const uint32_t s = (in && sp) ? sp[i] : 0u, d = (in && dp) ? dp[i] : 0u;
        int bad = 0;
        if (l < 1 || l > kMaxPrompt) bad = 1;
        else if (o < 1 || o > kMaxOutput) bad = 2;
        else if (!(t > 0.0f) || !(t <= 2000.0f)) bad = 3;      // NaN fails both comparisons
        else if (s >= ns || d >= nd) bad = 4;
        const bool ok = in && !bad;
        if (in && bad) {
            if (atomicCAS(&err[0], 0, bad) == 0) err[1] = (int32_t)i;
            keys[i] = 0;
        }
        // ticks = nearest integer (ties to even) of the fp64 product, as a host llrint would give
        const long long S = __double2ll_rn(__dmul_rn((double)t, 1e6));
        const uint32_t g = ok ? s * nd + d : 0u;
        if (ok && DBG_OK(g, G, DBG_K_INGEST, DBG_GROUP) && DBG_OK(l, kMaxPrompt + 1, DBG_K_INGEST, DBG_TABLE)) {
            keys[i] = ((uint64_t)g << 32) | (uint32_t)S;
            if (hist_groups) atomicAdd(&s_len[g * (kMaxPrompt + 1) + l], 1u); else atomicAdd(&cnt[g * (kMaxPrompt + 1) + l], 1u);
            l_out[i] = (uint16_t)l; n_out[i] = (uint16_t)o;
            if (counts0 && DBG_OK(i / per_block0, blocks0, DBG_K_INGEST, DBG_COUNTER))
                atomicAdd(&counts0[((uint32_t)S & 255u) * blocks0 + i / per_block0], 1u);
        }
        if (one) {                                             // one group: sums by warp reduction
            const uint32_t so = __reduce_add_sync(0xFFFFFFFFu, ok ? (uint32_t)o : 0u);
            const uint32_t mo = __reduce_max_sync(0xFFFFFFFFu, ok ? (uint32_t)o : 0u);
            const uint32_t co = __popc(__ballot_sync(0xFFFFFFFFu, ok));
            const uint32_t mt = __reduce_max_sync(0xFFFFFFFFu, ok ? (uint32_t)S : 0u);
            if ((threadIdx.x & 31) == 0 && co) {
                atomicAdd(&s_sum[0], (unsigned long long)so); atomicAdd(&s_cnt[0], co); atomicMax(&s_max, mo);
                atomicMax(&s_max_ticks, mt);
            }
        } else {
            // several groups: the lanes of each group present in the warp add up among themselves, one lane adds
            const uint32_t mo = __reduce_max_sync(0xFFFFFFFFu, ok ? (uint32_t)o : 0u);
            const uint32_t mt = __reduce_max_sync(0xFFFFFFFFu, ok ? (uint32_t)S : 0u);
            uint32_t rest = __ballot_sync(0xFFFFFFFFu, ok);
            const int lane = threadIdx.x & 31;
            if (lane == 0 && rest) { atomicMax(&s_max, mo); atomicMax(&s_max_ticks, mt); }
            while (rest) {
                const int first = __ffs(rest) - 1;
                const uint32_t g1 = __shfl_sync(0xFFFFFFFFu, g, first);
                const bool mine = ok && g == g1;
                const uint32_t same = __ballot_sync(0xFFFFFFFFu, mine);
                const uint32_t so = __reduce_add_sync(0xFFFFFFFFu, mine ? (uint32_t)o : 0u);
                if (lane == first) { atomicAdd(&s_sum[g1], (unsigned long long)so); atomicAdd(&s_cnt[g1], (uint32_t)__popc(same)); }
                rest &= ~same;
            }
        }
    }
    __syncthreads();
    for (int g = threadIdx.x; g < G; g += blockDim.x)
        if (s_cnt[g]) { atomicAdd(&grp_sum_n[g], s_sum[g]); atomicAdd(&grp_n[g], s_cnt[g]); }
    for (int i = threadIdx.x; i < hist_groups * (kMaxPrompt + 1); i += blockDim.x) if (s_len[i]) atomicAdd(&cnt[i], s_len[i]);
    if (threadIdx.x == 0 && s_max) { atomicMax(max_n, s_max); atomicMax(max_n + 1, s_max_ticks); }
}

// Inclusive prefix sum over the threads of a block (blockDim.x a multiple of 32, at most 1024): shuffles inside
// the warps, one pass over the warp totals, two barriers.  `wtot` is shared scratch of 32 entries; every thread
// of the block must call.  Returns this thread's inclusive sum; *total receives the block's sum.
template <class T>
__device__ __forceinline__ T block_inclusive_scan(T v, T* wtot, T* total) {
    const int lane = threadIdx.x & 31, w = threadIdx.x >> 5, nw = blockDim.x >> 5;
#pragma unroll
    for (int off = 1; off < 32; off <<= 1) {
        const T up = __shfl_up_sync(0xFFFFFFFFu, v, off);
        if (lane >= off) v += up;
    }
    if (lane == 31) wtot[w] = v;
    __syncthreads();
    if (w == 0) {
        T t = lane < nw ? wtot[lane] : T(0);
#pragma unroll
        for (int off = 1; off < 32; off <<= 1) {
            const T up = __shfl_up_sync(0xFFFFFFFFu, t, off);
            if (lane >= off) t += up;
        }
        wtot[lane] = t;                                   // inclusive over the warps
    }
    __syncthreads();
    if (total) *total = wtot[nw - 1];
    return w ? v + wtot[w - 1] : v;
}

// ---- one stable LSD radix pass over 64-bit keys (8-bit digit), optional 32-bit payload -------------------
constexpr int kRadixThreads = 256;
constexpr int kRadixWarps = kRadixThreads / 32;

__global__ void k_radix_hist(const uint64_t* __restrict__ keys, uint32_t n, uint32_t per_block, int shift,
                             uint32_t* __restrict__ counts /* [256][gridDim.x] */,
                             const uint32_t* __restrict__ max_key = nullptr, uint32_t skip_below = 0) {
    // max_key, skip_below: the pass is not needed (every key has this digit zero, the order is final) when the
    // largest key is below skip_below; the kernels of such a pass return at once
    __shared__ uint32_t h[256];
    h[threadIdx.x] = 0;
    grid_dependency_wait();
    if (max_key && *max_key < skip_below) return;
    __syncthreads();
    const uint32_t lo = min(n, blockIdx.x * per_block), hi = min(n, lo + per_block);
    for (uint32_t i = lo + threadIdx.x; i < hi; i += kRadixThreads)
        atomicAdd(&h[(uint32_t)(keys[i] >> shift) & 255u], 1u);
    __syncthreads();
    counts[threadIdx.x * gridDim.x + blockIdx.x] = h[threadIdx.x];
}

// One block per digit: exclusive scan of the digit's per-block counts, in place, and the digit's total.
__global__ void k_radix_rowscan(uint32_t* __restrict__ counts /* [256][blocks] */, uint32_t blocks,
                                uint32_t* __restrict__ totals /* [256] */,
                                const uint32_t* __restrict__ max_key = nullptr, uint32_t skip_below = 0) {
    __shared__ uint32_t wtot[32];
    grid_dependency_wait();
    if (max_key && *max_key < skip_below) return;
    uint32_t* row = counts + (size_t)blockIdx.x * blocks;
    const uint32_t per = (blocks + 127u) / 128u;
    const uint32_t lo = min(blocks, threadIdx.x * per), hi = min(blocks, lo + per);
    uint32_t s = 0;
    for (uint32_t i = lo; i < hi; ++i) s += row[i];
    uint32_t total;
    uint32_t run = block_inclusive_scan(s, wtot, &total) - s;
    for (uint32_t i = lo; i < hi; ++i) { const uint32_t c = row[i]; row[i] = run; run += c; }
    if (threadIdx.x == 0) totals[blockIdx.x] = total;
}

__global__ void k_radix_scatter(const uint64_t* __restrict__ keys_in, uint64_t* __restrict__ keys_out,
                                const uint32_t* __restrict__ pay_in, uint32_t* __restrict__ pay_out, uint32_t n,
                                uint32_t per_block, int shift, const uint32_t* __restrict__ offsets,
                                const uint32_t* __restrict__ totals, uint32_t* __restrict__ counts_next = nullptr,
                                int32_t* __restrict__ low_out = nullptr,
                                const uint32_t* __restrict__ max_key = nullptr, uint32_t skip_below = 0,
                                int32_t* __restrict__ low_out_if_last = nullptr, uint32_t last_below = 0) {
    // low_out: the last pass writes the low words (the sorted ticks) instead of the keys.  low_out_if_last: this
    // pass writes them as well when the largest key is below last_below (the later passes then skip themselves).
    __shared__ uint32_t run[256];                 // next output slot of each digit for this block
    __shared__ uint32_t wcnt[kRadixWarps][256];   // keys of each digit per warp in the current slab
    const int w = threadIdx.x >> 5, lane = threadIdx.x & 31;
    grid_dependency_wait();
    if (max_key && *max_key < skip_below) return;
    if (low_out_if_last && *max_key >= last_below) low_out_if_last = nullptr;
    {
        // offsets[d][b]: keys of digit d in earlier blocks (k_radix_rowscan); totals[d]: keys of digit d.
        // This block's first slot for digit d = keys of smaller digits + keys of d in earlier blocks.
        uint32_t* wtot = wcnt[0];                                    // scratch of the scan (32 words)
        const uint32_t total = totals[threadIdx.x], before = offsets[threadIdx.x * gridDim.x + blockIdx.x];
        const uint32_t incl = block_inclusive_scan(total, wtot, (uint32_t*)nullptr);
        run[threadIdx.x] = incl - total + before;
        __syncthreads();
    }
    const uint32_t lo = min(n, blockIdx.x * per_block), hi = min(n, lo + per_block);
    constexpr int kPer = 4;                                   // keys per thread and tile
    constexpr uint32_t kTile = kRadixThreads * kPer;          // a warp owns 128 consecutive keys of a tile
    for (uint32_t base = lo; base < hi; base += kTile) {
        for (int k = 0; k < kRadixWarps; ++k) wcnt[k][threadIdx.x] = 0;
        uint64_t key[kPer];
        uint32_t dig[kPer], peers[kPer];
        bool live[kPer];
#pragma unroll
        for (int j = 0; j < kPer; ++j) {
            const uint32_t i = base + w * (32 * kPer) + j * 32 + lane;
            live[j] = i < hi;
            key[j] = live[j] ? keys_in[i] : 0;
            dig[j] = (uint32_t)(key[j] >> shift) & 255u;
            // lanes holding the same digit, from eight ballots over the digit's bits
            uint32_t m = __ballot_sync(0xFFFFFFFFu, live[j]);
#pragma unroll
            for (int b = 0; b < 8; ++b) {
                const uint32_t bal = __ballot_sync(0xFFFFFFFFu, (dig[j] >> b) & 1u);
                m &= ((dig[j] >> b) & 1u) ? bal : ~bal;
            }
            peers[j] = m;
        }
        __syncthreads();
        // keys of each digit in each warp (a warp's row is its own: plain adds, rounds in order)
#pragma unroll
        for (int j = 0; j < kPer; ++j) {
            if (live[j] && (peers[j] & ((1u << lane) - 1u)) == 0) wcnt[w][dig[j]] += __popc(peers[j]);
            __syncwarp();
        }
        __syncthreads();
        {   // turn the counts into each warp's first slot per digit; advance the block's running slots
            uint32_t at = run[threadIdx.x];
            for (int k = 0; k < kRadixWarps; ++k) { const uint32_t c = wcnt[k][threadIdx.x]; wcnt[k][threadIdx.x] = at; at += c; }
            run[threadIdx.x] = at;
        }
        __syncthreads();
#pragma unroll
        for (int j = 0; j < kPer; ++j) {
            uint32_t nxt = 0xFFFFFFFFu;                          // next pass's counter for this key (none: dead lane)
            if (live[j]) {
                const uint32_t rank = __popc(peers[j] & ((1u << lane) - 1u));
                const uint32_t pos = wcnt[w][dig[j]] + rank;
                if (DBG_OK(pos, n, DBG_K_RADIX, DBG_ELEMENT)) {
                    if (low_out) low_out[pos] = (int32_t)(uint32_t)key[j]; else keys_out[pos] = key[j];
                    if (low_out_if_last) low_out_if_last[pos] = (int32_t)(uint32_t)key[j];
                    if (pay_out) {
                        const uint32_t i = base + w * (32 * kPer) + j * 32 + lane;
                        pay_out[pos] = pay_in ? pay_in[i] : i;
                    }
                }
                if (DBG_OK(pos / per_block, gridDim.x, DBG_K_RADIX, DBG_COUNTER))
                    nxt = ((uint32_t)(key[j] >> (shift + 8)) & 255u) * gridDim.x + pos / per_block;
            }
            __syncwarp();
            if (counts_next) {
                // lanes bound for the same counter add once: high digits take few values, and one add per key
                // would queue every key of the trace on a handful of addresses
                const uint32_t same = __match_any_sync(0xFFFFFFFFu, nxt);
                if (live[j] && (same & ((1u << lane) - 1u)) == 0) atomicAdd(&counts_next[nxt], (uint32_t)__popc(same));
            }
            if (live[j] && (peers[j] & ((1u << lane) - 1u)) == 0) wcnt[w][dig[j]] += __popc(peers[j]);
            __syncwarp();
        }
        __syncthreads();
    }
}

// Where the requests of each (group, prompt length) start in the internal order: the groups one after another,
// inside a group the prompt lengths ascending.  One block of 1024 threads per group.
__global__ void __launch_bounds__(1024)
k_length_cursors(const uint32_t* __restrict__ cnt, const uint32_t* __restrict__ ng, uint32_t* __restrict__ cursor) {
    constexpr int NT = 1024, L = kMaxPrompt + 1;
    __shared__ uint32_t wc[32];
    const int g = blockIdx.x;
    uint32_t base = 0;
    for (int h = 0; h < g; ++h) base += ng[h];
    const int per = (L + NT - 1) / NT;
    const int lo = min(L, (int)threadIdx.x * per), hi = min(L, lo + per);
    uint32_t k = 0;
    for (int l = lo; l < hi; ++l) k += cnt[(size_t)g * L + l];
    uint32_t run = base + block_inclusive_scan(k, wc, (uint32_t*)nullptr) - k;
    for (int l = lo; l < hi; ++l) { cursor[(size_t)g * L + l] = run; run += cnt[(size_t)g * L + l]; }
}

// The internal request order: each request takes the next free place of its (group, prompt length).  Requests of
// one group and length keep no particular order among themselves (nothing downstream depends on it: orig and inv
// map between the two orders).  The lanes of a warp that share a bucket take their places with one add.  A
// request goes to its place as one 16-byte record (ticks, lengths, caller's index): one scattered store instead
// of four; k_unpack_requests then writes the arrays side by side.
__global__ void k_scatter_by_length(uint32_t n, int G, const uint64_t* __restrict__ keys,
                                    const uint16_t* __restrict__ prompt, const uint16_t* __restrict__ outlen,
                                    const int32_t* __restrict__ err, uint32_t* __restrict__ cursor,
                                    uint4* __restrict__ placed, uint32_t* __restrict__ inv) {
    if (err[0] != 0) return;                          // a rejected trace: its lengths were not all written
    const int lane = threadIdx.x & 31;
    const uint32_t stride = gridDim.x * blockDim.x;
    for (uint32_t i0 = blockIdx.x * blockDim.x; i0 < n; i0 += stride) {       // whole warps iterate together
        const uint32_t i = i0 + threadIdx.x;
        bool in = i < n;
        const uint64_t key = in ? keys[i] : 0ull;
        const uint32_t g = (uint32_t)(key >> 32), len = in ? prompt[i] : 0u;
        in = in && DBG_OK(g, G, DBG_K_GATHER, DBG_GROUP) && DBG_OK(len, kMaxPrompt + 1, DBG_K_GATHER, DBG_TABLE);
        const uint32_t live = __ballot_sync(0xFFFFFFFFu, in);
        if (!in) continue;
        const uint32_t bucket = g * (uint32_t)(kMaxPrompt + 1) + len;
        const uint32_t peers = __match_any_sync(live, bucket);
        const int leader = __ffs(peers) - 1;
        uint32_t at = 0;
        if (lane == leader) at = atomicAdd(&cursor[bucket], (uint32_t)__popc(peers));
        at = __shfl_sync(peers, at, leader) + (uint32_t)__popc(peers & ((1u << lane) - 1u));
        if (!DBG_OK(at, n, DBG_K_GATHER, DBG_REQUEST)) continue;
        placed[at] = make_uint4((uint32_t)key, len | ((uint32_t)outlen[i] << 16), i, 0u);
        inv[i] = at;
    }
}

// The same for traces whose length histograms fit in shared memory (up to six groups).  A block takes slices of
// kSliceRequests requests: it counts the slice's requests per bucket in shared memory, reserves each bucket's places
// with ONE add to the global cursor, and hands the places out from shared memory.  A popular bucket's cursor then
// sees one add per slice instead of one per warp (adds to one address are served one after another).
constexpr uint32_t kSliceRequests = 16384;
constexpr int kSliceThreads = 1024;

__global__ void __launch_bounds__(kSliceThreads)
k_scatter_by_length_slices(uint32_t n, int G, const uint64_t* __restrict__ keys,
                           const uint16_t* __restrict__ prompt, const uint16_t* __restrict__ outlen,
                           const int32_t* __restrict__ err, uint32_t* __restrict__ cursor,
                           uint4* __restrict__ placed, uint32_t* __restrict__ inv) {
    extern __shared__ uint32_t s_at[];               // [G][kMaxPrompt + 1]: counts, then next free places
    if (err[0] != 0) return;                         // a rejected trace: its lengths were not all written
    const uint32_t buckets = (uint32_t)G * (uint32_t)(kMaxPrompt + 1);
    for (uint32_t lo = blockIdx.x * kSliceRequests; lo < n; lo += gridDim.x * kSliceRequests) {
        const uint32_t hi = min(n, lo + kSliceRequests);
        for (uint32_t b = threadIdx.x; b < buckets; b += kSliceThreads) s_at[b] = 0;
        __syncthreads();
        for (uint32_t i = lo + threadIdx.x; i < hi; i += kSliceThreads) {
            const uint32_t g = (uint32_t)(keys[i] >> 32), len = prompt[i];
            if (DBG_OK(g, G, DBG_K_GATHER, DBG_GROUP) && DBG_OK(len, kMaxPrompt + 1, DBG_K_GATHER, DBG_TABLE))
                atomicAdd(&s_at[g * (uint32_t)(kMaxPrompt + 1) + len], 1u);
        }
        __syncthreads();
        for (uint32_t b = threadIdx.x; b < buckets; b += kSliceThreads) {
            const uint32_t c = s_at[b];
            if (c) s_at[b] = atomicAdd(&cursor[b], c);
        }
        __syncthreads();
        for (uint32_t i = lo + threadIdx.x; i < hi; i += kSliceThreads) {
            const uint64_t key = keys[i];
            const uint32_t g = (uint32_t)(key >> 32), len = prompt[i];
            if (!DBG_OK(g, G, DBG_K_GATHER, DBG_GROUP) || !DBG_OK(len, kMaxPrompt + 1, DBG_K_GATHER, DBG_TABLE)) continue;
            const uint32_t at = atomicAdd(&s_at[g * (uint32_t)(kMaxPrompt + 1) + len], 1u);
            if (!DBG_OK(at, n, DBG_K_GATHER, DBG_REQUEST)) continue;
            placed[at] = make_uint4((uint32_t)key, len | ((uint32_t)outlen[i] << 16), i, 0u);
            inv[i] = at;
        }
        __syncthreads();
    }
}

__global__ void k_unpack_requests(uint32_t n, const uint4* __restrict__ placed, const int32_t* __restrict__ err,
                                  int32_t* __restrict__ S, uint16_t* __restrict__ l, uint16_t* __restrict__ nout,
                                  uint32_t* __restrict__ orig) {
    if (err[0] != 0) return;
    for (uint32_t k = blockIdx.x * blockDim.x + threadIdx.x; k < n; k += gridDim.x * blockDim.x) {
        const uint4 r = placed[k];
        S[k] = (int32_t)r.x;
        l[k] = (uint16_t)(r.y & 0xFFFFu);
        nout[k] = (uint16_t)(r.y >> 16);
        orig[k] = r.z;
    }
}

__global__ void k_low_words(uint32_t n, const uint64_t* __restrict__ keys, int32_t* __restrict__ out) {
    for (uint32_t k = blockIdx.x * blockDim.x + threadIdx.x; k < n; k += gridDim.x * blockDim.x)
        out[k] = (int32_t)(uint32_t)keys[k];
}

// One block of 1024 threads per group: cumulative input-token mass cum[L] = sum_{l<L} l*cnt[l], L = 0..4097, and N_g.
__device__ __forceinline__ void group_mass(const uint32_t* __restrict__ cnt, int64_t* __restrict__ cum,
                                           uint32_t* __restrict__ ng) {
    constexpr int NT = 1024, L = kMaxPrompt + 1;      // 4097 lengths
    __shared__ unsigned long long wm[32];
    __shared__ uint32_t wc[32];
    const int g = blockIdx.x;
    const uint32_t* c = cnt + (size_t)g * L;
    int64_t* out = cum + (size_t)g * (L + 1);
    const int per = (L + NT - 1) / NT;                 // 5
    const int lo = min(L, (int)threadIdx.x * per), hi = min(L, lo + per);
    unsigned long long m = 0; uint32_t k = 0;
    for (int l = lo; l < hi; ++l) { m += (unsigned long long)l * c[l]; k += c[l]; }
    unsigned long long m_total; uint32_t k_total;
    unsigned long long run = block_inclusive_scan(m, wm, &m_total) - m;
    block_inclusive_scan(k, wc, &k_total);
    for (int l = lo; l < hi; ++l) { out[l] = (int64_t)run; run += (unsigned long long)l * c[l]; }
    if (threadIdx.x == 0) { out[L] = (int64_t)m_total; ng[g] = k_total; }
}

// Group offsets in the partitioned order, the 257 knots K_g[k] = sorted_g[(k (N_g - 1)) / 256] and the few
// numbers the host reads back.  One block per group (ng: the group sizes counted at ingestion).
__device__ __forceinline__ void group_knots(int G, const uint32_t* __restrict__ ng, const int32_t* __restrict__ sorted,
                                            uint32_t* __restrict__ grp_off, int32_t* __restrict__ knots,
                                            const int32_t* __restrict__ err, const uint32_t* __restrict__ max_n,
                                            const unsigned long long* __restrict__ grp_sum_n,
                                            unsigned long long* __restrict__ fin_totals,
                                            LoadReadback* __restrict__ rb) {
    __shared__ uint32_t off[kMaxGroups + 1];
    const int g = blockIdx.x;
    if (threadIdx.x == 0) {
        uint32_t r = 0;
        for (int k = 0; k < G; ++k) { off[k] = r; r += ng[k]; }
        off[G] = r;
    }
    __syncthreads();
    const uint32_t N = off[g + 1] - off[g];
    for (int k = threadIdx.x; k < kNKnots; k += blockDim.x) {
        const uint32_t at = N ? (uint32_t)(((uint64_t)k * (N - 1)) / 256u) : 0u;
        knots[g * kNKnots + k] = (N && DBG_OK(at, N, DBG_K_TABLES, DBG_ELEMENT)) ? sorted[off[g] + at] : 0;
    }
    if (threadIdx.x == 0) {
        rb->knot_max[g] = N ? sorted[off[g] + N - 1] : 0;
        rb->ng[g] = N; rb->grp_sum_n[g] = grp_sum_n[g];
        fin_totals[g] = grp_sum_n[g]; fin_totals[G + g] = N;      // what the final reductions' totals refer to
        if (g == 0) {
            for (int k = 0; k <= G; ++k) { grp_off[k] = off[k]; rb->grp_off[k] = off[k]; }
            for (int k = 0; k < 4; ++k) rb->err[k] = err[k];
            rb->max_n = *max_n;
        }
    }
}

// The group tables in one launch: one block of 1024 threads per group.
__global__ void __launch_bounds__(1024)
k_group_tables(int G, const uint32_t* __restrict__ cnt, int64_t* __restrict__ cum, uint32_t* __restrict__ ng_exact,
               const uint32_t* __restrict__ ng, const int32_t* __restrict__ sorted, uint32_t* __restrict__ grp_off,
               int32_t* __restrict__ knots, const int32_t* __restrict__ err, const uint32_t* __restrict__ max_n,
               const unsigned long long* __restrict__ grp_sum_n, unsigned long long* __restrict__ fin_totals,
               LoadReadback* __restrict__ rb) {
    grid_dependency_wait();
    group_knots(G, ng, sorted, grp_off, knots, err, max_n, grp_sum_n, fin_totals, rb);
    group_mass(cnt, cum, ng_exact);
}

// The same tables from a length histogram and a sorted sample given by the caller (a whole trace's, of which
// the context holds a shard): one block of 1024 threads per group.
__global__ void __launch_bounds__(1024)
k_tables_imported(const uint32_t* __restrict__ cnt, int64_t* __restrict__ cum, uint32_t* __restrict__ ng_exact,
                  const int32_t* __restrict__ F_sorted, const uint32_t* __restrict__ F_off, int32_t* __restrict__ knots) {
    const int g = blockIdx.x;
    const uint32_t off = F_off[g], N = F_off[g + 1] - off;
    for (int k = threadIdx.x; k < kNKnots; k += blockDim.x) {
        const uint32_t at = N ? (uint32_t)(((uint64_t)k * (N - 1)) / 256u) : 0u;
        knots[g * kNKnots + k] = (N && DBG_OK(at, N, DBG_K_TABLES, DBG_ELEMENT)) ? F_sorted[off + at] : 0;
    }
    group_mass(cnt, cum, ng_exact);
}

int grid_for(uint32_t n, int threads, int sms) {
    long long b = ((long long)n + threads - 1) / threads;
    if (b < 1) b = 1;
    if (b > (long long)sms * 16) b = (long long)sms * 16;
    return (int)b;
}

cudaError_t radix_pass(const uint64_t* kin, uint64_t* kout, const uint32_t* pin, uint32_t* pout, uint32_t n,
                       int shift, uint32_t* counts, cudaStream_t st) {
    uint32_t blocks = (n + 1023u) / 1024u;
    if (blocks < 1) blocks = 1;
    if (blocks > kRadixMaxBlocks) blocks = kRadixMaxBlocks;
    uint32_t per_block = (n + blocks - 1) / blocks;
    per_block = (per_block + kRadixThreads - 1) / kRadixThreads * kRadixThreads;
    uint32_t* totals = counts + (size_t)256u * blocks;       // the caller's buffer has room for these 256 words
    k_radix_hist<<<blocks, kRadixThreads, 0, st>>>(kin, n, per_block, shift, counts);
    k_radix_rowscan<<<256, 128, 0, st>>>(counts, blocks, totals);
    k_radix_scatter<<<blocks, kRadixThreads, 0, st>>>(kin, kout, pin, pout, n, per_block, shift, counts, totals);
    return cudaGetLastError();
}

}  // namespace

DBG_TRANSLATION_UNIT()

uint32_t load_kernel_launches(uint32_t n, int G) {
    if (n == 0) return 1;
    // ingest, cursors, scatter by length, unpack; (row scan, scatter) x 4, two histograms; group tables
    if (G == 1 && n <= (1u << 20)) return 4 + 2 * 4 + 2 + 1;
    const uint32_t passes = G > 1 ? 5 : 4;                  // radix passes over (group, ticks)
    return 4 + 3 * passes + 1 + 1;                          // ..., passes, low words, group tables
}

cudaError_t run_load(const LoadArgs& a, cudaStream_t st) {
    const uint32_t n = a.n;
    const int G = (int)(a.ns * a.nd);
    cudaError_t e;
    // radix geometry (as in radix_pass)
    uint32_t blocks = (n + 1023u) / 1024u;
    if (blocks < 1) blocks = 1;
    if (blocks > kRadixMaxBlocks) blocks = kRadixMaxBlocks;
    uint32_t per_block = (n + blocks - 1) / blocks;
    per_block = (per_block + kRadixThreads - 1) / kRadixThreads * kRadixThreads;
    const bool small = G == 1 && n <= (1u << 20);      // fused histograms pay off while launches dominate
    // everything that must start at zero lies in one block: cnt, grp_sum_n, grp_n, max_n, err, counts A
    // (zero_bytes covers the tables; the per-pass digit counters of the small path follow them)
    if ((e = cudaMemsetAsync(a.zero_block, 0, a.zero_bytes + (small ? (size_t)2 * 256u * blocks * 4u : 0u), st))) return e;
    if (n) {
        uint32_t* counts_a = a.radix_counts;                                   // small path: pass p uses slice p
        uint32_t* counts_b = a.radix_counts + (size_t)4 * 256u * kRadixMaxBlocks;  // large path: one scanned buffer
        // block-private length histograms while they fit two blocks to a multiprocessor (up to six groups)
        const int hist_groups = (size_t)G * (kMaxPrompt + 1) * 4 <= 100 * 1024 ? G : 0;
        const size_t hist_bytes = (size_t)hist_groups * (kMaxPrompt + 1) * 4;
        if ((e = cudaFuncSetAttribute(k_ingest, cudaFuncAttributeMaxDynamicSharedMemorySize, 100 * 1024))) return e;
        k_ingest<<<std::min(grid_for(n, 4 * kIngestThreads, a.sms), 2 * a.sms), kIngestThreads, hist_bytes, st>>>(
            n, a.prompt, a.outlen, a.ttft, a.sp, a.dp, a.ns, a.nd, a.keys_a, a.cnt,
            (unsigned long long*)a.grp_sum_n, a.ng, a.max_n, a.err,
            a.l_tmp, a.n_tmp, small ? counts_a : nullptr, per_block, blocks, hist_groups);
        // internal request order: by group, then by prompt length
        k_length_cursors<<<G, 1024, 0, st>>>(a.cnt, a.ng, a.cursors);
        const size_t cursor_bytes = (size_t)G * (kMaxPrompt + 1) * 4;
        if (cursor_bytes <= 100 * 1024) {
            if ((e = cudaFuncSetAttribute(k_scatter_by_length_slices, cudaFuncAttributeMaxDynamicSharedMemorySize, 100 * 1024))) return e;
            const uint32_t slices = (n + kSliceRequests - 1) / kSliceRequests;
            k_scatter_by_length_slices<<<std::min<uint32_t>(slices, 2u * (uint32_t)a.sms), kSliceThreads, cursor_bytes, st>>>(
                n, G, a.keys_a, a.l_tmp, a.n_tmp, a.err, a.cursors, a.placed, a.inv);
        } else {
            k_scatter_by_length<<<grid_for(n, 256, a.sms), 256, 0, st>>>(n, G, a.keys_a, a.l_tmp, a.n_tmp, a.err, a.cursors,
                                                                         a.placed, a.inv);
        }
        k_unpack_requests<<<grid_for(n, 256, a.sms), 256, 0, st>>>(n, a.placed, a.err, a.S, a.l, a.nout, a.orig);
        // sort (group, ticks): four byte passes over the ticks, one over the group id
        uint64_t *src = a.keys_a, *dst = a.keys_b;
        const int passes = G > 1 ? 5 : 4;
        if (small) {
            uint32_t* totals = a.radix_counts + (size_t)5 * 256u * kRadixMaxBlocks;
            for (int p = 0; p < passes; ++p) {
                // The first scatter also counts the second pass's digits (the low bytes of the ticks are spread
                // evenly, so its adds meet little contention).  High bytes take few values: those passes count
                // with the block-private histogram kernel instead.
                const bool last = p == passes - 1, fused_next = p == 0;
                uint32_t* cur = a.radix_counts + (size_t)p * 256u * blocks;
                // Ticks below 2^24 (16.7 s) leave the fourth byte zero: the third pass then also writes the sorted
                // ticks and the kernels of the fourth return at once (a.max_n[1]: the largest tick, from ingestion).
                const uint32_t* max_key = a.max_n + 1;
                const uint32_t skip_below = p == 3 ? (1u << 24) : 0u;
                if (p >= 2 && (e = launch_after(k_radix_hist, blocks, kRadixThreads, 0, st, (const uint64_t*)src, n, per_block,
                                                8 * p, cur, max_key, skip_below))) return e;
                if ((e = launch_after(k_radix_rowscan, 256, 128, 0, st, cur, blocks, totals, max_key, skip_below))) return e;
                if ((e = launch_after(k_radix_scatter, blocks, kRadixThreads, 0, st, src, dst, nullptr, nullptr, n, per_block,
                                      8 * p, cur, totals, fused_next ? cur + 256u * blocks : nullptr,
                                      last ? a.sorted : nullptr, max_key, skip_below,
                                      p == 2 ? a.sorted : nullptr, 1u << 24))) return e;
                uint64_t* t = src; src = dst; dst = t;
            }
        } else {
            for (int p = 0; p < passes; ++p) {
                if ((e = radix_pass(src, dst, nullptr, nullptr, n, 8 * p, counts_b, st))) return e;
                uint64_t* t = src; src = dst; dst = t;
            }
            k_low_words<<<grid_for(n, 256, a.sms), 256, 0, st>>>(n, src, a.sorted);
        }
    }
    if ((e = launch_after(k_group_tables, G, 1024, 0, st, G, a.cnt, a.cum_mass, a.ng_exact, a.ng, a.sorted, a.grp_off,
                          a.knots, a.err, a.max_n, (const unsigned long long*)a.grp_sum_n,
                          (unsigned long long*)a.fin_totals, a.readback))) return e;
    return cudaGetLastError();
}

cudaError_t launch_tables_imported(int G, const uint32_t* cnt, int64_t* cum_mass, uint32_t* ng_exact,
                                   const int32_t* F_sorted, const uint32_t* F_off, int32_t* knots, cudaStream_t st) {
    k_tables_imported<<<G, 1024, 0, st>>>(cnt, cum_mass, ng_exact, F_sorted, F_off, knots);
    return cudaGetLastError();
}

namespace {
// Sort keys (group << 32 | ticks) for ticks stored group after group; a negative tick sets the error word.
__global__ void k_keys_of_grouped_ticks(uint32_t total, const int32_t* __restrict__ ticks, const uint32_t* __restrict__ off,
                                        int G, uint64_t* __restrict__ keys, int32_t* __restrict__ err) {
    for (uint32_t i = blockIdx.x * blockDim.x + threadIdx.x; i < total; i += gridDim.x * blockDim.x) {
        int g = 0;
        while (g + 1 < G && i >= off[g + 1]) ++g;
        const int32_t t = ticks[i];
        if (t < 0 && atomicCAS(&err[0], 0, 3) == 0) err[1] = (int32_t)i;
        keys[i] = ((uint64_t)(uint32_t)g << 32) | (uint32_t)max(t, 0);
    }
}
}  // namespace

cudaError_t sort_grouped_ticks(const int32_t* ticks, const uint32_t* off, int G, uint32_t total, uint64_t* keys_a,
                               uint64_t* keys_b, uint32_t* counts, int32_t* err, int32_t* out, int sms, cudaStream_t st) {
    if (total == 0) return cudaSuccess;
    cudaError_t e;
    k_keys_of_grouped_ticks<<<grid_for(total, 256, sms), 256, 0, st>>>(total, ticks, off, G, keys_a, err);
    if ((e = cudaGetLastError())) return e;
    uint64_t *src = keys_a, *dst = keys_b;
    const int passes = G > 1 ? 5 : 4;                   // the ticks' four bytes, then the group id
    for (int p = 0; p < passes; ++p) {
        if ((e = radix_pass(src, dst, nullptr, nullptr, total, 8 * p, counts, st))) return e;
        uint64_t* t = src; src = dst; dst = t;
    }
    k_low_words<<<grid_for(total, 256, sms), 256, 0, st>>>(total, src, out);
    return cudaGetLastError();
}

}  // namespace disco


// -----------------------------------------------------------------------------------------------------
// Sorting server TTFTs without allocating.  The scratch the radix sort needs (two key buffers, the digit
// counters, an error word) lives in a fixed array inside the library image instead of in cudaMalloc'd
// memory.  Every GPU that loads the library carries these bytes until the process exits, and every call
// on a GPU uses the same bytes.
// -----------------------------------------------------------------------------------------------------
namespace disco {
namespace {

constexpr uint32_t kNoAllocMaxN = DISCO_NOALLOC_MAX_N;
constexpr size_t kNaKeysBytes = (size_t)kNoAllocMaxN * sizeof(uint64_t);
constexpr size_t kNaCountsBytes = (256u * ((kNoAllocMaxN + 1023u) / 1024u) + 256u) * sizeof(uint32_t);   // as radix_pass sizes its grid, plus the digit totals
constexpr size_t kNaErrOff = 2 * kNaKeysBytes + kNaCountsBytes;

static __device__ __align__(256) unsigned char g_noalloc_scratch[kNaErrOff + 256];

__global__ void k_ttft_keys(uint32_t n, const float* __restrict__ ttft, uint64_t* __restrict__ keys,
                            int32_t* __restrict__ err) {
    for (uint32_t i = blockIdx.x * blockDim.x + threadIdx.x; i < n; i += gridDim.x * blockDim.x) {
        const float t = ttft[i];
        if (!(t > 0.0f) || !(t <= 2000.0f)) {
            if (atomicCAS(&err[0], 0, 3) == 0) err[1] = (int32_t)i;
            keys[i] = 0;
            continue;
        }
        keys[i] = (uint64_t)(uint32_t)__double2ll_rn(__dmul_rn((double)t, 1e6));
    }
}

std::mutex g_na_mutex;
unsigned char* g_na_base[64] = {};        // device address of the scratch array, per device ordinal
int g_na_sms[64] = {};                    // multiprocessors, per device ordinal

}  // namespace
}  // namespace disco

extern "C" int disco_sort_ttft_ticks_noalloc(const float* server_ttft_s, uint32_t n, int32_t* sorted_ticks,
                                             void* stream) {
    using namespace disco;
    if (n > kNoAllocMaxN)
        return set_error(DISCO_EINVAL, "disco_sort_ttft_ticks_noalloc: n exceeds DISCO_NOALLOC_MAX_N (262144); "
                                       "use disco_load_trace for larger traces");
    if (n && (!server_ttft_s || !sorted_ticks)) return set_error(DISCO_EINVAL, "null array");
    if (n == 0) return 0;
    cudaStream_t st = (cudaStream_t)stream;
    int dev = -1;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return set_error(DISCO_ECUDA, cudaGetErrorString(e));
    if (dev < 0 || dev >= 64) return set_error(DISCO_EINVAL, "device ordinal above 63");
    unsigned char* base;
    int sms;
    {
        // In host code the array's name is only a handle; its address on the current device has to be asked for.
        std::lock_guard<std::mutex> lock(g_na_mutex);
        if (!g_na_base[dev]) {
            int count = 0;
            if ((e = cudaDeviceGetAttribute(&count, cudaDevAttrMultiProcessorCount, dev)) != cudaSuccess || count < 1)
                return set_error(DISCO_ECUDA, "cannot read the multiprocessor count of the current device");
            e = cudaGetSymbolAddress((void**)&g_na_base[dev], g_noalloc_scratch);
            if (e != cudaSuccess) { g_na_base[dev] = nullptr; return set_error(DISCO_ECUDA, cudaGetErrorString(e)); }
            g_na_sms[dev] = count;
        }
        base = g_na_base[dev];
        sms = g_na_sms[dev];
    }
    uint64_t* keys_a = (uint64_t*)base;
    uint64_t* keys_b = (uint64_t*)(base + kNaKeysBytes);
    uint32_t* counts = (uint32_t*)(base + 2 * kNaKeysBytes);
    int32_t* err = (int32_t*)(base + kNaErrOff);
    // the array still holds the previous call's data: the error word must start at zero; keys and counters
    // are fully rewritten for the first n entries before they are read
    if ((e = cudaMemsetAsync(err, 0, 16, st)) != cudaSuccess) return set_error(DISCO_ECUDA, cudaGetErrorString(e));
    // Once a kernel has been queued the shared array is in use: every way out below, failures included, first
    // waits for the stream, so that a caller who retries cannot overlap kernels still writing the array.
    auto fail_after_launch = [&](cudaError_t err_code) {
        cudaStreamSynchronize(st);
        return set_error(DISCO_ECUDA, cudaGetErrorString(err_code));
    };
    k_ttft_keys<<<grid_for(n, 256, sms), 256, 0, st>>>(n, server_ttft_s, keys_a, err);
    if ((e = cudaGetLastError()) != cudaSuccess) return fail_after_launch(e);
    uint64_t *src = keys_a, *dst = keys_b;
    for (int p = 0; p < 4; ++p) {
        if ((e = radix_pass(src, dst, nullptr, nullptr, n, 8 * p, counts, st)) != cudaSuccess) return fail_after_launch(e);
        uint64_t* t = src; src = dst; dst = t;
    }
    k_low_words<<<grid_for(n, 256, sms), 256, 0, st>>>(n, src, sorted_ticks);
    if ((e = cudaGetLastError()) != cudaSuccess) return fail_after_launch(e);
    int32_t h_err[2] = {0, 0};
    if ((e = cudaMemcpyAsync(h_err, err, sizeof h_err, cudaMemcpyDeviceToHost, st)) != cudaSuccess) return fail_after_launch(e);
    if ((e = cudaStreamSynchronize(st)) != cudaSuccess) return set_error(DISCO_ECUDA, cudaGetErrorString(e));
    if (int rc = check_debug_record()) return rc;
    if (h_err[0]) return set_error(DISCO_EINVAL, "server TTFT not finite, not positive or above 2000 s");
    return 0;
}
