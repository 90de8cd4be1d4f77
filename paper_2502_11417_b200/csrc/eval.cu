// Policy preparation (Algorithms 1-3) and per-pair evaluation.
//
// Relative to its first token, a request's decode stream depends on a policy only through the winning
// endpoint, the pacing interval, the buffer size and whether a hand-off happens -- not on the budget.
// So each request is played out token by token once per timeline class for its (at most) three distinct
// streams (playout.cu): server decodes all, device decodes all, and the dearer winner hands off to the
// other endpoint.  The pair kernel here derives every policy's dispatch decision and picks the stream
// that applies.
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

// ------------------------------------------------------------------------------------------------------
// Pairs: one thread per request, looping over a tile of policies.  A block owns a request chunk of one
// group and a policy tile, with both histograms of the tile privatised in shared memory.
// ------------------------------------------------------------------------------------------------------
constexpr int kPT = 16;                 // policies per tile
constexpr int kPairThreads = 256;
constexpr int kHStride = kNBins + 1;    // odd stride: equal bins of neighbouring policies fall in different banks

__global__ void __launch_bounds__(kPairThreads)
k_pairs(TraceDev tr, const GroupConst* __restrict__ gcs, const ClassConst* __restrict__ ccp,
        const Prep* __restrict__ prep, uint32_t P, const uint32_t* __restrict__ pol_list, uint32_t n_list,
        const Chunk* __restrict__ chunks, TimelineRec rec, disco_pair_out_t out,
        unsigned long long* __restrict__ acc, unsigned long long* __restrict__ hist_ttft,
        unsigned long long* __restrict__ hist_tbt) {
    extern __shared__ uint32_t smem[];
    uint32_t* h_ttft = smem;                                  // [kPT][kHStride]
    uint32_t* h_tbt = h_ttft + kPT * kHStride;
    uint32_t* s_acc = h_tbt + kPT * kHStride;                 // [kPT][kNAcc]
    __shared__ Prep s_prep[kPT];
    __shared__ uint32_t s_pol[kPT];

    const Chunk ch = chunks[blockIdx.x];
    const int g = ch.g;
    const uint32_t tile0 = blockIdx.y * kPT;
    const int npol = (int)min((uint32_t)kPT, n_list - tile0);
    const GroupConst gc = gcs[g];
    const ClassConst& cc = *ccp;
    const int lane = threadIdx.x & 31;

    for (int i = threadIdx.x; i < 2 * kPT * kHStride + kPT * kNAcc; i += kPairThreads) smem[i] = 0;
    if ((int)threadIdx.x < npol) {
        const uint32_t p = pol_list[tile0 + threadIdx.x];
        s_pol[threadIdx.x] = p;
        s_prep[threadIdx.x] = prep[(size_t)g * P + p];
    }
    __syncthreads();

    const int bin_tau = cc.pacing ? bin_of_ticks((uint32_t)cc.tau) : 0;
    const int W[3] = {cc.W[0], cc.W[1], cc.W[2]};
    const int lo[3] = {cc.lo[g][0], cc.lo[g][1], cc.lo[g][2]};
    const int kt[3] = {cc.ktau[g][0], cc.ktau[g][1], cc.ktau[g][2]};
    const size_t N = tr.n;

    for (uint32_t base = 0; base < ch.len; base += kPairThreads) {
        const uint32_t r = base + threadIdx.x;
        const bool live = r < ch.len;
        const uint32_t k = ch.start + (live ? r : 0u);
        const uint32_t l = tr.l[k], n = tr.nout[k], S = (uint32_t)tr.S[k], orig = tr.orig[k];
        const uint32_t m = rec.m[k];
        const uint32_t Td = (uint32_t)gc.kappa * l + (uint32_t)gc.c0;
        const float saving = gc.delta_c * (float)(n - m);               // Eq. 4: delta_c * remaining
        const float inv_cnt = n > 1 ? 1.0f / (float)(n - 1) : 0.0f;

        for (int pi = 0; pi < npol; ++pi) {
            const Prep pr = s_prep[pi];
            // ---- dispatch (Algorithm 2's wait map / Algorithm 3's threshold) and the race
            const bool dev_only = !pr.device_constrained && (int32_t)l < pr.l_th;
            uint32_t w = 0;
            if (pr.device_constrained)
                w = (int32_t)l < pr.l_star ? 0u : ((int32_t)l == pr.l_star ? (uint32_t)pr.w_star : (uint32_t)pr.w_tail);
            const bool started = dev_only || S > w;
            const uint32_t wTd = w + Td;
            const bool dev_wins = dev_only || (started && S > wTd);     // a tie goes to the server
            const uint32_t ttft = dev_only ? Td : min(S, wTd);
            const int decision = dev_only ? DISCO_DEVICE_ONLY : (started ? DISCO_RACE : DISCO_SERVER_ONLY);
            // ---- migration trigger (Eq. 4) for a dearer winner whose buffer filled at m
            const bool migr = pr.mig_on && decision == DISCO_RACE && m != 0 &&
                              gc.candidate == (dev_wins ? 2 : 1) && saving > pr.theta;
            const int c = migr ? 2 : (dev_wins ? 1 : 0);
            const uint32_t sum = rec.sum[c][k], mx = rec.max[c][k];
            const uint32_t tok_src = migr ? m : n;
            const uint32_t tok_dev = dev_wins ? tok_src : n - tok_src;
            const uint32_t tok_srv = n - tok_dev;
            uint32_t pre_srv = dev_only ? 0u : l, pre_dev = started ? l : 0u;
            if (migr) { if (dev_wins) pre_srv += l + m; else pre_dev += l + m; }
            const uint32_t dly = migr ? rec.delayed[k] : 0u;

            // ---- reductions
            if (live) {
                atomicAdd(&h_ttft[pi * kHStride + bin_of_ticks(ttft)], 1u);
                const uint32_t* wp = rec.win[c] + (size_t)k * W[c];
                for (int kk = 0; kk < W[c]; ++kk) {
                    if (kk == kt[c]) continue;
                    const uint32_t v = wp[kk];
                    if (v) atomicAdd(&h_tbt[pi * kHStride + lo[c] + kk], v);
                }
                if (migr) atomicAdd(&h_tbt[pi * kHStride + bin_of_ticks(rec.stall[k])], 1u);
            }
            const uint32_t tau_cnt = (live && kt[c] >= 0) ? rec.win[c][(size_t)k * W[c] + kt[c]] : 0u;
            const uint32_t v_tau = __reduce_add_sync(0xFFFFFFFFu, tau_cnt);
            const uint32_t b_so = __ballot_sync(0xFFFFFFFFu, live && decision == DISCO_SERVER_ONLY);
            const uint32_t b_do = __ballot_sync(0xFFFFFFFFu, live && dev_only);
            const uint32_t b_rc = __ballot_sync(0xFFFFFFFFu, live && decision == DISCO_RACE);
            const uint32_t b_st = __ballot_sync(0xFFFFFFFFu, live && started);
            const uint32_t b_dw = __ballot_sync(0xFFFFFFFFu, live && decision == DISCO_RACE && dev_wins);
            const uint32_t b_mg = __ballot_sync(0xFFFFFFFFu, live && migr);
            const uint32_t v_td = __reduce_add_sync(0xFFFFFFFFu, live ? tok_dev : 0u);
            const uint32_t v_ps = __reduce_add_sync(0xFFFFFFFFu, live ? pre_srv : 0u);
            const uint32_t v_pd = __reduce_add_sync(0xFFFFFFFFu, live ? pre_dev : 0u);
            const uint32_t v_dl = b_mg ? __reduce_add_sync(0xFFFFFFFFu, live ? dly : 0u) : 0u;
            const uint32_t v_tl = __reduce_add_sync(0xFFFFFFFFu, live ? (ttft & 0xFFFFu) : 0u);
            const uint32_t v_th = __reduce_add_sync(0xFFFFFFFFu, live ? (ttft >> 16) : 0u);
            if (lane == 0) {
                uint32_t* a = s_acc + pi * kNAcc;
                atomicAdd(&a[A_SERVER_ONLY], __popc(b_so)); atomicAdd(&a[A_DEVICE_ONLY], __popc(b_do));
                atomicAdd(&a[A_RACE], __popc(b_rc)); atomicAdd(&a[A_STARTED], __popc(b_st));
                atomicAdd(&a[A_DEVICE_WON], __popc(b_dw)); atomicAdd(&a[A_MIGR], __popc(b_mg));
                atomicAdd(&a[A_TOK_DEVICE], v_td); atomicAdd(&a[A_PRE_SERVER], v_ps);
                atomicAdd(&a[A_PRE_DEVICE], v_pd); atomicAdd(&a[A_DELAYED], v_dl);
                atomicAdd(&a[A_TTFT_LO], v_tl); atomicAdd(&a[A_TTFT_HI], v_th);
                if (v_tau) atomicAdd(&h_tbt[pi * kHStride + bin_tau], v_tau);
            }

            // ---- per-pair outputs (requests contiguous within a policy row)
            if (live) {
                const size_t o = (size_t)s_pol[pi] * N + orig;
                if (out.ttft_s) out.ttft_s[o] = (float)ttft * 1e-6f;
                if (out.tbt_mean_s) out.tbt_mean_s[o] = (float)sum * 1e-6f * inv_cnt;
                if (out.tbt_max_s) out.tbt_max_s[o] = (float)mx * 1e-6f;
                if (out.cost) out.cost[o] = gc.cps * (float)pre_srv + gc.cds * (float)tok_srv +
                                            gc.lcpd * (float)pre_dev + gc.lcdd * (float)tok_dev;
                if (out.tok_server) out.tok_server[o] = tok_srv;
                if (out.tok_device) out.tok_device[o] = tok_dev;
                if (out.mig_at) out.mig_at[o] = migr ? m : 0u;
                if (out.delayed) out.delayed[o] = (uint16_t)dly;
                if (out.decision) out.decision[o] = (uint8_t)decision;
            }
        }
    }
    __syncthreads();
    // ---- flush the block's partial sums
    for (int i = threadIdx.x; i < npol * kHStride; i += kPairThreads) {
        const int pi = i / kHStride, b = i - pi * kHStride;
        if (b >= kNBins) continue;
        const size_t o = (size_t)s_pol[pi] * kNBins + b;
        if (h_ttft[i]) atomicAdd(&hist_ttft[o], (unsigned long long)h_ttft[i]);
        if (h_tbt[i]) atomicAdd(&hist_tbt[o], (unsigned long long)h_tbt[i]);
    }
    for (int i = threadIdx.x; i < npol * kNAcc; i += kPairThreads) {
        const int pi = i / kNAcc, s = i - pi * kNAcc;
        if (s_acc[i]) atomicAdd(&acc[((size_t)s_pol[pi] * tr.n_groups + g) * kNAcc + s], (unsigned long long)s_acc[i]);
    }
}

size_t pairs_smem_bytes() { return sizeof(uint32_t) * (2 * kPT * kHStride + kPT * kNAcc); }

}  // namespace

cudaError_t launch_prep(const PolicyConst* pol, uint32_t P, int G, const GroupConst* gc, const int64_t* cum_mass,
                        const uint32_t* cnt, const int32_t* sorted, const uint32_t* grp_off, Prep* prep,
                        cudaStream_t st) {
    const uint32_t total = P * (uint32_t)G;
    k_prep<<<(total + 127) / 128, 128, 0, st>>>(pol, P, G, gc, cum_mass, cnt, sorted, grp_off, prep);
    return cudaGetLastError();
}

cudaError_t launch_pairs(const TraceDev& tr, const GroupConst* gc, const ClassConst* cc, const Prep* prep, uint32_t P,
                         const uint32_t* pol_list, uint32_t n_list, const Chunk* chunks, uint32_t n_chunks,
                         TimelineRec rec, disco_pair_out_t out, uint64_t* acc, uint64_t* hist_ttft,
                         uint64_t* hist_tbt, cudaStream_t st) {
    if (n_chunks == 0 || n_list == 0) return cudaSuccess;
    cudaError_t e = cudaFuncSetAttribute(k_pairs, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                         (int)pairs_smem_bytes());
    if (e) return e;
    dim3 grid(n_chunks, (n_list + kPT - 1) / kPT);
    k_pairs<<<grid, kPairThreads, pairs_smem_bytes(), st>>>(tr, gc, cc, prep, P, pol_list, n_list, chunks, rec, out,
                                                            (unsigned long long*)acc, (unsigned long long*)hist_ttft,
                                                            (unsigned long long*)hist_tbt);
    return cudaGetLastError();
}

}  // namespace disco
