// Measurement aid: what the GPU sustains on the integer instruction mix of the play-out's token loop
// (Sec. 4.3: one jitter draw per generated token), with every multiprocessor full and no other work.
//
// A lane runs the lean loop of the clamp-free play-out exactly as that kernel writes it -- counter add,
// hash finaliser (three shift-xor pairs, two multiplies), one multiply-high range map, the tail test and
// the multiply-add into the running sum: 13 lane-instructions per token-step -- over a long run of tokens,
// with none of the per-request work around it (no lane sharing, no prefix sums, no hand-off search, no
// memory traffic).  Token-steps per second times 13 is the ceiling the play-out's fraction is quoted against.
#include <algorithm>

#include "disco_internal.cuh"

namespace disco {

namespace {

constexpr int kPeakThreads = 256;
constexpr int kPeakTokens = 1 << 15;       // token-steps per lane and launch

__device__ uint32_t sink[32];              // never written in practice: the store only keeps the loop's result live

__global__ void __launch_bounds__(kPeakThreads)
k_alu_peak(uint32_t k0, uint32_t mul, int tokens, int cnt, uint32_t one, uint32_t* __restrict__ out) {
    const uint32_t id = blockIdx.x * kPeakThreads + threadIdx.x;
    uint32_t hin = mix32(k0 + id * kHashReq) + 2u * kHashTok;
    uint32_t hC = 0;
#pragma unroll 4
    for (int t = 0; t < tokens; ++t) {
        const uint32_t x = __umulhi(mix32(hin), mul);
        hin += kHashTok;
        if (t < cnt) hC = x * one + hC;
    }
    if (hC == 0xFFFFFFFFu) out[id & 31u] = hC;      // keeps the loop alive; practically never taken
}

#ifdef DISCO_DEBUG
__global__ void k_debug_selftest(uint32_t* __restrict__ out, int bound) {
    const int i = bound + 2 + (int)threadIdx.x;                  // beyond the bound on purpose
    if (DBG_OK(i, bound, DBG_K_SELFTEST, DBG_ELEMENT)) out[i] = 1u;   // refused: the store never happens
}
#endif

}  // namespace

#ifdef DISCO_DEBUG
DBG_TRANSLATION_UNIT()
cudaError_t run_debug_selftest(cudaStream_t st) {
    uint32_t* d_sink = nullptr;
    cudaError_t e = cudaGetSymbolAddress((void**)&d_sink, sink);
    if (e) return e;
    k_debug_selftest<<<1, 32, 0, st>>>(d_sink, 32);
    return cudaGetLastError();
}
#endif

cudaError_t run_alu_peak(int sms, double* token_steps_per_s, cudaStream_t st) {
    uint32_t* d_sink = nullptr;
    cudaError_t e = cudaGetSymbolAddress((void**)&d_sink, sink);
    if (e) return e;
    int per_sm = 0;
    if ((e = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, k_alu_peak, kPeakThreads, 0))) return e;
    const int blocks = sms * std::max(per_sm, 1);
    cudaEvent_t e0, e1;
    if ((e = cudaEventCreate(&e0))) return e;
    if ((e = cudaEventCreate(&e1))) { cudaEventDestroy(e0); return e; }
    auto done = [&](cudaError_t r) { cudaEventDestroy(e0); cudaEventDestroy(e1); return r; };
    // one untimed launch (module load, clocks), then two timed back to back
    k_alu_peak<<<blocks, kPeakThreads, 0, st>>>(1u, 12001u, kPeakTokens, kPeakTokens, 1u, d_sink);
    if ((e = cudaEventRecord(e0, st))) return done(e);
    for (int r = 0; r < 2; ++r)
        k_alu_peak<<<blocks, kPeakThreads, 0, st>>>(2u + r, 12001u, kPeakTokens, kPeakTokens, 1u, d_sink);
    if ((e = cudaEventRecord(e1, st))) return done(e);
    if ((e = cudaGetLastError())) return done(e);
    if ((e = cudaEventSynchronize(e1))) return done(e);
    float ms = 0.f;
    if ((e = cudaEventElapsedTime(&ms, e0, e1))) return done(e);
    *token_steps_per_s = 2.0 * (double)blocks * kPeakThreads * kPeakTokens / ((double)ms * 1e-3);
    return done(cudaSuccess);
}

}  // namespace disco
