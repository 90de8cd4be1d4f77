// Arguments of the device-side trace ingestion (all pointers are device memory).
#pragma once

#include "disco_internal.cuh"

namespace disco {

constexpr uint32_t kRadixMaxBlocks = 1024;

struct LoadReadback {            // what the host needs after a load, gathered for one copy
    int32_t err[4];
    uint32_t max_n;
    uint32_t ng[kMaxGroups];
    uint32_t grp_off[kMaxGroups + 1];
    int32_t knot_max[kMaxGroups];
    uint64_t grp_sum_n[kMaxGroups];
};

struct LoadArgs {
    uint32_t n, ns, nd;
    // inputs in the caller's order
    const int32_t *prompt, *outlen;
    const float* ttft;
    const uint8_t *sp, *dp;               // may be null
    // scratch
    uint64_t *keys_a, *keys_b;            // [n] (group << 32 | ticks)
    uint16_t *l_tmp, *n_tmp;              // [n] each: lengths in the caller's order
    uint32_t* cursors;                    // [G][4097]: next free place of each (group, prompt length)
    uint4* placed;                        // [n]: the requests in the internal order, one record each
    uint32_t* radix_counts;               // [5][256 * kRadixMaxBlocks], directly after zero_block's tables
    void* zero_block; size_t zero_bytes;  // cnt, grp_sum_n, ng, max_n, err, contiguous
    uint32_t* ng_exact;                   // [G] group sizes recounted from the length histogram
    LoadReadback* readback;               // device copy of what the host reads back
    // outputs
    int32_t* S; uint16_t *l, *nout; uint32_t* orig;   // internal order (by group, then by prompt length), [n]
    uint32_t* inv;                        // [n]: place of each of the caller's requests in the internal order
    int32_t* sorted;                      // [n] ticks ascending within each group
    uint32_t* cnt;                        // [G][4097] requests per prompt length
    int64_t* cum_mass;                    // [G][4098]
    uint32_t *ng, *grp_off;               // [G], [G+1]
    int32_t* knots;                       // [G][257]
    uint64_t* grp_sum_n;                  // [kMaxGroups] output tokens per group
    uint32_t* max_n;                      // longest output
    int32_t* err;                         // [4]: code, request index, window flag
    uint64_t* fin_totals;                 // [2G]: output tokens per group, then requests per group
    int sms;                              // multiprocessors of the device (grid sizing)
};

cudaError_t run_load(const LoadArgs& a, cudaStream_t st);
uint32_t load_kernel_launches(uint32_t n, int G);   // kernels run_load launches for such a trace

}  // namespace disco
