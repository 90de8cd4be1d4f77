// What the two reduction kernels over (request, policy) pairs share: the six outcomes of a pair, the 16-bit
// block-private histogram counters, and how the zone-by-zone kernel (zones.cu) tells the pair-by-pair kernel
// (pairs.cu) what it left over.
#pragma once

#include "disco_internal.cuh"

namespace disco {

// How a pair ends (dispatch of Sec. 4.2, hand-off of Sec. 4.3).  Odd outcomes: the device won the first token;
// outcomes from O_RACE_SRV on: both endpoints ran; the last two: the winner handed the stream over.
enum Outcome { O_SERVER_ONLY = 0, O_DEVICE_ONLY = 1, O_RACE_SRV = 2, O_RACE_DEV = 3, O_MIGR_TO_DEV = 4, O_MIGR_TO_SRV = 5 };

constexpr int kHWords = 433;            // 866 sixteen-bit counters per histogram row; odd word stride

// A histogram increment as one word: byte offset of the counter pair in bits 2..11, the increment (low or
// high sixteen bits) in bits 0 and 16.
__device__ __forceinline__ uint32_t hist16_code(int bin) { return ((uint32_t)(bin >> 1) << 2) | ((bin & 1) ? 0x10000u : 1u); }
__device__ __forceinline__ void hist16_apply(uint32_t* row, uint32_t code) {
    atomicAdd((uint32_t*)((char*)row + (code & 0xFFCu)), code & 0x10001u);
}
// The same increment taken away again (the word is read as two signed sixteen-bit counts, see zones.cu).
__device__ __forceinline__ void hist16_retract(uint32_t* row, uint32_t code) {
    atomicAdd((uint32_t*)((char*)row + (code & 0xFFCu)), 0u - (code & 0x10001u));
}

// One more TTFT of t ticks, t < 2^31 (so its bin is below kNBins): the counter pair and the half come straight
// from the float's exponent and leading mantissa bits, 32 bins per octave as in bin_of_ticks.
__device__ __forceinline__ void hist16_add_ticks(uint32_t* row, uint32_t t) {
    if (t < 32u) { hist16_apply(row, hist16_code((int)t)); return; }
    const uint32_t fb = __float_as_uint(__uint2float_rz(t));
    atomicAdd((uint32_t*)((char*)row - 4 * (((127 + 4) << 5) >> 1) + ((fb >> 17) & 0x3FFCu)), 1u << ((fb >> 14) & 16u));
}

// A word that holds two signed sixteen-bit counts, W = hi * 65536 + lo (mod 2^32), each within +-32767.
__device__ __forceinline__ int32_t packed_lo(uint32_t w) { return (int32_t)(int16_t)(w & 0xFFFFu); }
__device__ __forceinline__ int32_t packed_hi(uint32_t w) { return (int32_t)(w - (uint32_t)packed_lo(w)) >> 16; }

// Requests a zone-by-zone kernel could not settle for a tile are flagged in a bit mask: word
// request * words_per_request + tile / 32, bit tile % 32.
__host__ __device__ __forceinline__ uint32_t left_words_per_request(uint32_t n_tiles) { return (n_tiles + 31u) / 32u; }
// The first kLeftList of them per (chunk, tile) are also listed by chunk position, so that the pair kernel need not
// scan the flags of a chunk for a handful of requests.
constexpr uint32_t kLeftList = 2048;
// The count of a (chunk, tile) whose policies the zone-by-zone kernel could not take at all.
constexpr uint32_t kNotByZones = 0xFFFFFFFFu;

}  // namespace disco
