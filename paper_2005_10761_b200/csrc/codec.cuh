// Packed message format (Section III: an index costs log d bits and a value a constant number of
// bits): ceil(log2 d)-bit indices in a little-endian bit stream of 32-bit words, bfloat16 values
// rounded to nearest even.  Algorithm 1 keeps m = a - ghat with ghat what is sent, so the rounding
// error of a sent value goes back into its residual slot.  The decoder lives in the aggregation
// kernels (PackedMsgs in aggregate.cuh).  A second format for ascending rows (a table of entry counts
// per span of coordinates plus 14 low bits per index) is encoded at the end of this file.
#pragma once

#include "common.cuh"

namespace rtopk {

constexpr int kCodecThreads = 256;

// binary32 -> bfloat16, round to nearest, ties to even; NaN -> 0x7FC0
__device__ __forceinline__ uint16_t bf16_round(float x) {
  uint32_t u = __float_as_uint(x);
  if ((u & 0x7FFFFFFFu) > 0x7F800000u) return (uint16_t)0x7FC0u;
  u += 0x7FFFu + ((u >> 16) & 1u);
  return (uint16_t)(u >> 16);
}

// grid (blocks over max(words, entries), W).  A thread builds one word of the index stream from
// the entries that overlap it (no atomics, no clearing) and converts one value.
__global__ void __launch_bounds__(kCodecThreads) k_encode(const uint32_t* __restrict__ msg_idx,
                                                          const float* __restrict__ msg_val, uint32_t K,
                                                          uint32_t bits, float* residual, int64_t ld_m,
                                                          uint32_t* __restrict__ words, uint32_t ld_words,
                                                          uint16_t* __restrict__ halves, uint32_t ld_halves) {
  const uint32_t w = blockIdx.y;
  const uint32_t t = blockIdx.x * kCodecThreads + threadIdx.x;
  const uint32_t* idx = msg_idx + (size_t)w * K;
  const float* val = msg_val + (size_t)w * K;
  if (t < ld_words) {
    const uint64_t first_bit = (uint64_t)t * 32u;
    uint32_t word = 0;
    for (uint64_t j = first_bit / bits; j < K && j * bits < first_bit + 32u; ++j) {
      const uint32_t v = __ldg(idx + j);
      const int64_t sh = (int64_t)(j * bits) - (int64_t)first_bit;     // where the entry starts in this word
      word |= sh >= 0 ? v << sh : v >> (-sh);
    }
    words[(size_t)w * ld_words + t] = word;
  }
  if (t < ld_halves) {
    uint16_t q = 0;
    if (t < K) {
      const float a = __ldg(val + t);
      q = bf16_round(a);
      if (residual) {
        const float back = __uint_as_float((uint32_t)q << 16);
        const bool finite = (__float_as_uint(back) & 0x7F800000u) != 0x7F800000u;
        residual[(size_t)w * (size_t)ld_m + __ldg(idx + t)] = finite ? __fsub_rn(a, back) : 0.0f;
      }
    }
    halves[(size_t)w * ld_halves + t] = q;
  }
}

// The span-table format (TiledMsgs in aggregate.cuh).  grid (blocks over max(ld_low, ld_halves), W).  A thread
// takes one entry: its 14 low index bits, its value, and the table words of the spans that begin between
// the entry before it and itself (each word is written by exactly one thread; the last entry also writes
// the words behind it).  `span` = coordinates per span.
__global__ void __launch_bounds__(kCodecThreads) k_encode_tiled(const uint32_t* __restrict__ msg_idx,
                                                                const float* __restrict__ msg_val, uint32_t K,
                                                                uint32_t d, uint32_t span, uint32_t spans, float* residual,
                                                                int64_t ld_m, uint32_t* __restrict__ tab,
                                                                uint16_t* __restrict__ low, uint32_t ld_low,
                                                                uint16_t* __restrict__ halves, uint32_t ld_halves) {
  const uint32_t w = blockIdx.y;
  const uint32_t t = blockIdx.x * kCodecThreads + threadIdx.x;
  const uint32_t* idx = msg_idx + (size_t)w * K;
  const float* val = msg_val + (size_t)w * K;
  uint16_t l = 0, q = 0;
  if (t < K) {
    const uint32_t i = __ldg(idx + t);
    uint32_t* row = tab + (size_t)w * (spans + 1);
    const uint32_t mine = min(i / span, spans);                      // (an index beyond d stays inside the table)
    const uint32_t from = t == 0 ? 0u : min(__ldg(idx + t - 1) / span, spans) + 1u;
    for (uint32_t s = from; s <= mine; ++s) row[s] = t;              // spans that begin at or before this entry
    if (t == K - 1)
      for (uint32_t s = mine + 1u; s <= spans; ++s) row[s] = K;
    l = (uint16_t)(i % span);
    const float a = __ldg(val + t);
    q = bf16_round(a);
    if (residual && i < d) {
      const float back = __uint_as_float((uint32_t)q << 16);
      const bool finite = (__float_as_uint(back) & 0x7F800000u) != 0x7F800000u;
      residual[(size_t)w * (size_t)ld_m + i] = finite ? __fsub_rn(a, back) : 0.0f;
    }
  }
  if (t < ld_low) low[(size_t)w * ld_low + t] = l;
  if (t < ld_halves) halves[(size_t)w * ld_halves + t] = q;
}

}  // namespace rtopk
