// Master step of Algorithm 1: ghat = (1/n) sum_i ghat_i, from the n = W sparse messages.
//
// Sort-free and atomic-free: every message row is ascending in index, so each worker's entries for
// an output range [lo, lo + kAggTile) are one contiguous run, found by binary search (k_agg_starts).
// The block that owns the range adds them worker by worker into a shared-memory tile of doubles (a worker's indices are distinct,
// so there is no conflict inside a round), and writes the tile once -- the zero fill of the dense
// output and the scatter are the same pass.  The sum order is fixed (worker 0, 1, ...), so the
// result is bit-reproducible.
#pragma once

#include "common.cuh"

namespace rtopk {

constexpr int kAggTile = 4096;
constexpr int kAggThreads = 256;

__device__ __forceinline__ uint32_t lower_bound_u32(const uint32_t* a, uint32_t n, uint32_t key) {
  uint32_t lo = 0, hi = n;
  while (lo < hi) {
    const uint32_t mid = (lo + hi) >> 1;
    if (__ldg(a + mid) < key) lo = mid + 1; else hi = mid;
  }
  return lo;
}

// starts[w * (ntiles + 1) + t] = first entry of worker w with index >= t * kAggTile (K for t = ntiles)
__global__ void __launch_bounds__(kAggThreads) k_agg_starts(const uint32_t* __restrict__ msg_idx, uint32_t W,
                                                            uint32_t K, uint32_t ntiles,
                                                            uint32_t* __restrict__ starts) {
  const uint32_t t = blockIdx.x * kAggThreads + threadIdx.x;
  const uint32_t w = blockIdx.y;
  if (t > ntiles || w >= W) return;
  const uint32_t* row = msg_idx + (size_t)w * K;
  starts[(size_t)w * (ntiles + 1) + t] = t == ntiles ? K : lower_bound_u32(row, K, t * (uint32_t)kAggTile);
}

__global__ void __launch_bounds__(kAggThreads) k_aggregate(const uint32_t* __restrict__ msg_idx,
                                                           const float* __restrict__ msg_val,
                                                           const uint32_t* __restrict__ starts, uint32_t d,
                                                           uint32_t W, uint32_t K, int mean,
                                                           float* __restrict__ out) {
  __shared__ double acc[kAggTile];
  __shared__ uint32_t s_beg[kAggThreads], s_end[kAggThreads];
  const uint32_t tid = threadIdx.x;
  const uint32_t ntiles = gridDim.x;
  const uint32_t lo = blockIdx.x * (uint32_t)kAggTile;
  const uint32_t hi = min(d, lo + (uint32_t)kAggTile);
  for (uint32_t i = tid; i < (uint32_t)kAggTile; i += kAggThreads) acc[i] = 0.0;
  for (uint32_t w0 = 0; w0 < W; w0 += kAggThreads) {
    const uint32_t nw = min((uint32_t)kAggThreads, W - w0);
    __syncthreads();
    if (tid < nw) {
      const uint32_t* st = starts + (size_t)(w0 + tid) * (ntiles + 1) + blockIdx.x;
      s_beg[tid] = __ldg(st); s_end[tid] = __ldg(st + 1);
    }
    __syncthreads();
    // round w adds worker w's entries; the next worker's first entry per thread is fetched early
    uint32_t nxt_i = 0; float nxt_v = 0.f;
    {
      const uint32_t b = s_beg[0], e = s_end[0];
      if (b + tid < e) { nxt_i = __ldg(msg_idx + (size_t)w0 * K + b + tid); nxt_v = __ldg(msg_val + (size_t)w0 * K + b + tid); }
    }
    for (uint32_t w = 0; w < nw; ++w) {
      const uint32_t b = s_beg[w], e = s_end[w];
      const uint32_t cur_i = nxt_i; const float cur_v = nxt_v;
      if (w + 1 < nw) {
        const uint32_t b2 = s_beg[w + 1], e2 = s_end[w + 1];
        const size_t row2 = (size_t)(w0 + w + 1) * K;
        if (b2 + tid < e2) { nxt_i = __ldg(msg_idx + row2 + b2 + tid); nxt_v = __ldg(msg_val + row2 + b2 + tid); }
      }
      const size_t row = (size_t)(w0 + w) * K;
      // the unsigned range check keeps a malformed (unsorted / out-of-range) row inside the tile
      if (b + tid < e && cur_i - lo < (uint32_t)kAggTile) acc[cur_i - lo] += (double)cur_v;
      for (uint32_t q = b + tid + kAggThreads; q < e; q += kAggThreads) {
        const uint32_t i = __ldg(msg_idx + row + q) - lo;
        if (i < (uint32_t)kAggTile) acc[i] += (double)__ldg(msg_val + row + q);
      }
      __syncthreads();
    }
  }
  __syncthreads();
  const double inv = (double)W;
  if (hi - lo == (uint32_t)kAggTile) {
    for (uint32_t i = tid * 4; i < (uint32_t)kAggTile; i += kAggThreads * 4) {
      float4 o;
      o.x = (float)(mean ? acc[i + 0] / inv : acc[i + 0]);
      o.y = (float)(mean ? acc[i + 1] / inv : acc[i + 1]);
      o.z = (float)(mean ? acc[i + 2] / inv : acc[i + 2]);
      o.w = (float)(mean ? acc[i + 3] / inv : acc[i + 3]);
      __stcs(reinterpret_cast<float4*>(out + lo + i), o);
    }
  } else {
    for (uint32_t i = tid; i < hi - lo; i += kAggThreads)
      out[lo + i] = (float)(mean ? acc[i] / inv : acc[i]);
  }
}

}  // namespace rtopk
