// Master step of Algorithm 1: ghat = (1/n) sum_i ghat_i, from the n = W sparse messages.
//
// Sort-free and atomic-free.  Every message row is ascending in index, so each worker's entries for
// an output range [lo, lo + kAggTile) are one contiguous run, found by binary search
// (k_agg_starts).  Sums run in double precision in worker order (0, 1, ...) and are rounded once, so
// the result is bit-reproducible.
//
//   k_aggregate_sparse  (W * k << d, the usual case): a block clears its tile of the output (or the caller
//                       has) and only the coordinates that some worker sent are computed;
//   k_aggregate         (dense messages): a block adds the runs worker by worker into a shared
//                       tile of doubles and writes the tile once (zero fill and scatter in one pass).
#pragma once

#include "common.cuh"

namespace rtopk {

constexpr int kAggTile = 4096;
constexpr int kAggThreads = 256;
constexpr int kAggStage = 1024;   // entries of one output tile staged in shared memory (dense kernel)
constexpr int kAggSparseTile = 16384;   // output coordinates per block of the sparse kernel
constexpr int kAggSparseStage = 2048;   // entries of one such tile staged in shared memory
constexpr int kAggMaxW = 1024;    // workers the sparse kernel keeps run tables for
constexpr int kAggSearchW = 64;   // up to this many workers the sparse kernel finds the runs itself

// How a coordinate's double-precision sum becomes the update: sum * num / den (Algorithm 1's 1/W:
// num = 1, den = W; the plain sum: 1, 1; the unbiased estimator's r / (W k): r, W k), or, with
// by_count, the sum divided by the number of workers that sent the coordinate.
struct AggScale { double num, den; int by_count; };
__device__ __forceinline__ double agg_scaled(double sum, uint32_t senders, const AggScale& sc) {
  if (sc.by_count) return senders ? sum / (double)senders : 0.0;
  return (sum * sc.num) / sc.den;
}

// What a coordinate's slot receives: the average itself, or (Algorithm 1's master update
// w <- w - eta * ghat, with eta < 0 meaning "store the average") the updated weight, rounded once
// from double; the product of two binary32 numbers is exact in double.
__device__ __forceinline__ float agg_result(float ghat, float old, float eta) {
  return eta < 0.0f ? ghat : (float)((double)old - (double)eta * (double)ghat);
}

// first entry of worker w's ascending row (n entries) whose index is >= key
template <typename M>
__device__ __forceinline__ uint32_t lower_bound_row(const M& msgs, uint32_t w, uint32_t n, uint32_t key) {
  uint32_t lo = 0, hi = n;
  while (lo < hi) {
    const uint32_t mid = (lo + hi) >> 1;
    if (msgs.index(w, mid) < key) lo = mid + 1; else hi = mid;
  }
  return lo;
}

// Where the sparse kernel puts a coordinate's average: into the update (or, eta >= 0, into the weight), or --
// heavy-ball momentum -- into velocity and weight, v <- mu v + ghat, w <- w - eta v, each rounded once from
// double; it then marks the coordinate in `sent` (one bit per coordinate), and k_momentum_rest takes the others.
struct AggOut {
  float* out;
  float eta, mu;
  float* velocity;
  uint32_t* sent;
  uint32_t clear;     // 1: `out` receives the average and holds anything: the block clears its tile first
  __device__ __forceinline__ void store(uint32_t idx, float ghat) const {
    if (velocity != nullptr) {
      const float v = (float)((double)mu * (double)velocity[idx] + (double)ghat);
      velocity[idx] = v;
      out[idx] = (float)((double)out[idx] - (double)eta * (double)v);
      atomicOr(sent + (idx >> 5), 1u << (idx & 31u));
    } else {
      out[idx] = agg_result(ghat, eta >= 0.0f ? out[idx] : 0.0f, eta);
    }
  }
};

// The coordinates no worker sent, under momentum: ghat is +0 there, so v <- fp32(mu v + 0), w <- fp32(w - eta v).
// grid-stride over groups of four coordinates (velocity and weights are 16-byte aligned).
__global__ void __launch_bounds__(256) k_momentum_rest(uint32_t d, float mu, float eta, const uint32_t* __restrict__ sent,
                                                        float* __restrict__ velocity, float* __restrict__ weights) {
  const uint32_t groups = (d + 3u) / 4u;
  auto one = [&](float& v, float& w) {
    v = (float)((double)mu * (double)v + 0.0);
    w = (float)((double)w - (double)eta * (double)v);
  };
  for (uint32_t g = blockIdx.x * blockDim.x + threadIdx.x; g < groups; g += gridDim.x * blockDim.x) {
    const uint32_t i = g * 4u;
    const uint32_t nib = (__ldg(sent + (i >> 5)) >> (i & 31u)) & 0xFu;
    if (i + 4u <= d) {
      if (nib == 0xFu) continue;
      float4 v = *reinterpret_cast<const float4*>(velocity + i), w = *reinterpret_cast<const float4*>(weights + i);
      if (!(nib & 1u)) one(v.x, w.x);
      if (!(nib & 2u)) one(v.y, w.y);
      if (!(nib & 4u)) one(v.z, w.z);
      if (!(nib & 8u)) one(v.w, w.w);
      *reinterpret_cast<float4*>(velocity + i) = v;
      *reinterpret_cast<float4*>(weights + i) = w;
    } else {
      for (uint32_t j = i; j < d; ++j)
        if (!((nib >> (j - i)) & 1u)) { float v = velocity[j], w = weights[j]; one(v, w); velocity[j] = v; weights[j] = w; }
    }
  }
}

// The W x K messages as the kernels read them: plain (u32 index, f32 value) rows, or the packed
// format (Section III: an index costs log d bits, a value a constant number): `bits` = ceil(log2 d)
// bits per index, entry j at bits [j * bits, (j + 1) * bits) of the row's little-endian stream of
// 32-bit words, and bfloat16 values (the upper half of the binary32 pattern).
// Every format offers index(w, j); index_in(w, j, base) for an entry known to lie in the span of
// kTiledSpan coordinates that starts at `base`; lower_bound(w, n, key) = the first of the row's n
// entries with an index >= key.
constexpr uint32_t kTiledSpan = 16384;
struct PlainMsgs {
  const uint32_t* idx;
  const float* val;
  uint32_t K;
  uint32_t stride;   // 1: two arrays of W x K words; 2: one array of W x K (index, value) pairs, val = idx + 1
  __device__ __forceinline__ uint32_t index(uint32_t w, uint32_t j) const { return __ldg(idx + ((size_t)w * K + j) * stride); }
  __device__ __forceinline__ float value(uint32_t w, uint32_t j) const { return __ldg(val + ((size_t)w * K + j) * stride); }
  __device__ __forceinline__ uint32_t index_in(uint32_t w, uint32_t j, uint32_t) const { return index(w, j); }
  __device__ __forceinline__ uint32_t lower_bound(uint32_t w, uint32_t n, uint32_t key) const { return lower_bound_row(*this, w, n, key); }
  // what worker w's value v adds to a coordinate's double-precision sum
  static constexpr bool kPerWorker = false;   // the term does not depend on the worker
  static constexpr bool kPadded = false;      // every row holds K valid entries
  __device__ __forceinline__ double term(uint32_t, float v) const { return (double)v; }
};
struct PackedMsgs {
  const uint32_t* words;
  const uint16_t* halves;
  uint32_t ld_words, ld_halves, bits;
  __device__ __forceinline__ uint32_t index(uint32_t w, uint32_t j) const {
    const uint32_t* row = words + (size_t)w * ld_words;
    const uint64_t p = (uint64_t)j * bits;
    const uint32_t wi = (uint32_t)(p >> 5), sh = (uint32_t)p & 31u;
    uint32_t v = __ldg(row + wi) >> sh;
    if (sh + bits > 32u) v |= __ldg(row + wi + 1) << (32u - sh);
    return bits >= 32u ? v : v & ((1u << bits) - 1u);
  }
  __device__ __forceinline__ float value(uint32_t w, uint32_t j) const {
    return __uint_as_float((uint32_t)__ldg(halves + (size_t)w * ld_halves + j) << 16);
  }
  __device__ __forceinline__ uint32_t index_in(uint32_t w, uint32_t j, uint32_t) const { return index(w, j); }
  __device__ __forceinline__ uint32_t lower_bound(uint32_t w, uint32_t n, uint32_t key) const { return lower_bound_row(*this, w, n, key); }
  static constexpr bool kPerWorker = false;
  static constexpr bool kPadded = false;
  __device__ __forceinline__ double term(uint32_t, float v) const { return (double)v; }
};
// The span-table format for ascending rows: the coordinates are cut into spans of kTiledSpan; a row says
// how many of its entries lie below every span boundary (tab[t], t = 0 .. spans: the entries of span t are
// tab[t] .. tab[t + 1] - 1) and keeps only the 14 low bits of each index; values are bfloat16.  The table
// is at the same time the table of run starts the sparse kernel works from.
struct TiledMsgs {
  const uint32_t* tab;      // [W][spans + 1]
  const uint16_t* low;      // [W][ld_low]
  const uint16_t* halves;   // [W][ld_halves]
  uint32_t spans, ld_low, ld_halves;
  __device__ __forceinline__ uint32_t index(uint32_t w, uint32_t j) const {     // the span of entry j: the last t with tab[t] <= j
    const uint32_t* row = tab + (size_t)w * (spans + 1);
    uint32_t a = 0, b = spans;
    while (b - a > 1) { const uint32_t mid = (a + b) >> 1; if (__ldg(row + mid) <= j) a = mid; else b = mid; }
    return a * kTiledSpan + __ldg(low + (size_t)w * ld_low + j);
  }
  __device__ __forceinline__ uint32_t index_in(uint32_t w, uint32_t j, uint32_t base) const {
    return base + __ldg(low + (size_t)w * ld_low + j);
  }
  __device__ __forceinline__ float value(uint32_t w, uint32_t j) const {
    return __uint_as_float((uint32_t)__ldg(halves + (size_t)w * ld_halves + j) << 16);
  }
  __device__ __forceinline__ uint32_t lower_bound(uint32_t w, uint32_t n, uint32_t key) const {
    const uint32_t t = key / kTiledSpan, rem = key % kTiledSpan;
    if (t >= spans) return n;
    const uint32_t* row = tab + (size_t)w * (spans + 1);
    uint32_t lo = min(n, __ldg(row + t)), hi = min(n, __ldg(row + t + 1));      // (a malformed table stays inside the row)
    const uint16_t* l = low + (size_t)w * ld_low;
    while (lo < hi) { const uint32_t mid = (lo + hi) >> 1; if (__ldg(l + mid) < rem) lo = mid + 1; else hi = mid; }
    return lo;
  }
  static constexpr bool kPerWorker = false;
  static constexpr bool kPadded = false;
  __device__ __forceinline__ double term(uint32_t, float v) const { return (double)v; }
};
// Messages of the threshold-then-subsample encoder (proof of Theorem 1): row w holds count[w] valid
// entries followed by padding (index 0xFFFFFFFF, which lies beyond every coordinate and keeps the row
// ascending), and a value enters the estimator divided by the worker's subsampling fraction
// S_w = count[w] / ones[w]: one division and one multiplication in double, each rounded to nearest.
struct ThresholdMsgs {
  const uint32_t* idx;
  const float* val;
  uint32_t K;
  const uint32_t* count;
  const uint32_t* ones;
  __device__ __forceinline__ uint32_t index(uint32_t w, uint32_t j) const { return __ldg(idx + (size_t)w * K + j); }
  __device__ __forceinline__ float value(uint32_t w, uint32_t j) const { return __ldg(val + (size_t)w * K + j); }
  __device__ __forceinline__ uint32_t index_in(uint32_t w, uint32_t j, uint32_t) const { return index(w, j); }
  __device__ __forceinline__ uint32_t lower_bound(uint32_t w, uint32_t n, uint32_t key) const { return lower_bound_row(*this, w, n, key); }
  static constexpr bool kPerWorker = true;
  static constexpr bool kPadded = true;
  __device__ __forceinline__ double term(uint32_t w, float v) const {
    return __dmul_rn((double)v, __ddiv_rn((double)__ldg(ones + w), (double)__ldg(count + w)));
  }
};

// The same as a 16-way search by each half of a warp (lanes 0-15 share one key, lanes 16-31
// another): every lane of a half returns that half's lower bound in worker w's ascending row.
template <typename M>
__device__ __forceinline__ uint32_t half_warp_lower_bound(const M& msgs, uint32_t w, uint32_t n, uint32_t key, uint32_t lane) {
  const uint32_t l = lane & 15u, sh = lane & 16u;
  uint32_t lo = 0, hi = n;                                   // the answer lies in [lo, hi]
  // both halves run the same number of steps (the range shrinks 16-fold per step whatever the key)
  for (uint32_t span = n; span > 0; span = span > 16u ? (span + 15u) / 16u - 1u : 0u) {
    const uint32_t step = (hi - lo + 15u) / 16u;              // 0 once this half is done
    const uint32_t probe = min(lo + (l + 1u) * step, hi) - 1u; // < hi; unused when step == 0
    const bool less = step != 0u && msgs.index(w, step ? probe : 0u) < key;
    const uint32_t cnt = __popc((__ballot_sync(0xFFFFFFFFu, less) >> sh) & 0xFFFFu);
    if (step != 0u) {
      const uint32_t nlo = min(hi, lo + cnt * step);
      hi = min(hi, lo + (cnt + 1u) * step - 1u);
      lo = nlo;
    }
  }
  return lo;
}

// starts[w * (ntiles + 1) + t] = first entry of worker w with index >= t * tile_size (K for t = ntiles)
template <typename M>
__global__ void __launch_bounds__(kAggThreads) k_agg_starts(M msgs, uint32_t W, uint32_t K, uint32_t ntiles,
                                                            uint32_t tile_size, uint32_t* __restrict__ starts) {
  const uint32_t t = blockIdx.x * kAggThreads + threadIdx.x;
  const uint32_t w = blockIdx.y;
  if (t > ntiles || w >= W) return;
  // padded rows end their last run at the first padding entry (padding indices exceed every tile bound)
  const uint32_t bound = t == ntiles ? 0xFFFFFFFFu : t * tile_size;
  starts[(size_t)w * (ntiles + 1) + t] = (t == ntiles && !M::kPadded) ? K : msgs.lower_bound(w, K, bound);
}

template <typename M, bool COUNT>   // COUNT: also keep the number of senders per coordinate (smaller stage to make room)
__global__ void __launch_bounds__(kAggThreads) k_aggregate(M msgs, const uint32_t* __restrict__ starts, uint32_t d,
                                                           uint32_t W, uint32_t K, AggScale sc,
                                                           float eta, float* __restrict__ out, float mu,
                                                           float* __restrict__ velocity) {
  static_assert(kTiledSpan % kAggTile == 0, "a tile lies inside one span");
  constexpr int kStage = COUNT ? kAggStage / 2 : kAggStage;
  __shared__ double acc[kAggTile];
  __shared__ uint16_t senders[COUNT ? kAggTile : 1];    // at most 65535 workers (checked by the host)
  __shared__ uint32_t s_beg[kAggThreads], s_pre[kAggThreads + 1];
  __shared__ uint32_t st_idx[kStage];
  __shared__ float st_val[kStage];
  __shared__ uint32_t s_warp[kAggThreads / 32];
  const uint32_t tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const uint32_t ntiles = gridDim.x;
  const uint32_t lo = blockIdx.x * (uint32_t)kAggTile;
  const uint32_t hi = min(d, lo + (uint32_t)kAggTile);
  const uint32_t span_lo = lo - lo % kTiledSpan;
  for (uint32_t i = tid; i < (uint32_t)kAggTile; i += kAggThreads) { acc[i] = 0.0; if (COUNT) senders[i] = 0; }
  for (uint32_t w0 = 0; w0 < W; w0 += kAggThreads) {
    const uint32_t nw = min((uint32_t)kAggThreads, W - w0);
    __syncthreads();
    // each worker's run for this tile, and the exclusive prefix of the run lengths
    uint32_t cnt = 0;
    if (tid < nw) {
      const uint32_t* st = starts + (size_t)(w0 + tid) * (ntiles + 1) + blockIdx.x;
      const uint32_t b = min(K, __ldg(st)), e = min(K, __ldg(st + 1));
      s_beg[tid] = b;
      cnt = e > b ? e - b : 0u;
    }
    const uint32_t incl = warp_incl_scan(cnt);
    if (lane == 31) s_warp[warp] = incl;
    __syncthreads();
    uint32_t woff = 0;
    for (uint32_t w = 0; w < warp; ++w) woff += s_warp[w];
    s_pre[tid] = woff + incl - cnt;
    if (tid == kAggThreads - 1) s_pre[kAggThreads] = woff + incl;
    __syncthreads();
    const uint32_t total = s_pre[kAggThreads];
    if (total <= (uint32_t)kStage) {
      // stage every entry of the tile with one round of loads, then add worker by worker
      for (uint32_t q = tid; q < total; q += kAggThreads) {
        uint32_t a = 0, b = nw;                       // last worker with s_pre[w] <= q
        while (b - a > 1) { const uint32_t mid = (a + b) >> 1; if (s_pre[mid] <= q) a = mid; else b = mid; }
        const uint32_t j = s_beg[a] + (q - s_pre[a]);
        st_idx[q] = msgs.index_in(w0 + a, j, span_lo);
        st_val[q] = msgs.value(w0 + a, j);
      }
      __syncthreads();
      for (uint32_t w = 0; w < nw; ++w) {
        const uint32_t b = s_pre[w], e = s_pre[w + 1];
        if (e > b) {                                   // block-uniform
          for (uint32_t q = b + tid; q < e; q += kAggThreads) {
            const uint32_t i = st_idx[q] - lo;        // the unsigned check keeps a malformed row inside the tile
            if (i < (uint32_t)kAggTile) { acc[i] += msgs.term(w0 + w, st_val[q]); if (COUNT) ++senders[i]; }
          }
          __syncthreads();
        }
      }
    } else {
      // worker after worker, a block barrier between them (two workers may hold the same coordinate).  The
      // first entry of every thread for the next worker is fetched before the barrier of the current one, so
      // that the barrier does not stand in front of a memory round trip.
      uint32_t nxt_i = 0;
      float nxt_v = 0.f;
      bool nxt_ok = false;
      auto fetch = [&](uint32_t w) {
        const uint32_t n = s_pre[w + 1] - s_pre[w];
        nxt_ok = tid < n;
        if (nxt_ok) { nxt_i = msgs.index_in(w0 + w, s_beg[w] + tid, span_lo) - lo; nxt_v = msgs.value(w0 + w, s_beg[w] + tid); }
      };
      fetch(0);
      for (uint32_t w = 0; w < nw; ++w) {
        const uint32_t b = s_beg[w], n = s_pre[w + 1] - s_pre[w];
        const bool ok = nxt_ok;
        const uint32_t i0 = nxt_i;
        const float v0 = nxt_v;
        if (w + 1 < nw) fetch(w + 1);
        if (ok && i0 < (uint32_t)kAggTile) { acc[i0] += msgs.term(w0 + w, v0); if (COUNT) ++senders[i0]; }
        for (uint32_t q = tid + kAggThreads; q < n; q += kAggThreads) {
          const uint32_t i = msgs.index_in(w0 + w, b + q, span_lo) - lo;
          if (i < (uint32_t)kAggTile) { acc[i] += msgs.term(w0 + w, msgs.value(w0 + w, b + q)); if (COUNT) ++senders[i]; }
        }
        __syncthreads();
      }
    }
  }
  __syncthreads();
  auto scaled = [&](uint32_t i) -> float {                 // most entries are zero: skip their division
    const double a = acc[i];
    return (float)(a != 0.0 ? agg_scaled(a, COUNT ? (uint32_t)senders[i] : 0u, sc) : a);
  };
  if (velocity != nullptr) {
    // heavy-ball momentum on the master: v <- mu v + ghat, w <- w - eta v, every coordinate, each line
    // rounded once from double (the products are exact in double)
    for (uint32_t i = tid; i < hi - lo; i += kAggThreads) {
      const float v = (float)((double)mu * (double)velocity[lo + i] + (double)scaled(i));
      velocity[lo + i] = v;
      out[lo + i] = (float)((double)out[lo + i] - (double)eta * (double)v);
    }
    return;
  }
  if (hi - lo == (uint32_t)kAggTile) {
    for (uint32_t i = tid * 4; i < (uint32_t)kAggTile; i += kAggThreads * 4) {
      float4 o;
      o.x = scaled(i + 0); o.y = scaled(i + 1); o.z = scaled(i + 2); o.w = scaled(i + 3);
      if (eta >= 0.0f) {                                   // master update: out holds the weights
        const float4 w4 = *reinterpret_cast<const float4*>(out + lo + i);
        o.x = agg_result(o.x, w4.x, eta); o.y = agg_result(o.y, w4.y, eta);
        o.z = agg_result(o.z, w4.z, eta); o.w = agg_result(o.w, w4.w, eta);
      }
      __stcs(reinterpret_cast<float4*>(out + lo + i), o);
    }
  } else {
    for (uint32_t i = tid; i < hi - lo; i += kAggThreads) {
      out[lo + i] = agg_result(scaled(i), eta >= 0.0f ? out[lo + i] : 0.0f, eta);
    }
  }
}

// Bulk asynchronous copy shared -> global (TMA): both addresses 16-byte aligned, the size a multiple of 16 bytes.
__device__ __forceinline__ void agg_bulk_store(void* dst, const void* src, uint32_t bytes) {
  asm volatile("cp.async.bulk.global.shared::cta.bulk_group [%0], [%1], %2;"
               ::"l"(__cvta_generic_to_global(dst)), "r"((uint32_t)__cvta_generic_to_shared(src)), "r"(bytes) : "memory");
}
__device__ __forceinline__ void agg_bulk_commit() { asm volatile("cp.async.bulk.commit_group;" ::: "memory"); }
// ... until every bulk copy of the calling thread has been written to its destination
__device__ __forceinline__ void agg_bulk_wait() {
  asm volatile("cp.async.bulk.wait_group 0;" ::: "memory");
  asm volatile("fence.proxy.async;" ::: "memory");                 // the block's own stores to the same words come later
}

// Named barriers of k_aggregate_sparse: its eight working warps meet on barrier 1; the clearing warp joins them
// on barrier 2.
template <int ID, int N> __device__ __forceinline__ void agg_bar_sync() { asm volatile("bar.sync %0, %1;" ::"n"(ID), "n"(N) : "memory"); }
template <int ID, int N> __device__ __forceinline__ void agg_bar_arrive() { asm volatile("bar.arrive %0, %1;" ::"n"(ID), "n"(N) : "memory"); }
template <int ID, int N> __device__ __forceinline__ bool agg_bar_or(bool flag) {
  uint32_t out;
  asm volatile(
      "{\n\t.reg .pred p, q;\n\t"
      "setp.ne.u32 q, %1, 0;\n\t"
      "bar.red.or.pred p, %2, %3, q;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(out) : "r"((uint32_t)flag), "n"(ID), "n"(N) : "memory");
  return out != 0;
}
constexpr int kAggSparseThreads = kAggThreads + 32;                 // eight working warps and the clearing warp

// A block stages the entries of its tile (all workers' runs, in worker order); the entry of the
// lowest worker that holds a coordinate owns it and sums that coordinate over the workers in
// ascending order (binary search in each staged run): the same fixed-order sum as k_aggregate.
// TILE: output coordinates per block: kAggSparseTile for sparse messages, kAggTile where a tile of that size
// would hold more entries than the stage (the bitmaps and slot tables are laid out for the larger one).
template <typename M, int TILE>
__global__ void __launch_bounds__(kAggSparseThreads, 5) k_aggregate_sparse(M msgs, const uint32_t* __restrict__ starts, uint32_t d,
                                                                  uint32_t W, uint32_t K, AggScale sc,
                                                                  float eta, float* __restrict__ out, float mu,
                                                                  float* __restrict__ velocity, uint32_t* __restrict__ sent,
                                                                  uint32_t clear, const uint32_t* __restrict__ run_cnt) {
  const AggOut dst = {out, eta, mu, velocity, sent, clear};
  __shared__ uint32_t s_beg[kAggMaxW], s_pre[kAggMaxW + 1], s_cnt[kAggSearchW];
  __shared__ uint32_t st_idx[kAggSparseStage];
  __shared__ float st_val[kAggSparseStage];
  __shared__ uint32_t s_warp[kAggThreads / 32];
  __shared__ uint32_t s_carry;
  const uint32_t tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const uint32_t ntiles = gridDim.x;
  static_assert(kTiledSpan % kAggSparseTile == 0, "a tile lies inside one span");
  static_assert(kRunTableTile == (uint32_t)kAggSparseTile, "the sparsifier's run table is kept per tile of the larger size");
  static_assert(TILE == kAggSparseTile || TILE == kAggTile, "two tile sizes");
  constexpr uint32_t kTile = (uint32_t)TILE;
  const uint32_t lo = blockIdx.x * kTile;
  const uint32_t span_lo = lo - lo % kTiledSpan;
  if (tid == 0) s_carry = 0;
  // The update is zero wherever no worker sent anything, and the block clears its tile itself.  That is the
  // ninth warp's only work: one of its lanes hands the tile to the copy engine, 4 KB of zeros from shared memory
  // at a time, and waits until they are written, while the eight working warps fetch and sort the tile's entries
  // (plain stores held every warp of the block for 3 to 6 us, and so did the copies' issue by a working thread:
  // the clearing runs at the speed at which HBM takes the zeros).  The working warps meet the clearing warp right
  // before the block's results.  (Starting the copies only once the entries have arrived, so that no load
  // queues behind them, was 1 to 3 us slower per launch.)
  constexpr uint32_t kZeroBytes = 4096;
  __shared__ __align__(128) unsigned char s_zero[kZeroBytes];
  if (warp == (uint32_t)(kAggThreads / 32)) {
    if (!clear) return;
    for (uint32_t i = lane; i < kZeroBytes / 16u; i += 32u) reinterpret_cast<uint4*>(s_zero)[i] = make_uint4(0u, 0u, 0u, 0u);
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");   // (the copy engine reads what the lanes wrote)
    __syncwarp();
    const uint32_t hi = min(d, lo + kTile), full = (hi - lo) & ~3u;
    if (lane == 0) {
      for (uint32_t b = 0; b < full * 4u; b += kZeroBytes)
        agg_bulk_store(reinterpret_cast<char*>(out + lo) + b, s_zero, min(kZeroBytes, full * 4u - b));
      agg_bulk_commit();
      agg_bulk_wait();
    }
    if (lo + full + lane < hi) out[lo + full + lane] = 0.f;           // (the last words of an update that is no multiple of 4)
    __syncwarp();
    agg_bar_sync<2, kAggSparseThreads>();                           // the results may follow
    return;
  }
  // every working warp passes this exactly once, on every path through the kernel
  auto tile_cleared = [&](bool wait) {
    if (!clear) return;
    if (wait) agg_bar_sync<2, kAggSparseThreads>(); else agg_bar_arrive<2, kAggSparseThreads>();
  };
  auto sync_w = [&]() { agg_bar_sync<1, kAggThreads>(); };
  if (starts == nullptr) {
    // no table of run starts: a warp per worker finds the run of this tile in the worker's sorted
    // row, half the warp searching for each end (16-way search: a few dependent loads)
    for (uint32_t w = warp; w < W; w += kAggThreads / 32) {
      const uint32_t end = lo > 0xFFFFFFFFu - kTile ? 0xFFFFFFFFu : lo + kTile;
      const uint32_t key = lane < 16 ? lo : end;                 // every index is below 2^32 - 1
      const uint32_t at = half_warp_lower_bound(msgs, w, K, key, lane);
      const uint32_t e = __shfl_sync(0xFFFFFFFFu, at, 16);
      if (lane == 0) { s_beg[w] = at; s_cnt[w] = e - at; }
    }
    sync_w();
  }
  for (uint32_t w0 = 0; w0 < W; w0 += kAggThreads) {
    const uint32_t w = w0 + tid;
    uint32_t cnt = 0;
    if (w < W) {
      if (run_cnt != nullptr) {
        // the run table the sparsifier kept while it wrote the messages: `starts` holds the complement of the
        // run's first place (0 where the tile got nothing), run_cnt its length
        const size_t at = (size_t)w * ntiles + blockIdx.x;
        const uint32_t b = min(K, ~__ldg(starts + at));
        s_beg[w] = b;
        cnt = min(K - b, __ldg(run_cnt + at));
      } else if (starts != nullptr) {
        const uint32_t* st = starts + (size_t)w * (ntiles + 1) + blockIdx.x;
        const uint32_t b = min(K, __ldg(st)), e = min(K, __ldg(st + 1));
        s_beg[w] = b;
        cnt = e > b ? e - b : 0u;
      } else {
        cnt = s_cnt[w];
      }
    }
    const uint32_t incl = warp_incl_scan(cnt);
    if (lane == 31) s_warp[warp] = incl;
    sync_w();
    uint32_t woff = s_carry;
    for (uint32_t x = 0; x < warp; ++x) woff += s_warp[x];
    if (w < W) s_pre[w] = woff + incl - cnt;
    sync_w();
    if (tid == kAggThreads - 1) s_carry = woff + incl;
    sync_w();
  }
  const uint32_t total = s_carry;
  if (total == 0) { tile_cleared(false); return; }
  if (tid == 0) s_pre[W] = total;
  sync_w();
  auto worker_of = [&](uint32_t q) {                 // last worker with s_pre[w] <= q
    uint32_t a = 0, b = W;
    while (b - a > 1) { const uint32_t mid = (a + b) >> 1; if (s_pre[mid] <= q) a = mid; else b = mid; }
    return a;
  };
  __shared__ uint16_t st_w[kAggSparseStage];                         // worker of every staged entry
  __shared__ uint32_t s_seen[kAggSparseTile / 32], s_shared[kAggSparseTile / 32];
  __shared__ uint16_t s_pool[kAggSparseStage];
  bool cleared = false;                                               // (block-uniform among the working warps)
  auto results_may_follow = [&]() { if (!cleared) { tile_cleared(true); cleared = true; } };
  // The entries with coordinates in [lo, lo + kTile) -- the tile, or a part of a crowded tile -- whose runs
  // s_beg / s_pre describe, `total` of them, at most the stage.
  auto staged_range = [&](const uint32_t lo, const uint32_t kTile, const uint32_t total) {
    // ---- the usual case: the entries fit the stage
    // (the run tables are not needed once the entries are staged with their workers, nor is the "seen"
    // bitmap once the shared coordinates are marked: the slot tables take their place)
    static_assert(kAggSparseStage / 2 <= kAggMaxW, "the slot tables fit the run tables");
    uint32_t* const s_off = s_pre;                                    // [kAggSparseStage / 2 + 1]
    uint32_t* const s_cur = s_beg;                                    // [kAggSparseStage / 2]
    uint32_t* const s_slot = s_seen;                                  // [kAggSparseTile / 32]
    for (uint32_t q = tid; q < total; q += kAggThreads) {
      const uint32_t a = worker_of(q);
      const uint32_t j = s_beg[a] + (q - s_pre[a]);
      st_idx[q] = msgs.index_in(a, j, span_lo);
      st_val[q] = msgs.value(a, j);
      st_w[q] = (uint16_t)a;
    }
    // Most coordinates are sent by a single worker.  Two bitmaps over the tile find the ones that are
    // not: the second entry that sets a coordinate's "seen" bit also sets its "shared" bit.
    for (uint32_t i = tid; i < (uint32_t)(kAggSparseTile / 32); i += kAggThreads) { s_seen[i] = 0; s_shared[i] = 0; }
    sync_w();
    bool any_shared = false;
    for (uint32_t q = tid; q < total; q += kAggThreads) {
      const uint32_t local = st_idx[q] - lo;
      if (local < kTile) {
        const uint32_t bit = 1u << (local & 31u);
        if (atomicOr(&s_seen[local >> 5], bit) & bit) { atomicOr(&s_shared[local >> 5], bit); any_shared = true; }
      }
    }
    any_shared = agg_bar_or<1, kAggThreads>(any_shared);                        // (block-uniform)
    // Shared coordinates (at most half the stage: each has two entries or more) get consecutive slots
    // in index order; a counting sort by slot brings every coordinate's entries together, and since
    // the stage is in worker order, taking a slot's entries by ascending stage position sums them in
    // worker order -- the same fixed-order double sum as everywhere else.
    static_assert(kAggSparseTile / 32 == 2 * kAggThreads, "two bitmap words per thread");
    uint32_t n_slots = 0;
    auto slot_of = [&](uint32_t local) { return s_slot[local >> 5] + __popc(s_shared[local >> 5] & ((1u << (local & 31u)) - 1u)); };
    if (any_shared) {
      for (uint32_t i = tid; i < (uint32_t)(kAggSparseStage / 2); i += kAggThreads) s_cur[i] = 0;
      {
        const uint32_t c0 = __popc(s_shared[2 * tid]), c1 = __popc(s_shared[2 * tid + 1]);
        const uint32_t incl = warp_incl_scan(c0 + c1);
        if (lane == 31) s_warp[warp] = incl;
        sync_w();
        uint32_t woff = 0, all = 0;
        for (uint32_t x = 0; x < (uint32_t)(kAggThreads / 32); ++x) { if (x < warp) woff += s_warp[x]; all += s_warp[x]; }
        s_slot[2 * tid] = woff + incl - c0 - c1;
        s_slot[2 * tid + 1] = woff + incl - c1;
        n_slots = all;
        sync_w();
      }
      for (uint32_t q = tid; q < total; q += kAggThreads) {            // entries per slot
        const uint32_t local = st_idx[q] - lo;
        if (local < kTile && st_idx[q] < d && ((s_shared[local >> 5] >> (local & 31u)) & 1u))
          atomicAdd(&s_cur[slot_of(local)], 1u);
      }
      sync_w();
      {                                                                 // exclusive prefix over the slots (up to 1024)
        constexpr int kPer = kAggSparseStage / 2 / kAggThreads;
        uint32_t c[kPer], sum = 0;
#pragma unroll
        for (int u = 0; u < kPer; ++u) { c[u] = s_cur[tid * kPer + u]; sum += c[u]; }
        const uint32_t incl = warp_incl_scan(sum);
        sync_w();
        if (lane == 31) s_warp[warp] = incl;
        sync_w();
        uint32_t run = incl - sum;
        for (uint32_t x = 0; x < warp; ++x) run += s_warp[x];
#pragma unroll
        for (int u = 0; u < kPer; ++u) { s_off[tid * kPer + u] = run; s_cur[tid * kPer + u] = 0; run += c[u]; }
        if (tid == kAggThreads - 1) s_off[kAggSparseStage / 2] = run;
        sync_w();
      }
      for (uint32_t q = tid; q < total; q += kAggThreads) {            // scatter the stage positions
        const uint32_t local = st_idx[q] - lo;
        if (local < kTile && st_idx[q] < d && ((s_shared[local >> 5] >> (local & 31u)) & 1u)) {
          const uint32_t sl = slot_of(local);
          s_pool[s_off[sl] + atomicAdd(&s_cur[sl], 1u)] = (uint16_t)q;
        }
      }
    }
    // the results, behind the clearing of the tile
    sync_w();                                                         // (the pool is complete)
    results_may_follow();
    for (uint32_t q = tid; q < total; q += kAggThreads) {              // a sole sender's coordinate: the sum is the value
      const uint32_t idx = st_idx[q], local = idx - lo;
      if (local >= kTile || idx >= d) continue;                      // malformed row: ignore
      if (!((s_shared[local >> 5] >> (local & 31u)) & 1u)) {
        const double v = 0.0 + msgs.term(st_w[q], st_val[q]);          // (the sum starts from +0: a lone -0 gives +0)
        dst.store(idx, (float)agg_scaled(v, 1u, sc));
      }
    }
    for (uint32_t sl = tid; sl < n_slots; sl += kAggThreads) {       // one thread per shared coordinate
      const uint32_t b = s_off[sl], e = s_off[sl + 1];
      if (e == b) continue;                                           // (only entries of a malformed row)
      double sum = 0.0;
      int32_t last = -1;
      uint32_t idx = 0;
      for (uint32_t n = b; n < e; ++n) {                              // next stage position above `last`
        uint32_t best = 0xFFFFFFFFu;
        for (uint32_t x = b; x < e; ++x) { const uint32_t q = s_pool[x]; if ((int32_t)q > last && q < best) best = q; }
        last = (int32_t)best;
        idx = st_idx[best];
        sum += msgs.term(st_w[best], st_val[best]);
      }
      dst.store(idx, (float)agg_scaled(sum, e - b, sc));
    }
  };
  // ---- more entries than the stage holds, in a range that cannot be split further: every entry looks the
  // other workers' runs up in global memory; the entry of the lowest worker that holds a coordinate owns it
  // and sums that coordinate over the workers in ascending order
  auto idx_at = [&](uint32_t w, uint32_t j) { return msgs.index_in(w, s_beg[w] + j, span_lo); };
  auto val_at = [&](uint32_t w, uint32_t j) { return msgs.value(w, s_beg[w] + j); };
  auto searched_range = [&](const uint32_t lo, const uint32_t kTile, const uint32_t total) {
  results_may_follow();
  for (uint32_t q = tid; q < total; q += kAggThreads) {
    const uint32_t w = worker_of(q);
    const uint32_t idx = idx_at(w, q - s_pre[w]);
    if (idx - lo >= kTile || idx >= d) continue;                      // malformed row: ignore
    double sum = 0.0;
    uint32_t senders = 0;
    bool owner = true;
    for (uint32_t x = 0; x < W; ++x) {
      if (x == w) { sum += msgs.term(w, val_at(w, q - s_pre[w])); ++senders; continue; }
      const uint32_t n = s_pre[x + 1] - s_pre[x];
      uint32_t a = 0, b = n;
      while (a < b) { const uint32_t mid = (a + b) >> 1; if (idx_at(x, mid) < idx) a = mid + 1; else b = mid; }
      if (a < n && idx_at(x, a) == idx) {
        if (x < w) { owner = false; break; }          // a lower worker owns this coordinate
        sum += msgs.term(x, val_at(x, a));
        ++senders;
      }
    }
    if (owner) {
      dst.store(idx, (float)agg_scaled(sum, senders, sc));
    }
  }
  };
  if (total <= (uint32_t)kAggSparseStage) { staged_range(lo, kTile, total); return; }
  // ---- a crowded tile (messages that concentrate on a part of the vector): the tile is taken in equal parts
  // small enough that a part's entries are expected to fill half the stage; a thread keeps the tile's runs of
  // its workers and finds every part's end in them by binary search (the start is the last part's end)
  constexpr int kMine = kAggMaxW / kAggThreads;
  uint32_t t_beg[kMine], t_cnt[kMine], t_cur[kMine];
#pragma unroll
  for (int i = 0; i < kMine; ++i) {
    const uint32_t w = (uint32_t)i * kAggThreads + tid;
    t_beg[i] = w < W ? s_beg[w] : 0u;
    t_cnt[i] = w < W ? s_pre[w + 1] - s_pre[w] : 0u;
    t_cur[i] = 0;
  }
  uint32_t parts = 2;
  while (parts < kTile / 32u && total / parts > (uint32_t)(kAggSparseStage / 2)) parts *= 2;
  const uint32_t part_len = kTile / parts;
  sync_w();
  for (uint32_t p = 0; p < parts; ++p) {
    const uint32_t p_lo = lo + p * part_len;
    const bool last_part = p + 1 == parts;
    if (tid == 0) s_carry = 0;
    sync_w();
#pragma unroll
    for (int i = 0; i < kMine; ++i) {
      if ((uint32_t)i * kAggThreads >= W) break;                        // (block-uniform)
      const uint32_t w = (uint32_t)i * kAggThreads + tid;
      uint32_t cnt = 0;
      if (w < W) {
        uint32_t a = t_cur[i], b = t_cnt[i];
        if (!last_part) {
          const uint32_t end = p_lo + part_len;                         // first entry of the run at or above it
          while (a < b) { const uint32_t mid = (a + b) >> 1; if (msgs.index_in(w, t_beg[i] + mid, span_lo) < end) a = mid + 1; else b = mid; }
        } else {
          a = b;
        }
        s_beg[w] = t_beg[i] + t_cur[i];
        cnt = a - t_cur[i];
        t_cur[i] = a;
      }
      const uint32_t incl = warp_incl_scan(cnt);
      if (lane == 31) s_warp[warp] = incl;
      sync_w();
      uint32_t woff = s_carry;
      for (uint32_t x = 0; x < warp; ++x) woff += s_warp[x];
      if (w < W) s_pre[w] = woff + incl - cnt;
      sync_w();
      if (tid == kAggThreads - 1) s_carry = woff + incl;
      sync_w();
    }
    const uint32_t part_total = s_carry;
    if (tid == 0) s_pre[W] = part_total;
    sync_w();
    if (part_total != 0) {
      if (part_total <= (uint32_t)kAggSparseStage) staged_range(p_lo, part_len, part_total);
      else searched_range(p_lo, part_len, part_total);
    }
    sync_w();                                                           // (the run tables are rebuilt for the next part)
  }
  if (!cleared) tile_cleared(false);
}

}  // namespace rtopk
