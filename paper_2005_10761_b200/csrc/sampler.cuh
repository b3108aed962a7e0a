// The uniformly random k-subset of Definition 3, as positions in the top-r list.
//
// The contract is Floyd's sequential loop: for j = r-k .. r-1 draw t_j uniform on {0..j}; insert
// t_j unless it is already in the set, else insert j.  The kernels below compute the same set
// without the sequential dependence.  Let F(v) be the first iteration that draws v.  Iteration j
// finds t_j already present iff an earlier iteration drew it (F(t_j) < j), or t_j is itself an
// earlier iteration index (r-k <= t_j < j) that had to insert its own index -- which is the same
// question asked of iteration t_j, so the chain strictly descends and ends.  F is built with
// atomicMin, hence independent of scheduling.
#pragma once

#include "common.cuh"

namespace rtopk {

constexpr int kDrawThreads = 256;

// First-occurrence table F(v) = first iteration that draws v.  Dense (one entry per position) while
// r is within 16 k; beyond that (random-k like settings, r >> k) a hash table over the k drawn
// values: keys[slot] | first[slot], linear probing, both halves start at 0xFFFFFFFF.  The slot a
// value lands in depends on scheduling, the minimum stored under the value does not.
__device__ __forceinline__ uint32_t first_hash(uint32_t v, uint32_t mask) { return ((v * 2654435761u) >> 5) & mask; }

__device__ __forceinline__ void first_note(uint32_t* table, uint32_t mask, uint32_t v, uint32_t j) {
  if (mask == 0) { atomicMin(&table[v], j); return; }
  uint32_t* keys = table;
  uint32_t* firsts = table + mask + 1u;
  uint32_t h = first_hash(v, mask);
  for (uint32_t probe = 0; probe <= mask; ++probe) {          // the table has at least 2 k slots: a free one exists
    const uint32_t old = atomicCAS(&keys[h], 0xFFFFFFFFu, v);
    if (old == 0xFFFFFFFFu || old == v) { atomicMin(&firsts[h], j); return; }
    h = (h + 1u) & mask;
  }
}

__device__ __forceinline__ uint32_t first_of(const uint32_t* table, uint32_t mask, uint32_t v) {
  if (mask == 0) return table[v];
  uint32_t h = first_hash(v, mask);
  for (uint32_t probe = 0; probe <= mask; ++probe) {
    const uint32_t key = table[h];
    if (key == v) return table[mask + 1u + h];
    if (key == 0xFFFFFFFFu) break;
    h = (h + 1u) & mask;
  }
  return 0xFFFFFFFFu;                                          // never drawn
}

// grid: (ceil(k_max / kDrawThreads), n_slices)
__global__ void __launch_bounds__(kDrawThreads) k_draw(Launch L) {
  const Slice S = L.s.slices[blockIdx.y];
  if (S.k == S.r) return;
  const uint32_t i = blockIdx.x * kDrawThreads + threadIdx.x;
  if (i >= S.k) return;
  const uint32_t j = S.r - S.k + i;
  const uint32_t step = L.step_ptr ? __ldg(L.step_ptr) : L.step;
  const uint32_t t = floyd_draw(j, L.worker_base + S.row, S.segment, step, L.seed_lo, L.seed_hi);
  L.s.draws[S.samp_off + i] = t;
  first_note(L.s.first + S.first_off, S.first_mask, t, j);
}

__global__ void __launch_bounds__(kDrawThreads) k_resolve(Launch L) {
  const Slice S = L.s.slices[blockIdx.y];
  if (S.k == S.r) return;
  const uint32_t i = blockIdx.x * kDrawThreads + threadIdx.x;
  if (i >= S.k) return;
  const uint32_t lo = S.r - S.k;
  const uint32_t* draws = L.s.draws + S.samp_off;
  const uint32_t* first = L.s.first + S.first_off;
  const uint32_t j0 = lo + i;
  const uint32_t t0 = draws[i];
  uint32_t j = j0, t = t0;
  bool present;
  // bounded by the chain's strict descent (at most k links)
  for (uint32_t guard = 0; ; ++guard) {
    if (first_of(first, S.first_mask, t) != j) { present = true; break; }   // an earlier iteration drew t
    if (t < lo || t == j || guard > S.k) { present = false; break; }
    j = t;                                                  // t was inserted iff iteration t collided
    t = draws[j - lo];
  }
  const uint32_t chosen = present ? j0 : t0;
  atomicOr(&L.s.sel[S.sel_off + (chosen >> 5)], 1u << (chosen & 31u));
}

// Exclusive prefix of the bitmap's popcounts.  A block owns kSelChunk consecutive words of one slice:
// k_sel_count sums the chunk's popcounts (not launched while every bitmap is a single chunk, r <= 262144),
// k_sel_scan adds the totals of the earlier chunks and scans inside the chunk (8 consecutive words per thread).
// grid of both: (ceil(most bitmap words of a slice / kSelChunk), n_slices); blk_tot is [n_slices][gridDim.x]
constexpr int kScanThreads = 1024;
constexpr int kSelPer = 8;
constexpr int kSelChunk = kScanThreads * kSelPer;

__global__ void __launch_bounds__(kScanThreads) k_sel_count(Launch L) {
  __shared__ uint32_t s_warp[32];
  const Slice S = L.s.slices[blockIdx.y];
  if (S.k == S.r) return;
  const uint32_t nwords = (S.r + 31u) >> 5;
  const uint32_t w0 = blockIdx.x * (uint32_t)kSelChunk + threadIdx.x * (uint32_t)kSelPer;
  if (blockIdx.x * (uint32_t)kSelChunk >= nwords) return;
  const uint32_t* sel = L.s.sel + S.sel_off;
  uint32_t c = 0;
#pragma unroll
  for (int u = 0; u < kSelPer; ++u) if (w0 + u < nwords) c += __popc(sel[w0 + u]);
  c = warp_sum(c);
  if ((threadIdx.x & 31) == 0) s_warp[threadIdx.x >> 5] = c;
  __syncthreads();
  if (threadIdx.x < 32) {
    const uint32_t t = warp_sum(s_warp[threadIdx.x]);
    if (threadIdx.x == 0) L.s.sel_blk[blockIdx.y * gridDim.x + blockIdx.x] = t;
  }
}

__global__ void __launch_bounds__(kScanThreads) k_sel_scan(Launch L) {
  __shared__ uint32_t s_warp[32];
  __shared__ uint32_t s_base;
  const Slice S = L.s.slices[blockIdx.y];
  if (S.k == S.r) return;
  const uint32_t nwords = (S.r + 31u) >> 5;
  if (blockIdx.x * (uint32_t)kSelChunk >= nwords) return;
  const uint32_t tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  // selected positions in the chunks before mine
  uint32_t before = 0;
  for (uint32_t b = tid; b < blockIdx.x; b += kScanThreads) before += L.s.sel_blk[blockIdx.y * gridDim.x + b];
  before = warp_sum(before);
  if (lane == 0) s_warp[warp] = before;
  __syncthreads();
  if (warp == 0) {
    const uint32_t t = warp_sum(s_warp[lane]);
    if (lane == 0) s_base = t;
  }
  __syncthreads();
  const uint32_t* sel = L.s.sel + S.sel_off;
  uint32_t* pre = L.s.sel_pre + S.sel_off;
  const uint32_t w0 = blockIdx.x * (uint32_t)kSelChunk + tid * (uint32_t)kSelPer;
  uint32_t cnt[kSelPer], mine = 0;
#pragma unroll
  for (int u = 0; u < kSelPer; ++u) { cnt[u] = w0 + u < nwords ? __popc(sel[w0 + u]) : 0u; mine += cnt[u]; }
  const uint32_t incl = warp_incl_scan(mine);
  __syncthreads();                                             // s_warp is free again
  if (lane == 31) s_warp[warp] = incl;
  __syncthreads();
  uint32_t run = s_base + incl - mine;
  for (uint32_t w = 0; w < warp; ++w) run += s_warp[w];
#pragma unroll
  for (int u = 0; u < kSelPer; ++u) {
    if (w0 + u < nwords) pre[w0 + u] = run;
    run += cnt[u];
  }
}

// The context's round counter (RTOPK_OPT_DEVICE_STEP): set, and advanced by one at the end of a call.
__global__ void k_step_set(uint32_t* word, uint32_t value) { if (blockIdx.x == 0 && threadIdx.x == 0) *word = value; }
__global__ void k_step_bump(uint32_t* word) { if (blockIdx.x == 0 && threadIdx.x == 0) *word += 1u; }

// Expands one slice's bitmap into the ascending list of chosen positions.
__global__ void __launch_bounds__(kThreads) k_positions(Launch L, uint32_t* pos) {
  const Slice S = L.s.slices[0];
  const uint32_t w = blockIdx.x * kThreads + threadIdx.x;
  const uint32_t nwords = (S.r + 31u) >> 5;
  if (w >= nwords) return;
  uint32_t word, pre;
  if (S.k == S.r) {
    word = (w + 1 == nwords && (S.r & 31u)) ? ((1u << (S.r & 31u)) - 1u) : 0xFFFFFFFFu;
    pre = w * 32u;
  } else {
    word = L.s.sel[S.sel_off + w];
    pre = L.s.sel_pre[S.sel_off + w];
  }
  while (word) {
    const uint32_t b = __ffs(word) - 1;
    word &= word - 1;
    if (pre < S.k) pos[pre] = w * 32u + b;
    ++pre;
  }
}

}  // namespace rtopk
