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

// grid: (ceil(k_max / kDrawThreads), n_slices)
__global__ void __launch_bounds__(kDrawThreads) k_draw(Launch L) {
  const Slice S = L.s.slices[blockIdx.y];
  if (S.k == S.r) return;
  const uint32_t i = blockIdx.x * kDrawThreads + threadIdx.x;
  if (i >= S.k) return;
  const uint32_t j = S.r - S.k + i;
  const uint32_t t = floyd_draw(j, L.worker_base + S.row, S.segment, L.step, L.seed_lo, L.seed_hi);
  L.s.draws[S.samp_off + i] = t;
  atomicMin(&L.s.first[S.first_off + t], j);
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
    if (first[t] != j) { present = true; break; }          // an earlier iteration drew t
    if (t < lo || t == j || guard > S.k) { present = false; break; }
    j = t;                                                  // t was inserted iff iteration t collided
    t = draws[j - lo];
  }
  const uint32_t chosen = present ? j0 : t0;
  atomicOr(&L.s.sel[S.sel_off + (chosen >> 5)], 1u << (chosen & 31u));
}

// Exclusive prefix of the bitmap's popcounts, one block per slice.
constexpr int kScanThreads = 1024;
__global__ void __launch_bounds__(kScanThreads) k_sel_scan(Launch L) {
  __shared__ uint32_t s_warp[32];
  __shared__ uint32_t s_carry, s_total;
  const Slice S = L.s.slices[blockIdx.x];
  if (S.k == S.r) return;
  const uint32_t nwords = (S.r + 31u) >> 5;
  const uint32_t* sel = L.s.sel + S.sel_off;
  uint32_t* pre = L.s.sel_pre + S.sel_off;
  const uint32_t tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  if (tid == 0) s_carry = 0;
  __syncthreads();
  for (uint32_t base = 0; base < nwords; base += kScanThreads) {
    const uint32_t w = base + tid;
    const uint32_t c = w < nwords ? __popc(sel[w]) : 0u;
    const uint32_t incl = warp_incl_scan(c);
    if (lane == 31) s_warp[warp] = incl;
    __syncthreads();
    if (warp == 0) {
      const uint32_t v = s_warp[lane];
      const uint32_t vi = warp_incl_scan(v);
      s_warp[lane] = vi - v;
      if (lane == 31) s_total = vi;
    }
    __syncthreads();
    const uint32_t carry = s_carry;
    if (w < nwords) pre[w] = carry + s_warp[warp] + incl - c;
    __syncthreads();
    if (tid == 0) s_carry = carry + s_total;
    __syncthreads();
  }
}

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
