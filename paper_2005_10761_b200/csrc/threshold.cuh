// Threshold-then-subsample encoder: the scheme in the proof of Theorem 1, for real-valued vectors
// as Section II describes it for continuous observations (quantise by magnitude at a threshold,
// then subsample the marked coordinates).
//
// The streaming pass (k_stream) is the same as for rTop-k, with the fixed threshold in place of a
// sampled bracket: it forms a = g + m, writes it back and gathers every coordinate whose magnitude
// exceeds theta into per-chunk runs.  What differs comes after it: the size of the marked set is
// only known on the device, so
//   k_thr_init    sets the slices' gather threshold and clears the streaming pass's counters;
//   k_thr_sizes   reads the number of marked coordinates ||X||_1 of each worker, turns the slice
//                 into a "k' of ||X||_1" subset problem for the sampler kernels (or "all of them"
//                 when ||X||_1 <= k'), numbers the chunks' runs in index order and pads the message;
//   k_thr_emit    walks the runs: a marked coordinate's position in index order is its run's first
//                 position plus its place in the run; the ones the subset holds become (index,
//                 value) messages -- the value a_i, or sign(a_i) * 2 theta in sign mode -- and their
//                 residual slots keep what was not sent (Algorithm 1's m' = a - ghat: zero, or the
//                 difference in sign mode).
#pragma once

#include "common.cuh"
#include "select.cuh"

namespace rtopk {

constexpr int kThrThreads = 256;
constexpr int kThrSizeThreads = 1024;
constexpr uint32_t kThrPadIndex = 0xFFFFFFFFu;   // index of an unused message slot

// grid: n_slices.  gather_key: keys >= gather_key are marked (bit pattern of theta, plus one).
__global__ void __launch_bounds__(kThrThreads) k_thr_init(Launch L, uint32_t gather_key) {
  const uint32_t sl = blockIdx.x;
  const Slice S = L.s.slices[sl];
  clear_slice_counters(L, sl, S, 0, 1);
  if (threadIdx.x == 0) {
    SelState st;
    st.tau_lo = gather_key; st.eq_quota = kNoQuota; st.prefix = gather_key - 1u; st.resolved = 31;
    st.n_gt = 0; st.need = 0; st.n_cand = 0; st.stage = STAGE_DONE; st.flags = 0; st.n_cand_first = 0;
    st.tau_hi = 0x7FFFFFFFu; st.pred = 0;
    L.s.state[sl] = st;
  }
}

// grid: n_slices (one slice per worker row).  `limit` is the largest marked set the scratch holds,
// `k` the message capacity k'.  Rewrites the slice's (r, k) in the device table to
// (||X||_1, min(||X||_1, k')), which is what the subset kernels and k_thr_emit read.
__global__ void __launch_bounds__(kThrSizeThreads) k_thr_sizes(Launch L, uint32_t limit, uint32_t k,
                                                               uint32_t* __restrict__ msg_count,
                                                               uint32_t* __restrict__ msg_ones) {
  __shared__ uint32_t s_warp[kThrSizeThreads / 32];
  const uint32_t sl = blockIdx.x, tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const Slice S = L.s.slices[sl];
  const uint32_t ones = L.s.cursor[sl];
  uint32_t n = ones;
  if (ones > limit || ones > S.cand_cap) {           // more marked coordinates than the scratch holds:
    n = 0;                                           // the worker sends nothing, everything stays in m
    if (tid == 0) atomicOr(L.s.error, ERR_CANDIDATE_OVERFLOW);
  }
  const uint32_t count = min(n, k);
  // first position (in index order) of every chunk's run: exclusive prefix of the run lengths
  const uint32_t nchunks = slice_chunks(S);
  const uint32_t per = (nchunks + kThrSizeThreads - 1) / kThrSizeThreads;
  const uint32_t c0 = min(nchunks, tid * per), c1 = min(nchunks, c0 + per);
  const uint32_t* ccount = L.s.chunk_count + S.chunk_begin;
  uint32_t* cpre = L.s.chunk_pre + S.chunk_begin;
  uint32_t mine = 0;
  for (uint32_t c = c0; c < c1; ++c) mine += ccount[c];
  const uint32_t incl = warp_incl_scan(mine);
  if (lane == 31) s_warp[warp] = incl;
  __syncthreads();
  uint32_t run = incl - mine;
  for (uint32_t w = 0; w < warp; ++w) run += s_warp[w];
  for (uint32_t c = c0; c < c1; ++c) { cpre[c] = run; run += ccount[c]; }
  // unused message slots
  for (uint32_t j = count + tid; j < k; j += kThrSizeThreads) {
    L.msg_idx[S.msg_off + j] = kThrPadIndex;
    L.msg_val[S.msg_off + j] = 0.0f;
  }
  __syncthreads();                                   // every thread has read the slice before it changes
  if (tid == 0) {
    L.s.slices[sl].r = n;
    L.s.slices[sl].k = count;
    L.s.state[sl].n_cand = ones;
    L.s.state[sl].n_cand_first = ones;
    L.s.state[sl].n_gt = n;
    msg_count[S.row] = count;
    msg_ones[S.row] = ones;
  }
}

// grid: (ceil(most chunks of a slice / warps per block), n_slices); one warp per chunk.
// signs != 0: a kept coordinate carries sign(a) * M (Section II: after the quantisation an observation
// is 0 or +-M) and its residual slot keeps a - sign(a) * M, one binary32 subtraction (a NaN difference
// is stored as the default quiet NaN, like a NaN sum).
__global__ void __launch_bounds__(kThrThreads) k_thr_emit(Launch L, uint32_t signs, float M) {
  const uint32_t sl = blockIdx.y;
  const Slice S = L.s.slices[sl];
  const uint32_t lane = threadIdx.x & 31u;
  const uint32_t c = blockIdx.x * (kThrThreads / 32) + (threadIdx.x >> 5);
  if (S.r == 0 || c >= slice_chunks(S)) return;
  const uint32_t tile = S.chunk_begin + c;
  const uint32_t n = L.s.chunk_count[tile];
  if (n == 0) return;
  const uint32_t first = L.s.chunk_pre[tile], src = L.s.chunk_start[tile];
  const uint32_t* ridx = L.s.raw_idx + S.cand_off + src;
  const float* rval = L.s.raw_val + S.cand_off + src;
  const bool all = S.k == S.r;
  for (uint32_t e = lane; e < n; e += 32u) {
    const uint32_t p = first + e;                    // position among the marked coordinates
    if (p >= S.r) break;
    uint32_t slot = p;
    if (!all) {
      const uint32_t word = L.s.sel[S.sel_off + (p >> 5)];
      if (!((word >> (p & 31u)) & 1u)) continue;
      slot = L.s.sel_pre[S.sel_off + (p >> 5)] + __popc(word & ((1u << (p & 31u)) - 1u));
    }
    if (slot >= S.k) continue;
    const uint32_t idx = ridx[e];
    const float a = rval[e];
    float sent = a, rest = 0.0f;
    if (signs) {
      sent = __uint_as_float((__float_as_uint(a) & 0x80000000u) | __float_as_uint(M));
      rest = __fsub_rn(a, sent);
      if (rest != rest) rest = __uint_as_float(0x7FC00000u);
    }
    L.msg_idx[S.msg_off + slot] = S.idx_base + idx;
    L.msg_val[S.msg_off + slot] = sent;
    L.residual[S.m_off + idx] = rest;
  }
}

}  // namespace rtopk
