// Top-r selection kernels (Definition 1 with the lower-index tie rule), fused with the
// error-feedback add of Algorithm 1 (a = g + m, written back into the residual buffer).
//
//   k_sample        brackets the r-th largest key of every slice from a strided sample of a = g + m
//                   (or, with threshold reuse, from the slice's last exact thresholds) and clears
//                   the counters of the streaming pass (k_stream, stream.cuh)
//   k_bracket       the same bracket from a histogram of the 11 leading key bits over the whole slice
//                   instead of a sample, when the caller asks for it (one more pass over g and m)
//   k_finish        one cluster per slice: candidate runs -> index order, exact r-th largest key
//                   among the candidates, then a walk over the candidates in index order that
//                   numbers the members of the top-r set and writes the ones the k-of-r sampler
//                   chose as (index, value) messages, zeroing their residual slots (m' = a - ghat);
//                   a slice whose bracket missed is first selected exactly over all of its a = g + m
//                   inside the cluster (cluster_exact_collect)
//   k_emit_all      r = d (Definition 2): positions are indices, no selection
#pragma once

#include <cooperative_groups.h>

#include "common.cuh"
#include "element.cuh"

namespace rtopk {

__device__ __forceinline__ uint32_t slice_chunks(const Slice& S) {
  return (S.head + S.len + kChunk - 1) / kChunk;
}

// Clears the counters of slice `sl` that the streaming pass, the run kernels and the exact path expect
// to be zero (run cursor, block counter, list length, chunk-group totals, the histogram over the bracket;
// plus the launch-wide tickets).  The sampling
// kernels do this instead of a memset node in front of them; `part` of `nparts` thread blocks of
// blockDim.x threads share the work.
__device__ __forceinline__ void clear_slice_counters(const Launch& L, uint32_t sl, const Slice& S, uint32_t part, uint32_t nparts) {
  const uint32_t t = part * blockDim.x + threadIdx.x, nt = nparts * blockDim.x;
  const uint32_t nchunks = slice_chunks(S);
  const uint32_t ngroups = (nchunks + (1u << S.gshift) - 1u) >> S.gshift;
  for (uint32_t g = t; g < ngroups; g += nt) L.s.group_total[S.group_begin + g] = 0;
  for (uint32_t b = t; b < (uint32_t)kBins; b += nt) L.s.hist[(size_t)sl * kBins + b] = 0;
  if (t == 0) { L.s.cursor[sl] = 0; L.s.done[sl] = 0; L.s.fin[sl].list_n = 0; L.s.fin[sl].done2 = 0; }
  if (sl == 0 && t < 4u) L.s.tickets[t] = 0;
}

// ----------------------------------------------------------------------------- state init
__global__ void k_init_state(Launch L, uint32_t general) {
  const uint32_t s = blockIdx.x * blockDim.x + threadIdx.x;
  if (s >= L.n_slices) return;
  const Slice S = L.s.slices[s];
  SelState st;
  st.tau_lo = 0x80000000u;           // above every key: nothing is a candidate
  st.eq_quota = kNoQuota;
  st.prefix = 0; st.n_gt = 0; st.need = S.r; st.n_cand = 0; st.n_cand_first = 0;
  st.tau_hi = 0x7FFFFFFFu; st.pred = 0;
  if (S.r == S.len) { st.resolved = 31; st.stage = STAGE_DONE; st.flags = 0; }   // top-r is everything
  else { st.resolved = 0; st.stage = STAGE_PASS0; st.flags = general ? FLAG_GENERAL : 0u; }
  L.s.state[s] = st;
  L.s.fin[s].list_n = 0; L.s.fin[s].done2 = 0;
}

// ----------------------------------------------------------------------------- sampled threshold
// One block per slice.  Reads up to kSampleMax coordinates of a = g + m in 128-byte groups spread
// evenly over the slice and brackets the r-th largest key from below (tau_lo: the keys >= tau_lo
// must number at least r) and from above (tau_hi).  The streaming pass gathers the keys >= tau_lo
// and counts them; a miss is repaired by the exact path, and a tau_hi that is too low only costs
// k_finish one more round, so the estimates affect speed, never the result.
//
// Both sample ranks are small (about 1.4 % of the sample), so the bulk is never histogrammed: every
// thread keeps only the maximum of each group of 4 sampled keys, and the rho-th largest of these
// 8192 maxima is a lower bound of the rho-th largest key (there are at least rho keys that large;
// with groups this small the bound is within a few per cent of the exact sample rank).  tau_lo is that bound at
// rank expect + 4.5 sigma; tau_hi the same at rank (expect - 4.5 sigma) * 3/4, which as a sample rank
// stays clearly above the r-th largest.  Samples whose ranks exceed the thread count take a radix
// select over all sample keys instead.
constexpr int kSampleHold = 8;   // maxima a thread keeps (one per 4 sampled keys)

// Two ranks at once in two histograms of kBins bins whose totals stay below 2^16 (ha == hb is
// allowed): the counts travel packed, a's in the low and b's in the high half of a word, so one
// block scan serves both.  For each: the digit D with count(> D) < need <= count(>= D), and
// count(> D).  Called by all kSampleThreads threads; scratch holds 32 + 4 words.  A digit of
// 0xFFFFFFFF means the histogram holds fewer than `need` keys.
__device__ __forceinline__ void pick_two(const uint32_t* ha, const uint32_t* hb, uint32_t need_a, uint32_t need_b,
                                         uint32_t* scratch, uint32_t& Da, uint32_t& above_a, uint32_t& Db, uint32_t& above_b) {
  static_assert(kBins == 2 * kSampleThreads, "two bins per thread");
  const uint32_t tid = threadIdx.x, lane = tid & 31u, warp = tid >> 5;
  const int hi = kBins - 1 - 2 * (int)tid;                      // thread 0 holds the largest digits
  const uint32_t p0 = ha[hi] | (hb[hi] << 16), p1 = ha[hi - 1] | (hb[hi - 1] << 16);
  const uint32_t mine = p0 + p1;
  uint32_t incl = warp_incl_scan(mine);
  if (lane == 31) scratch[warp] = incl;
  if (tid == 0) { scratch[32] = 0xFFFFFFFFu; scratch[33] = 0; scratch[34] = 0xFFFFFFFFu; scratch[35] = 0; }
  __syncthreads();
  {
    const uint32_t wt = scratch[lane];
    const uint32_t wincl = warp_incl_scan(wt);
    incl += __shfl_sync(0xFFFFFFFFu, wincl - wt, warp);
  }
  const uint32_t excl = incl - mine;
  {
    const uint32_t ex = excl & 0xFFFFu, in = incl & 0xFFFFu, h0 = p0 & 0xFFFFu;
    if (ex < need_a && need_a <= in) {
      if (ex + h0 >= need_a) { scratch[32] = (uint32_t)hi; scratch[33] = ex; }
      else { scratch[32] = (uint32_t)(hi - 1); scratch[33] = ex + h0; }
    }
  }
  {
    const uint32_t ex = excl >> 16, in = incl >> 16, h0 = p0 >> 16;
    if (ex < need_b && need_b <= in) {
      if (ex + h0 >= need_b) { scratch[34] = (uint32_t)hi; scratch[35] = ex; }
      else { scratch[34] = (uint32_t)(hi - 1); scratch[35] = ex + h0; }
    }
  }
  __syncthreads();
  Da = scratch[32]; above_a = scratch[33]; Db = scratch[34]; above_b = scratch[35];
}

// The rank_a-th and rank_b-th largest (1-based) of the held keys of all threads, to 22 of the 31
// key bits: slot u of thread t is in use iff t + u * blockDim.x < n_held (fewer than 2^16 in all).
// pa <= the rank_a-th largest key <= pa + 511, and the same for pb.  Two radix passes of at most
// kSampleHold (then 2 * kSampleHold) shared-memory increments per thread; hist holds 2 * kBins words.
__device__ __forceinline__ void block_select_two(const uint32_t (&key)[kSampleHold], uint32_t n_held,
                                                 uint32_t rank_a, uint32_t rank_b, uint32_t* hist, uint32_t* scratch,
                                                 uint32_t& pa, uint32_t& pb) {
  const uint32_t tid = threadIdx.x;
  uint32_t* ha = hist;
  uint32_t* hb = hist + kBins;
  for (uint32_t b = tid; b < 2u * kBins; b += blockDim.x) hist[b] = 0;
  __syncthreads();
#pragma unroll
  for (int u = 0; u < kSampleHold; ++u)
    if (tid + u * blockDim.x < n_held) atomicAdd(&ha[key[u] >> 20], 1u);
  __syncthreads();
  uint32_t Da, Db, above_a, above_b;
  pick_two(ha, ha, rank_a, rank_b, scratch, Da, above_a, Db, above_b);
  const uint32_t need_a = rank_a - above_a, need_b = rank_b - above_b;
  __syncthreads();                                               // everyone has read pass 0's result
  for (uint32_t b = tid; b < (uint32_t)kBins; b += blockDim.x) ha[b] = 0;
  __syncthreads();
#pragma unroll
  for (int u = 0; u < kSampleHold; ++u)
    if (tid + u * blockDim.x < n_held) {
      const uint32_t top = key[u] >> 20, next = (key[u] >> 9) & 0x7FFu;
      if (top == Da) atomicAdd(&ha[next], 1u);
      if (top == Db) atomicAdd(&hb[next], 1u);
    }
  __syncthreads();
  uint32_t Ea, Eb;
  pick_two(ha, hb, need_a, need_b, scratch, Ea, above_a, Eb, above_b);
  pa = Da == 0xFFFFFFFFu || Ea == 0xFFFFFFFFu ? 0u : ((Da << 11) | Ea) << 9;
  pb = Db == 0xFFFFFFFFu || Eb == 0xFFFFFFFFu ? 0x7FFFFE00u : ((Db << 11) | Eb) << 9;
}

template <typename GradT>
__global__ void __launch_bounds__(kSampleThreads) k_sample(Launch L) {
  extern __shared__ uint32_t smem[];
  uint32_t* keys = smem;                       // [kSampleMax]
  uint32_t* hist = smem + kSampleMax;          // [2 * kBins]
  uint32_t* scratch = hist + 2 * kBins;        // [64]
  const uint32_t sl = blockIdx.x;
  const Slice S = L.s.slices[sl];
  const uint32_t tid = threadIdx.x;
  clear_slice_counters(L, sl, S, 0, 1);
  SelState st;
  st.eq_quota = kNoQuota; st.prefix = 0; st.resolved = 0; st.n_gt = 0; st.need = S.r;
  st.n_cand = 0; st.n_cand_first = 0; st.stage = STAGE_PASS0; st.flags = 0; st.tau_hi = 0x7FFFFFFFu; st.pred = 0;
  if (S.r == S.len) {
    st.tau_lo = 0x80000000u; st.resolved = 31; st.stage = STAGE_DONE;
    if (tid == 0) L.s.state[sl] = st;
    return;
  }
  if (L.reuse) {
    // Step-to-step reuse: a = g + m changes slowly from one round to the next, so the last two exact
    // thresholds predict this one.  Only a smooth history is trusted (two thresholds within 25 % of
    // each other: while a fresh residual builds up the threshold still jumps, and sampling costs far
    // less than a miss); a ratio beyond 5 % is damped to its square root, because a threshold that
    // moves that fast is slowing down, and a prediction that is too low only adds candidates whereas
    // one that is too high misses.  The bracket is the prediction widened by a few times the error
    // the predictions have shown so far.  A bracket that misses is repaired by the exact path and
    // makes the next two calls sample again.
    const TauHistory h = L.s.history[sl];                       // the same for every thread
    if (h.valid >= 2 && h.tau1 > 0x00800000u && h.tau1 < 0x7E800000u && h.tau2 > 0x00800000u && h.tau2 < 0x7E800000u) {
      const float t1 = __uint_as_float(h.tau1);
      float ratio = t1 / __uint_as_float(h.tau2);
      if (ratio >= 0.8f && ratio <= 1.25f) {
        if (ratio < 0.95f || ratio > 1.05f) ratio = sqrtf(ratio);
        const float p = t1 * ratio;
        const float delta = fminf(fmaxf(3.0f * h.err + 0.01f, 0.02f), 0.15f);
        st.tau_lo = mag_key(p * (1.0f - delta));
        st.tau_hi = max(mag_key(p * (1.0f + delta)), st.tau_lo);
        st.pred = mag_key(p);
        if (tid == 0) L.s.state[sl] = st;
        return;
      }
    }
  }
  const float* m = L.residual;
  uint32_t n_s, rho_lo, rho_hi, n_held;
  uint32_t mine[kSampleHold];
#pragma unroll
  for (int u = 0; u < kSampleHold; ++u) mine[u] = 0;
  if (S.len <= (uint32_t)kSampleMax) {
    n_s = S.len; rho_lo = S.r; rho_hi = max(1u, S.r - S.r / 4u);   // the sample is the whole slice
    n_held = min(n_s, (uint32_t)(kSampleHold * kSampleThreads));
#pragma unroll
    for (int u = 0; u < kSampleMax / kSampleThreads; ++u) {        // slot u % kSampleHold
      const uint32_t i = tid + u * kSampleThreads;
      if (i < n_s) {
        const uint32_t key = mag_key(ef_add(Grad<GradT>::ld1(L.grad, S.g_off + i), m[S.m_off + i]));
        keys[i] = key;
        mine[u % kSampleHold] = max(mine[u % kSampleHold], key);
      }
    }
  } else {
    const uint32_t v0 = (S.head + 3u) >> 2, v1 = (S.head + S.len) >> 2;   // fully valid vectors
    const uint32_t ngroups_avail = (v1 - v0) >> 3;
    const uint32_t G = min((uint32_t)(kSampleMax / 32), ngroups_avail);
    n_s = G * 32u;
    const int64_t base_g = S.g_off - S.head, base_m = S.m_off - S.head;
    // all of a thread's sample loads are issued before the first use (one memory latency in total)
    constexpr int kPer = kSampleMax / 4 / kSampleThreads;
    static_assert(kPer == kSampleHold, "one held maximum per sampled vector");
    n_held = G * 8u;
    float4 g4[kPer], m4[kPer];
#pragma unroll
    for (int u = 0; u < kPer; ++u) {
      const uint32_t n = tid + u * kSampleThreads;
      if (n < G * 8u) {
        const uint32_t gi = n >> 3, vv = n & 7u;
        // group gi of G sits at floor(gi * avail / G); G is 1024 whenever avail >= 1024, else avail
        const uint32_t grp = G == (uint32_t)(kSampleMax / 32) ? (uint32_t)(((uint64_t)gi * ngroups_avail) >> 10) : gi;
        const uint32_t vec = v0 + grp * 8u + vv;
        g4[u] = Grad<GradT>::ld4(L.grad, base_g + (int64_t)vec * 4);
        m4[u] = __ldg(reinterpret_cast<const float4*>(m + base_m + (int64_t)vec * 4));
      }
    }
#pragma unroll
    for (int u = 0; u < kPer; ++u) {
      const uint32_t n = tid + u * kSampleThreads;
      if (n < G * 8u) {
        const uint32_t k0 = mag_key(ef_add(g4[u].x, m4[u].x)), k1 = mag_key(ef_add(g4[u].y, m4[u].y));
        const uint32_t k2 = mag_key(ef_add(g4[u].z, m4[u].z)), k3 = mag_key(ef_add(g4[u].w, m4[u].w));
        keys[n * 4 + 0] = k0; keys[n * 4 + 1] = k1; keys[n * 4 + 2] = k2; keys[n * 4 + 3] = k3;
        mine[u] = max(max(k0, k1), max(k2, k3));
      }
    }
    const float expect = (float)n_s * ((float)S.r / (float)S.len);
    const float margin = 4.5f * sqrtf(expect) + 4.0f;             // a miss (about 3e-6 per slice) costs one exact pass
    rho_lo = expect + margin >= (float)n_s ? n_s : (uint32_t)(expect + margin);
    rho_hi = expect - margin < 2.0f ? 1u : (uint32_t)((expect - margin) * 0.75f);
  }
  __syncthreads();
  uint32_t tau_lo, tau_hi;
  if (rho_lo <= n_held) {
    // 22 of the 31 key bits are enough for estimates: tau_lo rounds down, tau_hi up
    block_select_two(mine, n_held, rho_lo, rho_hi, hist, scratch, tau_lo, tau_hi);
    tau_hi |= 0x1FFu;
  } else {
    // radix select of the rho_lo-th largest over all sample keys; no upper estimate
    uint32_t prefix = 0, need = rho_lo;
    for (int pass = 0; pass < 3; ++pass) {
      const int bits = digit_bits(pass), shift = digit_shift(pass);
      for (uint32_t b = tid; b < (uint32_t)kBins; b += kSampleThreads) hist[b] = 0;
      __syncthreads();
      for (uint32_t i = tid; i < n_s; i += kSampleThreads) {
        const uint32_t key = keys[i];
        if (pass == 0 || (key >> (shift + bits)) == prefix) atomicAdd(&hist[(key >> shift) & ((1u << bits) - 1u)], 1u);
      }
      __syncthreads();
      uint32_t D, above;
      pick_digit(hist, 1 << bits, need, scratch, D, above);
      need -= above;
      prefix = (prefix << bits) | D;
    }
    tau_lo = prefix; tau_hi = 0x7FFFFFFFu;
  }
  st.tau_lo = tau_lo;
  st.tau_hi = max(tau_hi, tau_lo);
  if (tid == 0) L.s.state[sl] = st;
}

__device__ __forceinline__ bool is_last_block(uint32_t* counter, uint32_t nblocks) {
  __shared__ uint32_t s_last;
  __syncthreads();
  if (threadIdx.x == 0) {
    __threadfence();
    s_last = (atomicAdd(counter, 1u) == nblocks - 1u);
  }
  __syncthreads();
  if (s_last) __threadfence();
  return s_last != 0;
}

// Did the sampled pass gather too few or too many candidates for this slice?  (The slice's cursor
// is the number of candidates the stream pass reserved room for.)
__device__ __forceinline__ bool first_pass_missed(uint32_t n_gathered, const Slice& S) {
  return S.r < S.len && (n_gathered < S.r || n_gathered > S.cand_cap);
}

// The bracket of the r-th largest key from a histogram instead of a sample (RTOPK_OPT_SELECT_PATH = 1): one
// pass reads g and m, forms a = g + m (nothing is stored: the streaming pass does that) and counts the 11
// leading bits of every key; the last block of a slice picks the bucket that holds the r-th largest key, and
// the bucket's bounds are the bracket.  It cannot miss; the streaming pass then gathers the keys of this
// bucket and above -- more than a sampled bracket would let through, and more than the candidate list
// holds when very many keys share 11 leading bits, which the finishing kernels repair like any overflow.
// grid: up to total_blocks blocks; a unit is kHistChunks chunks of one slice.
template <typename GradT>
__global__ void __launch_bounds__(kThreads, 8) k_bracket(Launch L, uint32_t total_blocks) {
  __shared__ uint32_t hist_s[kBins];
  __shared__ uint32_t scratch[kWarps + 2];
  const uint32_t tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const Slice* slices = L.s.slices;
  for (uint32_t unit = blockIdx.x; unit < total_blocks; unit += gridDim.x) {
    __syncthreads();                                   // hist_s / scratch of the previous unit are free
    const uint32_t sl = find_slice(L.n_slices, unit, [&](uint32_t i) { return slices[i].hist_begin; });
    const Slice S = slices[sl];
    if (S.r == S.len) continue;                        // nothing to select
    for (uint32_t b = tid; b < (uint32_t)kBins; b += kThreads) hist_s[b] = 0;
    __syncthreads();
    const uint32_t nchunks = slice_chunks(S);
    const uint32_t hb = unit - S.hist_begin;
    const uint32_t c0 = hb * kHistChunks, c1 = min(nchunks, c0 + kHistChunks);
    const uint32_t span = S.head + S.len;
    const int64_t base_g = S.g_off - S.head, base_m = S.m_off - S.head;
    for (uint32_t c = c0; c < c1; ++c) {
      const uint32_t e_w = c * (uint32_t)kChunk + warp * (uint32_t)kWarpSpan;
      float a[kIter][4];
      uint32_t valid[kIter];
#pragma unroll
      for (int it = 0; it < kIter; ++it)
        valid[it] = load_vec<GradT, true, false>(L.grad, L.residual, base_g, base_m, e_w + it * 128u + lane * 4u,
                                                 S.head, span, a[it]);
#pragma unroll
      for (int it = 0; it < kIter; ++it)
#pragma unroll
        for (int j = 0; j < 4; ++j)
          if ((valid[it] >> j) & 1u) atomicAdd(&hist_s[mag_key(a[it][j]) >> 20], 1u);
    }
    __syncthreads();
    uint32_t* gh = L.s.hist + (size_t)sl * kBins;
    for (uint32_t b = tid; b < (uint32_t)kBins; b += kThreads) {
      const uint32_t v = hist_s[b];
      if (v) atomicAdd(gh + b, v);
    }
    const uint32_t nblocks = (nchunks + kHistChunks - 1) / kHistChunks;
    if (!is_last_block(&L.s.done[sl], nblocks)) continue;
    for (uint32_t b = tid; b < (uint32_t)kBins; b += kThreads) {
      hist_s[b] = __ldcg(gh + b);
      gh[b] = 0;                                         // the run kernels' histogram starts from zero
    }
    __syncthreads();
    uint32_t D, above;
    const bool ok = pick_digit(hist_s, kBins, S.r, scratch, D, above);
    if (tid == 0) {
      L.s.done[sl] = 0;
      SelState* st = &L.s.state[sl];
      if (ok) { st->tau_lo = D << 20; st->tau_hi = (D << 20) | 0xFFFFFu; }
      else atomicOr(L.s.error, ERR_SELECT_INCONSISTENT);   // fewer than r keys: cannot happen for a valid slice
    }
  }
}

// ----------------------------------------------------------------------------- finish
// One thread-block cluster per slice finishes the selection in a single launch:
//   1. the r-th largest key among the slice's candidates.  It lies in [lo_key, hi_key): after the
//      exact path that is the resolved radix bucket and n_gt counts the keys above it; after the
//      sampled pass it is [tau_lo, tau_hi] and the keys above are still uncounted.  Each round
//      spreads the interval over 2047 equal power-of-two buckets (the candidates are nearly uniform
//      over so narrow a range, so the shared-memory increments do not pile up on a few addresses)
//      plus one bucket for "above"; every CTA histograms its contiguous share, the CTAs read each
//      other's histograms through distributed shared memory and pick the bucket redundantly;
//   2. with tau and the tie quota known, every warp counts the members (key > tau, or key == tau)
//      in its contiguous part; the counts are exchanged, giving each warp its first position;
//   3. each warp walks its part in index order, numbers the members of the top-r set and writes the
//      ones the sampler chose as (index, value) messages, zeroing their residual slots.
constexpr int kMaxCluster = 16;
constexpr int kFinishThreads = 1024;
constexpr int kFinishWarps = kFinishThreads / 32;
constexpr int kFinishCache = 46 * 1024;   // candidate values a CTA keeps in shared memory (184 KB)
constexpr int kFinishBatch = 8;           // independent loads in flight per thread
constexpr int kFinishList = 2048;         // bucket population up to which the CTAs gather the bucket and finish on the list (fits hist / red)
constexpr int kFinishSelWords = 2048;     // bitmap words (64 Ki positions) a CTA keeps in shared memory

struct alignas(16) FinishSmem {           // the value cache behind it is read as float4
  uint32_t hist[kBins];
  uint32_t red[kBins];                 // the cluster's histogram, summed by every CTA for itself
  uint32_t sel[kFinishSelWords];       // the sampler's bitmap over this CTA's positions ...
  uint32_t sel_pre[kFinishSelWords];   // ... and its running popcount
  uint32_t scratch[kFinishWarps + 2];
  uint32_t counts[2 * kMaxCluster];    // (members above tau, equal to tau) of every CTA's share
  uint32_t warpA[kFinishWarps], warpB[kFinishWarps];
  uint32_t list_pre[kMaxCluster + 1];  // list round: exclusive prefix of the CTAs' list lengths
  uint32_t list_n, pad_;               // list round: my list length
};
static_assert(sizeof(FinishSmem) % 16 == 0, "the value cache must start 16-byte aligned");
constexpr size_t kFinishSmemBytes = sizeof(FinishSmem) + (size_t)kFinishCache * sizeof(float);

// 4-byte asynchronous copy global -> shared (no register holds the value in between) ...
__device__ __forceinline__ void async_copy_4(void* smem_dst, const void* gmem_src) {
  asm volatile("cp.async.ca.shared.global [%0], [%1], 4;" ::"r"((uint32_t)__cvta_generic_to_shared(smem_dst)), "l"(gmem_src) : "memory");
}
// ... and the wait for all such copies of the calling thread.
__device__ __forceinline__ void async_copy_wait_all() { asm volatile("cp.async.wait_all;" ::: "memory"); }

// The exact path inside the finishing cluster, for a slice whose first bracket missed (too few
// candidates gathered, or more than the list holds).  This is rare -- a sampled bracket misses about
// once in 10^5 slices, a predicted one after an abrupt change of the data -- so it is written for
// clarity, not speed: three radix passes over the slice's a = g + m (already materialised in the
// residual buffer by the streaming pass), each CTA histogramming its range of chunks and all CTAs
// summing the histograms through distributed shared memory, give the r-th largest key tau, the count
// n_gt of larger keys and the quota of keys equal to tau; an ordered sweep then writes exactly the
// top-r set (keys above tau, and the first `quota` keys equal to it) into the candidate list in index
// order.  Called by every thread of every CTA of the cluster; returns false (to all of them) if the
// slice holds fewer than r keys, which cannot happen for a valid slice.
template <typename Cluster>
__device__ __forceinline__ bool cluster_exact_collect(const Launch& L, const Slice& S, Cluster& cluster, FinishSmem& sm,
                                                      uint32_t CS, uint32_t q, uint32_t& tau_out, uint32_t& n_gt_out,
                                                      uint32_t& quota_out) {
  const uint32_t tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const uint32_t nchunks = slice_chunks(S);
  const uint32_t cpc = (nchunks + CS - 1) / CS;                       // chunks per CTA
  const uint32_t span = S.head + S.len;
  const uint32_t e_lo = max(S.head, min(span, q * cpc * (uint32_t)kChunk));
  const uint32_t e_hi = max(e_lo, min(span, (q + 1u) * cpc * (uint32_t)kChunk));
  const float* a = L.residual + (S.m_off - S.head);                   // element e of the slice's grid
  uint32_t prefix = 0, need = S.r, n_gt = 0;
  for (int pass = 0; pass < 3; ++pass) {
    const int bits = digit_bits(pass), shift = digit_shift(pass);
    for (uint32_t b = tid; b < (uint32_t)kBins; b += kFinishThreads) sm.hist[b] = 0;
    __syncthreads();
    for (uint32_t e = e_lo + tid; e < e_hi; e += kFinishThreads) {
      const uint32_t key = mag_key(a[e]);
      if (pass == 0 || (key >> (shift + bits)) == prefix) atomicAdd(&sm.hist[(key >> shift) & ((1u << bits) - 1u)], 1u);
    }
    cluster.sync();
    for (uint32_t b = tid; b < (uint32_t)kBins; b += kFinishThreads) {
      uint32_t sum = 0;
      for (uint32_t rr = 0; rr < CS; ++rr) sum += cluster.map_shared_rank(sm.hist, rr)[b];
      sm.red[b] = sum;
    }
    __syncthreads();
    uint32_t D, above;
    const bool ok = pick_digit(sm.red, 1 << bits, need, sm.scratch, D, above);
    cluster.sync();                                                    // all remote reads of sm.hist are done
    if (!ok) return false;                                             // the same in every CTA
    n_gt += above; need -= above;
    prefix = (prefix << bits) | D;
  }
  const uint32_t tau = prefix, quota = need;
  // members of my range: keys above tau (A) and keys equal to tau (B)
  uint32_t cA = 0, cB = 0;
  for (uint32_t e = e_lo + tid; e < e_hi; e += kFinishThreads) {
    const uint32_t key = mag_key(a[e]);
    cA += key > tau; cB += key == tau;
  }
  cA = warp_sum(cA); cB = warp_sum(cB);
  if (lane == 0) { sm.warpA[warp] = cA; sm.warpB[warp] = cB; }
  __syncthreads();
  if (tid < CS) {
    uint32_t tA = 0, tB = 0;
    for (int w = 0; w < kFinishWarps; ++w) { tA += sm.warpA[w]; tB += sm.warpB[w]; }
    uint32_t* c = cluster.map_shared_rank(sm.counts, tid);             // my counts, into CTA `tid`
    c[2 * q] = tA; c[2 * q + 1] = tB;
  }
  cluster.sync();
  uint32_t runA = 0, runB = 0;                                         // members before my range
  for (uint32_t p = 0; p < q; ++p) { runA += sm.counts[2 * p]; runB += sm.counts[2 * p + 1]; }
  // ordered sweep, 1024 consecutive elements at a time
  uint32_t* cidx = L.s.cand_idx + S.cand_off;
  float* cval = L.s.cand_val + S.cand_off;
  for (uint32_t base = e_lo; base < e_hi; base += kFinishThreads) {
    const uint32_t e = base + tid;
    const bool in = e < e_hi;
    const float v = in ? a[e] : 0.f;
    const uint32_t key = mag_key(v);
    const bool isA = in && key > tau, isB = in && key == tau;
    const uint32_t mA = __ballot_sync(0xFFFFFFFFu, isA), mB = __ballot_sync(0xFFFFFFFFu, isB);
    __syncthreads();                                                   // the previous tile's warp totals are consumed
    if (lane == 0) { sm.warpA[warp] = __popc(mA); sm.warpB[warp] = __popc(mB); }
    __syncthreads();
    uint32_t gA = runA + __popc(mA & ((1u << lane) - 1u)), gB = runB + __popc(mB & ((1u << lane) - 1u));
    uint32_t tA = 0, tB = 0;
    for (uint32_t w = 0; w < (uint32_t)kFinishWarps; ++w) {
      const uint32_t wa = sm.warpA[w], wb = sm.warpB[w];
      if (w < warp) { gA += wa; gB += wb; }
      tA += wa; tB += wb;
    }
    if (isA || (isB && gB < quota)) {
      const uint32_t pos = gA + min(gB, quota);
      if (pos < S.cand_cap) { cidx[pos] = e - S.head; cval[pos] = v; }
    }
    runA += tA; runB += tB;
  }
  __threadfence();
  cluster.sync();                                                      // the whole list is written and visible
  tau_out = tau; n_gt_out = n_gt; quota_out = quota;
  return true;
}

__global__ void __launch_bounds__(kFinishThreads) k_finish(Launch L) {
  namespace cg = cooperative_groups;
  extern __shared__ __align__(16) unsigned char finish_raw[];
  FinishSmem& sm = *reinterpret_cast<FinishSmem*>(finish_raw);
  float* cache = reinterpret_cast<float*>(finish_raw + sizeof(FinishSmem));
  cg::cluster_group cluster = cg::this_cluster();
  const uint32_t CS = cluster.num_blocks();                    // 1 .. kMaxCluster
  const uint32_t q = cluster.block_rank();
  const uint32_t sl = blockIdx.x / CS;
  const uint32_t tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const Slice S = L.s.slices[sl];
  SelState* st = &L.s.state[sl];
  // every early exit below depends on the slice only, so a cluster leaves as a whole
  if (S.r == S.len) return;
  if (st->flags & FLAG_FINISHED) return;                       // the run kernels have finished this slice
  bool general = (st->flags & FLAG_GENERAL) != 0;               // the list was built by the exact path
  uint32_t n_cand = general ? st->n_cand : L.s.cursor[sl];
  if (st->resolved > 31) return;                               // an earlier pass already failed
  uint32_t n_gt = st->n_gt, need = st->need, lo_key, hi_key;
  bool count_above;
  if (n_cand < S.r || n_cand > S.cand_cap) {
    // the first bracket missed (and no exact pass has repaired it): select exactly, here
    if (general) {                                             // cannot happen after an exact pass
      if (q == 0 && tid == 0) atomicOr(L.s.error, ERR_CANDIDATE_OVERFLOW);
      return;
    }
    uint32_t tau_x, gt_x, quota_x;
    if (!cluster_exact_collect(L, S, cluster, sm, CS, q, tau_x, gt_x, quota_x)) {
      if (q == 0 && tid == 0) { atomicOr(L.s.error, ERR_SELECT_INCONSISTENT); st->resolved = 32; }
      return;
    }
    if (q == 0 && tid == 0) { st->flags |= FLAG_GENERAL | FLAG_FELL_BACK; st->n_cand_first = n_cand; st->n_cand = S.r; }
    general = true; n_cand = S.r;
    n_gt = gt_x; need = quota_x; lo_key = tau_x; hi_key = tau_x + 1u; count_above = false;
  } else if (general) {
    const uint32_t free_bits = 31u - st->resolved;
    lo_key = st->prefix << free_bits; hi_key = lo_key + (1u << free_bits); count_above = false;
  } else {
    lo_key = st->tau_lo; hi_key = st->tau_hi + 1u; count_above = true; n_gt = 0; need = S.r;
    if (q == 0 && tid == 0) { st->n_cand = n_cand; st->n_cand_first = n_cand; }
  }
  // the slice's candidate list in index order: complete already after the exact path; after the
  // sampled pass this kernel builds its own part of it from the stream pass's runs
  uint32_t* cidx = L.s.cand_idx + S.cand_off;
  float* cval = L.s.cand_val + S.cand_off;
  const uint32_t per = ((n_cand + CS - 1) / CS + 31u) & ~31u;
  const uint32_t lo = min(n_cand, q * per), hi = min(n_cand, lo + per);
  const uint32_t n_mine = hi - lo;
  const uint32_t n_cached = min(n_mine, (uint32_t)kFinishCache);
  // a share of at most half the cache keeps its indices in shared memory as well (never written to
  // the global list); runs then reach the cache by asynchronous copies, all in flight at once
  const bool idx_cached = !general && n_mine <= (uint32_t)(kFinishCache / 2);
  uint32_t* cache_idx = reinterpret_cast<uint32_t*>(cache + kFinishCache / 2);

  if (general) {
    // my share of the candidate values -> shared memory (the share starts 128-byte aligned)
    const float4* src = reinterpret_cast<const float4*>(cval + lo);
    float4* dst = reinterpret_cast<float4*>(cache);
    const uint32_t nv = n_cached >> 2;
    for (uint32_t base = tid; base < nv; base += kFinishThreads * 4) {
      float4 v[4];
#pragma unroll
      for (int u = 0; u < 4; ++u) if (base + u * kFinishThreads < nv) v[u] = src[base + u * kFinishThreads];
#pragma unroll
      for (int u = 0; u < 4; ++u) if (base + u * kFinishThreads < nv) dst[base + u * kFinishThreads] = v[u];
    }
    for (uint32_t i = (nv << 2) + tid; i < n_cached; i += kFinishThreads) cache[i] = cval[lo + i];
  } else {
    // Runs -> my share.  The place of a run in index order is the number of candidates in earlier
    // chunks: the prefix over the chunk groups (summed by the stream pass) plus a warp scan inside
    // the group.  Places inside [lo, hi) are mine: the value goes to the shared-memory cache (to
    // the global list beyond the cache's size), the index to the global list.
    const uint32_t nchunks = slice_chunks(S), gsh = S.gshift;
    const uint32_t ngroups = (nchunks + (1u << gsh) - 1u) >> gsh;
    uint32_t* gpre = sm.hist;                                    // [ngroups + 1] exclusive prefix (hist + red)
    {
      static_assert(kGroupsMax == 2 * kFinishThreads && kGroupsMax + 1 <= 2 * kBins, "two groups per thread");
      static_assert(kFinishThreads == 1024 && kFinishWarps == 32, "a window is 1024 chunks, scanned by 32 warps");
      const uint32_t ga = 2u * tid, gb = 2u * tid + 1u;
      const uint32_t ta = ga < ngroups ? L.s.group_total[S.group_begin + ga] : 0u;
      const uint32_t tb = gb < ngroups ? L.s.group_total[S.group_begin + gb] : 0u;
      const uint32_t incl = warp_incl_scan(ta + tb);
      if (lane == 31) sm.warpA[warp] = incl;
      __syncthreads();
      uint32_t woff = 0;
      for (uint32_t w = 0; w < warp; ++w) woff += sm.warpA[w];
      if (ga < ngroups) gpre[ga + 1] = woff + incl - tb;
      if (gb < ngroups) gpre[gb + 1] = woff + incl;
      if (tid == 0) gpre[0] = 0;
      __syncthreads();
    }
    const uint32_t* cstart = L.s.chunk_start + S.chunk_begin;
    const uint32_t* ccount = L.s.chunk_count + S.chunk_begin;
    const uint32_t* ridx = L.s.raw_idx + S.cand_off;
    const float* rval = L.s.raw_val + S.cand_off;
    auto put = [&](uint32_t at, uint32_t i, float v) {          // candidate (i, v) belongs at place `at`
      cidx[at] = i;
      if (at - lo < n_cached) cache[at - lo] = v; else cval[at] = v;
    };
    uint32_t g0 = 0;
    if (n_mine > 0) {                                            // last group that starts at or before lo
      uint32_t g1 = ngroups;
      while (g1 - g0 > 1) { const uint32_t mid = (g0 + g1) >> 1; if (gpre[mid] <= lo) g0 = mid; else g1 = mid; }
    }
    if (n_mine > 0) {
      // Windows of kFinishThreads chunks (a whole number of groups: a group has at most as many
      // chunks as a window).  One thread per chunk: the first place and the source of its run go to
      // shared memory (block scan on top of the group prefix); then all threads copy the window's
      // places that lie inside [lo, hi), kFinishBatch gathers in flight each.
      uint32_t* dstTab = sm.sel;                                 // [1025] first place of each run of the window
      uint32_t* srcTab = sm.sel_pre;                             // [1024] where the run sits in the raw buffer
      const uint32_t gpw = 10u - gsh;                            // log2(groups per window)
      for (uint32_t wi = g0 >> gpw; (wi << 10) < nchunks && gpre[wi << gpw] < hi; ++wi) {
        const uint32_t c = (wi << 10) + tid;
        const bool has = c < nchunks;
        const uint32_t cnt = has ? __ldg(ccount + c) : 0u;
        const uint32_t src0 = has ? __ldg(cstart + c) : 0u;
        const uint32_t incl = warp_incl_scan(cnt);
        __syncthreads();                                         // the previous window's tables are free
        if (lane == 31) sm.warpA[warp] = incl;
        __syncthreads();
        uint32_t first = gpre[wi << gpw] + incl - cnt;
        {
          const uint32_t wt = sm.warpA[lane];
          const uint32_t wincl = warp_incl_scan(wt);
          first += __shfl_sync(0xFFFFFFFFu, wincl - wt, warp);
        }
        dstTab[tid] = first;
        srcTab[tid] = src0;
        if (tid == kFinishThreads - 1) dstTab[kFinishThreads] = first + cnt;
        __syncthreads();
        const uint32_t r_lo = max(lo, dstTab[0]), r_hi = min(hi, dstTab[kFinishThreads]);
        if (r_lo >= r_hi) continue;
        // the window's runs that reach into [r_lo, r_hi): j_lo .. j_hi (block-uniform searches)
        uint32_t j_lo = 0, j_hi = 0;
        {
          uint32_t c1 = kFinishThreads, d1 = kFinishThreads;
#pragma unroll
          for (int step = 0; step < 10; ++step) {
            const uint32_t ma = (j_lo + c1) >> 1, mb = (j_hi + d1) >> 1;
            if (dstTab[ma] <= r_lo) j_lo = ma; else c1 = ma;
            if (dstTab[mb] < r_hi) j_hi = mb; else d1 = mb;
          }
          ++j_hi;
        }
        // Copy the window's places inside [r_lo, r_hi): a warp takes 256 consecutive places at a time,
        // lane l the places l, l + 32, ... of them (neighbouring lanes read neighbouring entries of a
        // run and write neighbouring places).  The run of a lane's first place comes from a binary
        // search in the window's table, the following ones by stepping forward; the 8 gathers of a
        // lane are all in flight before the first is stored.
        if (idx_cached) {
          // everything goes to shared memory by asynchronous copies (no register holds a value), so a
          // lane keeps 16 places in flight
          for (uint32_t wb = r_lo + warp * 512u; wb < r_hi; wb += (uint32_t)kFinishWarps * 512u) {
            const uint32_t at0 = wb + lane;
            uint32_t j = j_lo;
            if (at0 < r_hi) {                                      // last run that starts at or before at0
              uint32_t hi_j = j_hi;
              while (hi_j - j > 1u) { const uint32_t mid = (j + hi_j) >> 1; if (dstTab[mid] <= at0) j = mid; else hi_j = mid; }
            }
#pragma unroll
            for (int u = 0; u < 16; ++u) {
              const uint32_t at = at0 + 32u * u;
              if (at < r_hi) {
                while (dstTab[j + 1] <= at) ++j;                   // dstTab[j_hi] >= r_hi > at ends it
                const uint32_t src = srcTab[j] + (at - dstTab[j]);
                async_copy_4(cache_idx + (at - lo), ridx + src);
                async_copy_4(cache + (at - lo), rval + src);
              }
            }
          }
          continue;
        }
        for (uint32_t wb = r_lo + warp * 256u; wb < r_hi; wb += (uint32_t)kFinishWarps * 256u) {
          const uint32_t at0 = wb + lane;
          uint32_t j = j_lo;
          if (at0 < r_hi) {
            uint32_t hi_j = j_hi;
            while (hi_j - j > 1u) { const uint32_t mid = (j + hi_j) >> 1; if (dstTab[mid] <= at0) j = mid; else hi_j = mid; }
          }
          uint32_t ri[kFinishBatch];
          float rv[kFinishBatch];
#pragma unroll
          for (int u = 0; u < kFinishBatch; ++u) {
            const uint32_t at = at0 + 32u * u;
            if (at < r_hi) {
              while (dstTab[j + 1] <= at) ++j;
              const uint32_t src = srcTab[j] + (at - dstTab[j]);
              ri[u] = __ldg(ridx + src); rv[u] = __ldg(rval + src);
            }
          }
#pragma unroll
          for (int u = 0; u < kFinishBatch; ++u) {
            const uint32_t at = at0 + 32u * u;
            if (at < r_hi) put(at, ri[u], rv[u]);
          }
        }
      }
      async_copy_wait_all();
    }
  }
  __syncthreads();
  auto value_at = [&](uint32_t i) -> float { return i < n_cached ? cache[i] : cval[lo + i]; };
  // visits every key of my share once (order is irrelevant to the callers)
  auto for_each_key = [&](auto&& f) {
    const float4* c4 = reinterpret_cast<const float4*>(cache);
    const uint32_t nv = n_cached >> 2;
    for (uint32_t t = tid; t < nv; t += kFinishThreads) {
      const float4 v = c4[t];
      f(mag_key(v.x)); f(mag_key(v.y)); f(mag_key(v.z)); f(mag_key(v.w));
    }
    for (uint32_t i = (nv << 2) + tid; i < n_cached; i += kFinishThreads) f(mag_key(cache[i]));
    for (uint32_t base = n_cached + tid; base < n_mine; base += kFinishThreads * kFinishBatch) {
      float v[kFinishBatch];
#pragma unroll
      for (int u = 0; u < kFinishBatch; ++u) {
        const uint32_t i = base + u * kFinishThreads;
        v[u] = i < n_mine ? cval[lo + i] : 0.f;
      }
#pragma unroll
      for (int u = 0; u < kFinishBatch; ++u)
        if (base + u * kFinishThreads < n_mine) f(mag_key(v[u]));
    }
  };

  // keys inside [lo_key, hi_key) over the whole cluster, when known
  uint32_t bucket_n = general ? n_cand - n_gt : 0xFFFFFFFFu;
  // a bucket of up to kFinishList keys is gathered by every CTA and resolved there without further passes over the shares
  const uint32_t list_max = (uint32_t)kFinishList;
  for (int round = 0; (hi_key - lo_key > 1u || count_above) && round < 8; ++round) {
    if (!count_above && bucket_n <= list_max) {
      // Few keys are left in the interval: instead of more histogram rounds, every CTA lists its own,
      // reads the other CTAs' lists through distributed shared memory and finishes on the union alone.
      if (tid == 0) sm.list_n = 0;
      __syncthreads();
      for_each_key([&](uint32_t key) {
        if (key >= lo_key && key < hi_key) {
          const uint32_t at = atomicAdd(&sm.list_n, 1u);
          if (at < (uint32_t)kBins) sm.hist[at] = key;
        }
      });
      cluster.sync();
      if (warp == 0) {
        const uint32_t n = lane < CS ? *cluster.map_shared_rank(&sm.list_n, lane) : 0u;
        const uint32_t incl = warp_incl_scan(n);
        if (lane < (uint32_t)kMaxCluster) sm.list_pre[lane + 1] = incl;
        if (lane == 0) sm.list_pre[0] = 0;
      }
      __syncthreads();
      const uint32_t total = sm.list_pre[CS];
      if (total > list_max || total < need) {       // the same on every CTA
        if (q == 0 && tid == 0) { atomicOr(L.s.error, ERR_SELECT_INCONSISTENT); st->resolved = 32; }
        cluster.sync();
        return;
      }
      for (uint32_t t = tid; t < total; t += kFinishThreads) {
        uint32_t rr = 0;
        while (sm.list_pre[rr + 1] <= t) ++rr;
        sm.red[t] = cluster.map_shared_rank(sm.hist, rr)[t - sm.list_pre[rr]];
      }
      cluster.sync();                                            // all remote reads of the lists are done
      // Every CTA now holds the whole list and finishes alone: histogram rounds over the list only
      // (equal buckets over what is left of the interval; one round when it spans at most 2048 keys).
      uint32_t found = lo_key, end = hi_key, above = 0, rank = need;
      bool ok = true;
      while (end - found > 1u) {
        const uint32_t w = end - found;
        uint32_t s2 = 0;
        while (((w - 1u) >> s2) >= (uint32_t)kBins) ++s2;
        for (uint32_t bkt = tid; bkt < (uint32_t)kBins; bkt += kFinishThreads) sm.hist[bkt] = 0;
        __syncthreads();
        for (uint32_t t = tid; t < total; t += kFinishThreads) {
          const uint32_t key = sm.red[t];
          if (key >= found && key < end) atomicAdd(&sm.hist[(key - found) >> s2], 1u);
        }
        __syncthreads();
        uint32_t D, ab;
        ok = pick_digit(sm.hist, kBins, rank, sm.scratch, D, ab);
        if (!ok) break;                                          // the same on every thread
        above += ab; rank -= ab;
        found += D << s2;
        end = min(end, found + (1u << s2));
      }
      if (!ok) {
        if (q == 0 && tid == 0) { atomicOr(L.s.error, ERR_SELECT_INCONSISTENT); st->resolved = 32; }
        return;                                                  // every CTA of the cluster takes this exit
      }
      n_gt += above; need -= above;
      lo_key = found; hi_key = found + 1u;
      break;
    }
    const uint32_t width = hi_key - lo_key;                    // >= 1
    uint32_t sh = 0;
    while (((width - 1u) >> sh) >= (uint32_t)(kBins - 1)) ++sh;
    for (uint32_t b = tid; b < (uint32_t)kBins; b += kFinishThreads) sm.hist[b] = 0;
    __syncthreads();
    uint32_t n_above = 0;                                      // keys above the interval: counted in registers
    for_each_key([&](uint32_t key) {
      if (key >= hi_key) ++n_above;
      else if (key >= lo_key) atomicAdd(&sm.hist[(key - lo_key) >> sh], 1u);
    });
    if (count_above) {
      n_above = warp_sum(n_above);
      if (lane == 0 && n_above) atomicAdd(&sm.hist[kBins - 1], n_above);
    }
    cluster.sync();
    // every CTA sums the cluster's histograms for itself (independent remote loads, one latency)
    // and picks the bucket redundantly: no broadcast, no serial section in one CTA
    for (uint32_t b = tid; b < (uint32_t)kBins; b += kFinishThreads) {
      uint32_t part[kMaxCluster];
#pragma unroll
      for (int rr = 0; rr < kMaxCluster; ++rr)
        part[rr] = (uint32_t)rr < CS ? cluster.map_shared_rank(sm.hist, rr)[b] : 0u;
      uint32_t sum = 0;
#pragma unroll
      for (int rr = 0; rr < kMaxCluster; ++rr) sum += part[rr];
      sm.red[b] = sum;
    }
    __syncthreads();
    uint32_t D, above;
    pick_digit(sm.red, kBins, need, sm.scratch, D, above);
    bucket_n = D < (uint32_t)kBins ? sm.red[D] : 0u;
    cluster.sync();                                            // all remote reads of sm.hist are done
    if (D == 0xFFFFFFFFu) {                                    // fewer keys than the rank asked for
      if (q == 0 && tid == 0) { atomicOr(L.s.error, ERR_SELECT_INCONSISTENT); st->resolved = 32; }
      return;
    }
    if (D == (uint32_t)(kBins - 1)) {
      // only possible while the keys above the interval were being counted: the sampled upper
      // estimate was too low and the target lies above it
      lo_key = hi_key; hi_key = 0x80000000u;                    // bucket_n: the keys above, all still inside
    } else {
      n_gt += above; need -= above;
      lo_key += D << sh;
      hi_key = min(hi_key, lo_key + (1u << sh));
    }
    count_above = false;
  }
  if (hi_key - lo_key != 1u) {                                 // did not converge (cannot happen: <= 5 rounds)
    if (q == 0 && tid == 0) { atomicOr(L.s.error, ERR_SELECT_INCONSISTENT); st->resolved = 32; }
    return;
  }
  const uint32_t tau = lo_key, quota = need;
  if (q == 0 && tid == 0) {
    st->prefix = tau; st->resolved = 31; st->n_gt = n_gt; st->need = need;
    if (L.reuse) {
      TauHistory h = L.s.history[sl];
      const uint32_t pred = st->pred;
      if (pred != 0 && (st->flags & FLAG_FELL_BACK)) {        // the predicted bracket missed: sample next time
        // A bracket that began above the threshold (too few candidates) was too narrow: the next ones are
        // wider.  One that let more candidates through than the list holds reached too far down: on data
        // with a steep tail (a Gaussian bulk) a wider bracket would overflow again, so the next ones are narrower.
        if (st->n_cand_first > S.cand_cap) h.err = fmaxf(0.5f * h.err, 0.002f);
        else h.err = fminf(fmaxf(2.0f * h.err, 0.05f), 0.2f);
        h.tau1 = tau; h.tau2 = 0; h.valid = 0;
      } else {
        if (pred != 0) {
          const float rel = fabsf(__uint_as_float(tau) / __uint_as_float(pred) - 1.0f);
          h.err = rel == rel ? fmaxf(rel, 0.7f * h.err) : 0.2f;
        } else if (h.valid == 0 && h.err == 0.0f) {
          h.err = 0.03f;                                         // nothing known yet about this slice
        }
        h.tau2 = h.valid >= 1 ? h.tau1 : 0u;
        h.tau1 = tau;
        h.valid = min(h.valid + 1u, 2u);
      }
      L.s.history[sl] = h;
    }
  }

  // Members of my share (keys above tau, keys equal to tau), per warp: warp w owns the w-th
  // contiguous part of the share, so that the walk below needs no block-wide barrier.
  const uint32_t wper = ((n_mine + kFinishWarps - 1) / kFinishWarps + 127u) & ~127u;   // multiple of 128
  const uint32_t w_lo = min(n_mine, warp * wper), w_hi = min(n_mine, w_lo + wper);
  auto load4 = [&](uint32_t i, float (&v)[4]) {               // values i..i+3 of my share (i % 4 == 0)
    if (i + 4u <= n_cached) {
      const float4 x = *reinterpret_cast<const float4*>(cache + i);
      v[0] = x.x; v[1] = x.y; v[2] = x.z; v[3] = x.w;
    } else if (i >= n_cached && i + 4u <= n_mine) {
      const float4 x = *reinterpret_cast<const float4*>(cval + lo + i);
      v[0] = x.x; v[1] = x.y; v[2] = x.z; v[3] = x.w;
    } else {
#pragma unroll
      for (int j = 0; j < 4; ++j) v[j] = i + j < n_mine ? value_at(i + j) : 0.f;
    }
  };
  uint32_t cA = 0, cB = 0;
  for (uint32_t base = w_lo; base < w_hi; base += 128u) {
    const uint32_t i0 = base + lane * 4u;
    float v[4];
    load4(i0, v);
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      const uint32_t key = mag_key(v[j]);
      const bool in = i0 + j < w_hi;
      cA += in && key > tau; cB += in && key == tau;
    }
  }
  cA = warp_sum(cA); cB = warp_sum(cB);
  if (lane == 0) { sm.warpA[warp] = cA; sm.warpB[warp] = cB; }
  __syncthreads();
  if (tid < CS) {
    uint32_t tA = 0, tB = 0;
#pragma unroll
    for (int w = 0; w < kFinishWarps; ++w) { tA += sm.warpA[w]; tB += sm.warpB[w]; }
    uint32_t* c = cluster.map_shared_rank(sm.counts, tid);   // my counts, into CTA `tid`
    c[2 * q] = tA; c[2 * q + 1] = tB;
  }
  cluster.sync();                                              // last remote access of the kernel
  uint32_t gt_before = 0, eq_before = 0;
  for (uint32_t p = 0; p < q; ++p) { gt_before += sm.counts[2 * p]; eq_before += sm.counts[2 * p + 1]; }

  // the part of the sampler's bitmap that covers my members' positions -> shared memory
  const uint32_t pos0 = gt_before + min(eq_before, quota);
  const uint32_t pos1 = min(S.r, pos0 + sm.counts[2 * q] + sm.counts[2 * q + 1]);
  const uint32_t word0 = pos0 >> 5, nwords = pos1 > pos0 ? ((pos1 + 31u) >> 5) - word0 : 0u;
  const bool sel_all = S.k == S.r;
  const bool sel_cached = !sel_all && nwords <= (uint32_t)kFinishSelWords;
  if (sel_cached)
    for (uint32_t w = tid; w < nwords; w += kFinishThreads) {
      sm.sel[w] = L.s.sel[S.sel_off + word0 + w];
      sm.sel_pre[w] = L.s.sel_pre[S.sel_off + word0 + w];
    }
  __syncthreads();
  // Bitmap words of a walk step: the members met in one step of 128 candidates take consecutive
  // positions first_pos, first_pos + 1, ..., so they fall into at most 5 consecutive bitmap words.
  // Lane l < 6 fetches word (first_pos / 32) + l and its running popcount; the walk reads them by shuffle.
  const uint32_t sel_words_all = (S.r + 31u) >> 5;
  auto fetch_sel = [&](uint32_t first_pos, uint32_t& word, uint32_t& pre) {
    word = 0; pre = 0;
    const uint32_t wi = (first_pos >> 5) + lane;
    if (!sel_all && lane < 6u && wi < sel_words_all) {
      if (sel_cached) {
        if (wi - word0 < nwords) { word = sm.sel[wi - word0]; pre = sm.sel_pre[wi - word0]; }
      } else {
        word = L.s.sel[S.sel_off + wi];
        pre = L.s.sel_pre[S.sel_off + wi];
      }
    }
  };
  // values and indices of a walk step (4 consecutive candidates per lane, 128 per step); the index
  // list's capacity is a multiple of 32 entries, so the vector stays inside the slice's list
  auto fetch_step = [&](uint32_t base, float (&v)[4], uint4& ci) {
    const uint32_t i0 = base + lane * 4u;
    load4(i0, v);
    ci = make_uint4(0u, 0u, 0u, 0u);
    if (i0 < w_hi) ci = idx_cached ? *reinterpret_cast<const uint4*>(cache_idx + i0)
                                   : *reinterpret_cast<const uint4*>(cidx + lo + i0);
  };

  // Walk my warp's part in index order.  Everything a step loads is requested one step ahead (the
  // next step's candidates, and -- as soon as this step's member count is known -- the next step's
  // bitmap words), so that no store of the current step waits behind a load.
  for (uint32_t w = 0; w < warp; ++w) { gt_before += sm.warpA[w]; eq_before += sm.warpB[w]; }
  float v_next[4] = {0.f, 0.f, 0.f, 0.f};
  uint4 ci_next = make_uint4(0u, 0u, 0u, 0u);
  uint32_t sw_next, sp_next;
  if (w_lo < w_hi) fetch_step(w_lo, v_next, ci_next);
  fetch_sel(gt_before + min(eq_before, quota), sw_next, sp_next);
  for (uint32_t base = w_lo; base < w_hi; base += 128u) {
    const uint32_t i0 = base + lane * 4u;
    const float v[4] = {v_next[0], v_next[1], v_next[2], v_next[3]};
    const uint32_t cj[4] = {ci_next.x, ci_next.y, ci_next.z, ci_next.w};
    const uint32_t sw = sw_next, sp = sp_next;
    if (base + 128u < w_hi) fetch_step(base + 128u, v_next, ci_next);
    uint32_t mA = 0, mB = 0;
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      const uint32_t key = mag_key(v[j]);
      const bool in = i0 + j < w_hi;
      mA |= (uint32_t)(in && key > tau) << j;
      mB |= (uint32_t)(in && key == tau) << j;
    }
    const uint32_t pack = (uint32_t)__popc(mA) | ((uint32_t)__popc(mB) << 16);   // <= 128 each per warp
    const uint32_t incl = warp_incl_scan(pack);
    const uint32_t tot = __shfl_sync(0xFFFFFFFFu, incl, 31);
    const uint32_t excl = incl - pack;
    const uint32_t first_pos = gt_before + min(eq_before, quota);
    const uint32_t gt_after = gt_before + (tot & 0xFFFFu), eq_after = eq_before + (tot >> 16);
    fetch_sel(gt_after + min(eq_after, quota), sw_next, sp_next);
    // A lane's members take consecutive positions p0, p0 + 1, ... (at most four): their bitmap bits are
    // one funnel shift of two neighbouring words, and the slot of the first is the word's running
    // popcount plus the selected positions below p0 inside the word.
    const uint32_t g0 = gt_before + (excl & 0xFFFFu), e0 = eq_before + (excl >> 16);
    const uint32_t p0 = g0 + min(e0, quota);
    uint32_t members = mA;                                                   // bit j: candidate j is in the top-r set
    {
      uint32_t e = e0;
#pragma unroll
      for (int j = 0; j < 4; ++j) {
        const uint32_t isB = (mB >> j) & 1u;
        members |= (isB & (uint32_t)(e < quota)) << j;
        e += isB;
      }
    }
    const uint32_t rel = members ? (p0 >> 5) - (first_pos >> 5) : 0u;       // 0 .. 4
    const uint32_t w0 = __shfl_sync(0xFFFFFFFFu, sw, rel);
    const uint32_t w1 = __shfl_sync(0xFFFFFFFFu, sw, rel + 1u);
    const uint32_t pre = __shfl_sync(0xFFFFFFFFu, sp, rel);
    if (members) {
      const uint32_t sh = p0 & 31u;
      const uint32_t bits = sel_all ? 0xFu : __funnelshift_r(w0, w1, sh);    // bit o: the o-th member of the lane is chosen
      const uint32_t slot0 = sel_all ? p0 : pre + __popc(w0 & ((1u << sh) - 1u));
      uint32_t o = 0;
#pragma unroll
      for (int j = 0; j < 4; ++j) {
        if ((members >> j) & 1u) {
          if (((bits >> o) & 1u) && p0 + o < S.r) {
            const uint32_t slot = slot0 + __popc(bits & ((1u << o) - 1u));
            const uint32_t idx = cj[j];
            if (slot < S.k && idx < S.len) {                     // (idx < len always, unless an earlier wait gave up and left the list incomplete)
              L.msg_idx[(size_t)(S.msg_off + slot) * L.msg_stride] = S.idx_base + idx;
              L.msg_val[(size_t)(S.msg_off + slot) * L.msg_stride] = v[j];
              L.residual[S.m_off + idx] = 0.0f;
              note_message(L, S, slot, S.idx_base + idx);
            }
          }
          ++o;
        }
      }
    }
    gt_before = gt_after; eq_before = eq_after;
  }
}

// r = d (Definition 2, random-k): every coordinate is in the "top-r" set and position = index.
// One thread per bitmap word of each such slice.
__global__ void __launch_bounds__(kThreads) k_emit_all(Launch L, uint32_t words_per_slice_max) {
  const uint32_t sl = blockIdx.y;
  const Slice S = L.s.slices[sl];
  if (S.r != S.len) return;
  const uint32_t w = blockIdx.x * kThreads + threadIdx.x;
  const uint32_t nwords = (S.r + 31u) >> 5;
  if (w >= nwords || w >= words_per_slice_max) return;
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
    const uint32_t p = w * 32u + b;
    if (pre < S.k) {
      L.msg_idx[(size_t)(S.msg_off + pre) * L.msg_stride] = S.idx_base + p;
      L.msg_val[(size_t)(S.msg_off + pre) * L.msg_stride] = L.residual[S.m_off + p];
      L.residual[S.m_off + p] = 0.0f;
      note_message(L, S, pre, S.idx_base + p);
    }
    ++pre;
  }
}

}  // namespace rtopk
