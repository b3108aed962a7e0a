// Top-r selection kernels (Definition 1 with the lower-index tie rule), fused with the
// error-feedback add of Algorithm 1 (a = g + m, written back into the residual buffer).
//
//   k_sample        estimates a threshold from a strided sample of a = g + m
//   k_collect       one streaming pass: a = g + m -> residual, keys above the threshold are appended
//                   to an index-ordered candidate list (ballot/prefix compaction + look-back)
//   k_hist          full-vector radix histogram pass (exact path and fallback)
//   k_cand_hist     radix select of the r-th largest key among the candidates
//   k_emit          walks the candidates in index order, numbers the members of the top-r set and
//                   writes the ones the k-of-r sampler chose as (index, value) messages, zeroing
//                   their residual slots (m' = a - ghat)
#pragma once

#include "common.cuh"

namespace rtopk {

// ----------------------------------------------------------------------------- element access
template <typename GradT> struct Grad;
template <> struct Grad<float> {
  static __device__ __forceinline__ float4 ld4(const void* base, int64_t off) {
    return __ldcs(reinterpret_cast<const float4*>(static_cast<const float*>(base) + off));
  }
  static __device__ __forceinline__ float ld1(const void* base, int64_t off) {
    return __ldcs(static_cast<const float*>(base) + off);
  }
};
template <> struct Grad<__nv_bfloat16> {
  static __device__ __forceinline__ float4 ld4(const void* base, int64_t off) {
    const uint2 v = __ldcs(reinterpret_cast<const uint2*>(static_cast<const uint16_t*>(base) + off));
    float4 f;   // bfloat16 is the upper half of binary32: widening is a shift
    f.x = __uint_as_float(v.x << 16); f.y = __uint_as_float(v.x & 0xFFFF0000u);
    f.z = __uint_as_float(v.y << 16); f.w = __uint_as_float(v.y & 0xFFFF0000u);
    return f;
  }
  static __device__ __forceinline__ float ld1(const void* base, int64_t off) {
    return __uint_as_float((uint32_t)__ldcs(static_cast<const uint16_t*>(base) + off) << 16);
  }
};

// The error-feedback add a = g + m of Algorithm 1: one round-to-nearest binary32 add.  IEEE 754 does
// not fix the payload of a NaN result, so a NaN sum is stored as the default quiet NaN.
__device__ __forceinline__ float ef_add(float g, float m) {
  const float s = __fadd_rn(g, m);
  return s != s ? __uint_as_float(0x7FC00000u) : s;
}

// Loads the 4 elements e..e+3 of the slice's aligned element grid (element `head` is the slice's
// first coordinate, `span` = head + len is one past its last), forms a = g + m when FUSE and
// stores it back, and returns the values with a 4-bit validity mask.
template <typename GradT, bool FUSE>
__device__ __forceinline__ uint32_t load_vec(const void* grad, float* residual, int64_t base_g, int64_t base_m,
                                             uint32_t e, uint32_t head, uint32_t span, float (&a)[4]) {
  if (e >= span) { a[0] = a[1] = a[2] = a[3] = 0.f; return 0u; }
  if (e >= head && e + 4u <= span) {
    float4 m4 = FUSE ? __ldcs(reinterpret_cast<const float4*>(residual + base_m + e))
                     : __ldg(reinterpret_cast<const float4*>(residual + base_m + e));
    if (FUSE) {
      const float4 g4 = Grad<GradT>::ld4(grad, base_g + e);
      m4.x = ef_add(g4.x, m4.x); m4.y = ef_add(g4.y, m4.y);
      m4.z = ef_add(g4.z, m4.z); m4.w = ef_add(g4.w, m4.w);
      __stcs(reinterpret_cast<float4*>(residual + base_m + e), m4);
    }
    a[0] = m4.x; a[1] = m4.y; a[2] = m4.z; a[3] = m4.w;
    return 0xFu;
  }
  uint32_t valid = 0;
#pragma unroll
  for (int j = 0; j < 4; ++j) {
    const uint32_t ee = e + j;
    a[j] = 0.f;
    if (ee >= head && ee < span) {
      float v = residual[base_m + ee];
      if (FUSE) { v = ef_add(Grad<GradT>::ld1(grad, base_g + ee), v); residual[base_m + ee] = v; }
      a[j] = v;
      valid |= 1u << j;
    }
  }
  return valid;
}

__device__ __forceinline__ uint32_t slice_chunks(const Slice& S) {
  return (S.head + S.len + kChunk - 1) / kChunk;
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
  st.pad[0] = st.pad[1] = 0;
  if (S.r == S.len) { st.resolved = 31; st.stage = STAGE_DONE; st.flags = 0; }   // top-r is everything
  else { st.resolved = 0; st.stage = STAGE_PASS0; st.flags = general ? FLAG_GENERAL : 0u; }
  L.s.state[s] = st;
}

// ----------------------------------------------------------------------------- sampled threshold
// One block per slice.  Reads up to kSampleMax coordinates of a = g + m in 128-byte groups spread
// evenly over the slice, and picks as threshold the sample key whose sample rank, scaled to the
// slice, lies six standard deviations above r.  The collect pass then verifies the count; a miss
// is repaired by the exact path, so the estimate only affects speed, never the result.
template <typename GradT>
__global__ void __launch_bounds__(kSampleThreads) k_sample(Launch L) {
  extern __shared__ uint32_t smem[];
  uint32_t* keys = smem;
  uint32_t* hist = smem + kSampleMax;
  uint32_t* scratch = hist + kBins;
  const uint32_t sl = blockIdx.x;
  const Slice S = L.s.slices[sl];
  const uint32_t tid = threadIdx.x;
  SelState st;
  st.eq_quota = kNoQuota; st.prefix = 0; st.resolved = 0; st.n_gt = 0; st.need = S.r;
  st.n_cand = 0; st.n_cand_first = 0; st.stage = STAGE_PASS0; st.flags = 0; st.pad[0] = st.pad[1] = 0;
  if (S.r == S.len) {
    st.tau_lo = 0x80000000u; st.resolved = 31; st.stage = STAGE_DONE;
    if (tid == 0) L.s.state[sl] = st;
    return;
  }
  const float* m = L.residual;
  uint32_t n_s, rho;
  if (S.len <= (uint32_t)kSampleMax) {
    n_s = S.len; rho = S.r;
    for (uint32_t i = tid; i < n_s; i += kSampleThreads)
      keys[i] = mag_key(ef_add(Grad<GradT>::ld1(L.grad, S.g_off + i), m[S.m_off + i]));
  } else {
    const uint32_t v0 = (S.head + 3u) >> 2, v1 = (S.head + S.len) >> 2;   // fully valid vectors
    const uint32_t ngroups_avail = (v1 - v0) >> 3;
    const uint32_t G = min((uint32_t)(kSampleMax / 32), ngroups_avail);
    n_s = G * 32u;
    const int64_t base_g = S.g_off - S.head, base_m = S.m_off - S.head;
    for (uint32_t n = tid; n < G * 8u; n += kSampleThreads) {
      const uint32_t gi = n >> 3, vv = n & 7u;
      const uint32_t vec = v0 + (uint32_t)(((uint64_t)gi * ngroups_avail) / G) * 8u + vv;
      const float4 g4 = Grad<GradT>::ld4(L.grad, base_g + (int64_t)vec * 4);
      const float4 m4 = __ldg(reinterpret_cast<const float4*>(m + base_m + (int64_t)vec * 4));
      keys[n * 4 + 0] = mag_key(ef_add(g4.x, m4.x));
      keys[n * 4 + 1] = mag_key(ef_add(g4.y, m4.y));
      keys[n * 4 + 2] = mag_key(ef_add(g4.z, m4.z));
      keys[n * 4 + 3] = mag_key(ef_add(g4.w, m4.w));
    }
    const float expect = (float)n_s * ((float)S.r / (float)S.len);
    const float target = expect + 6.0f * sqrtf(expect) + 8.0f;
    rho = target >= (float)n_s ? n_s : (uint32_t)target;
  }
  __syncthreads();
  uint32_t prefix = 0, need = rho;
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
  st.tau_lo = prefix;
  if (tid == 0) L.s.state[sl] = st;
}

// ----------------------------------------------------------------------------- collect
// TIES = false: candidates are the keys >= tau_lo.  TIES = true: keys > tau_lo and the first
// eq_quota keys == tau_lo in index order.  The candidate list keeps index order: inside a block by
// ballot-free packed prefix sums, across blocks by the look-back on (count above, count equal).
template <typename GradT, bool FUSE, bool TIES>
__global__ void __launch_bounds__(kThreads) k_collect(Launch L) {
  __shared__ uint32_t s_tile, s_wA[kWarps], s_wB[kWarps], s_ex[2];
  const uint32_t tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  if (tid == 0) s_tile = atomicAdd(&L.s.tickets[FUSE ? 0 : 1], 1u);
  __syncthreads();
  const uint32_t tile = s_tile;
  const Slice* slices = L.s.slices;
  const uint32_t sl = find_slice(L.n_slices, tile, [&](uint32_t i) { return slices[i].chunk_begin; });
  const Slice S = slices[sl];
  SelState* st = &L.s.state[sl];
  if (!FUSE) {
    if (!((st->flags & FLAG_GENERAL) && st->stage == STAGE_COLLECT)) return;
  }
  const uint32_t tau = st->tau_lo;
  const uint32_t quota = TIES ? st->eq_quota : kNoQuota;
  const uint32_t c = tile - S.chunk_begin;
  const uint32_t span = S.head + S.len;
  const int64_t base_g = S.g_off - S.head, base_m = S.m_off - S.head;
  const uint32_t e_w = c * (uint32_t)kChunk + warp * (uint32_t)kWarpSpan;

  float a[kIter][4];
  uint32_t maskA = 0, maskB = 0;
#pragma unroll
  for (int it = 0; it < kIter; ++it) {
    const uint32_t e = e_w + it * 128u + lane * 4u;
    const uint32_t valid = load_vec<GradT, FUSE>(L.grad, L.residual, base_g, base_m, e, S.head, span, a[it]);
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      const uint32_t key = mag_key(a[it][j]);
      const bool ok = (valid >> j) & 1u;
      if (TIES) {
        maskA |= (uint32_t)(ok && key > tau) << (it * 4 + j);
        maskB |= (uint32_t)(ok && key == tau) << (it * 4 + j);
      } else {
        maskA |= (uint32_t)(ok && key >= tau) << (it * 4 + j);
      }
    }
  }
  // per-iteration counts packed one byte each (a byte holds at most 32 lanes x 4 = 128)
  uint32_t packA = 0, packB = 0;
#pragma unroll
  for (int it = 0; it < kIter; ++it) {
    packA |= (uint32_t)__popc((maskA >> (it * 4)) & 0xFu) << (it * 8);
    if (TIES) packB |= (uint32_t)__popc((maskB >> (it * 4)) & 0xFu) << (it * 8);
  }
  const uint32_t inclA = warp_incl_scan(packA);
  const uint32_t inclB = TIES ? warp_incl_scan(packB) : 0u;
  const uint32_t totA = __shfl_sync(0xFFFFFFFFu, inclA, 31), totB = __shfl_sync(0xFFFFFFFFu, inclB, 31);
  const uint32_t exLaneA = inclA - packA, exLaneB = inclB - packB;
  uint32_t wA = 0, wB = 0;
#pragma unroll
  for (int it = 0; it < kIter; ++it) { wA += (totA >> (it * 8)) & 0xFFu; wB += (totB >> (it * 8)) & 0xFFu; }
  if (lane == 0) { s_wA[warp] = wA; s_wB[warp] = wB; }
  __syncthreads();
  if (warp == 0) {
    uint32_t bA = 0, bB = 0;
#pragma unroll
    for (int w = 0; w < kWarps; ++w) { bA += s_wA[w]; bB += s_wB[w]; }
    uint32_t exA, exB;
    unsigned long long* words = (FUSE ? L.s.look_a : L.s.look_b) + S.chunk_begin;
    lookback_exclusive(words, c, bA, bB, exA, exB, L.s.error);
    if (lane == 0) {
      s_ex[0] = exA; s_ex[1] = exB;
      if (c + 1 == slice_chunks(S)) {      // last tile of the slice: publish the total
        const uint32_t n = exA + bA + min(exB + bB, quota);
        st->n_cand = n;
        if (FUSE) st->n_cand_first = n;
      }
    }
  }
  __syncthreads();
  if ((maskA | maskB) == 0) return;
  uint32_t gt_before = s_ex[0], eq_before = s_ex[1];
  for (uint32_t w = 0; w < warp; ++w) { gt_before += s_wA[w]; eq_before += s_wB[w]; }
  uint32_t* cidx = L.s.cand_idx + S.cand_off;
  float* cval = L.s.cand_val + S.cand_off;
#pragma unroll
  for (int it = 0; it < kIter; ++it) {
    uint32_t bitsA = (maskA >> (it * 4)) & 0xFu, bitsB = (maskB >> (it * 4)) & 0xFu;
    if (bitsA | bitsB) {
      uint32_t g = gt_before + ((exLaneA >> (it * 8)) & 0xFFu);
      uint32_t q = eq_before + ((exLaneB >> (it * 8)) & 0xFFu);
      const uint32_t e = e_w + it * 128u + lane * 4u;
#pragma unroll
      for (int j = 0; j < 4; ++j) {
        const bool isA = (bitsA >> j) & 1u, isB = (bitsB >> j) & 1u;
        if (isA || (isB && q < quota)) {
          const uint32_t pos = g + min(q, quota);
          if (pos < S.cand_cap) { cidx[pos] = e + j - S.head; cval[pos] = a[it][j]; }
        }
        g += isA; q += isB;
      }
    }
    gt_before += (totA >> (it * 8)) & 0xFFu;
    eq_before += (totB >> (it * 8)) & 0xFFu;
  }
}

// ----------------------------------------------------------------------------- radix passes
// Runs in the last block of a slice's histogram pass: turns the finished histogram into the next
// digit of the r-th largest key.  `full_vector` passes also decide whether the bucket is small
// enough to collect (or, with all 31 bits resolved, fix the exact threshold and tie quota).
__device__ __forceinline__ void finish_pass(const Launch& L, uint32_t sl, const Slice& S, int pass,
                                            bool full_vector, bool fell_back, uint32_t* hist_s,
                                            uint32_t* scratch) {
  const int bits = digit_bits(pass);
  uint32_t* gh = L.s.hist + (size_t)sl * kBins;
  for (uint32_t b = threadIdx.x; b < (uint32_t)kBins; b += blockDim.x) {
    hist_s[b] = __ldcg(gh + b);
    gh[b] = 0;
  }
  __syncthreads();
  SelState* st = &L.s.state[sl];
  const uint32_t need = st->need;
  uint32_t D, above;
  const bool ok = pick_digit(hist_s, 1 << bits, need, scratch, D, above);
  if (threadIdx.x == 0) {
    L.s.done[sl] = 0;
    if (!ok) {
      atomicOr(L.s.error, ERR_SELECT_INCONSISTENT);
      st->stage = STAGE_DONE;
      st->resolved = 32;     // blocks the later passes of this slice
    } else {
      const uint32_t n_gt = st->n_gt + above, need2 = need - above;
      const uint32_t prefix = (st->prefix << bits) | D;
      const uint32_t resolved = st->resolved + bits;
      st->n_gt = n_gt; st->need = need2; st->prefix = prefix; st->resolved = resolved;
      if (full_vector) {
        const uint32_t n_ge = n_gt + hist_s[D];
        if (n_ge <= S.cand_cap) { st->tau_lo = prefix << (31 - resolved); st->eq_quota = kNoQuota; st->stage = STAGE_COLLECT; }
        else if (resolved == 31) { st->tau_lo = prefix; st->eq_quota = need2; st->stage = STAGE_COLLECT; }
        else st->stage = pass + 1;
        st->flags |= FLAG_GENERAL | (fell_back ? FLAG_FELL_BACK : 0u);
      }
    }
  }
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

__device__ __forceinline__ bool first_pass_missed(const SelState* st, const Slice& S) {
  return st->n_cand < S.r || st->n_cand > S.cand_cap;
}

// Histogram of one digit over the whole slice.  FUSE (pass 0 of the exact path) also performs the
// add and the write-back; otherwise a is read from the residual buffer.  Pass p > 0 counts only keys
// whose higher bits equal the resolved prefix.
template <typename GradT, bool FUSE>
__global__ void __launch_bounds__(kThreads) k_hist(Launch L, int pass) {
  __shared__ uint32_t hist_s[kBins];
  __shared__ uint32_t scratch[kWarps + 2];
  const uint32_t tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const Slice* slices = L.s.slices;
  const uint32_t sl = find_slice(L.n_slices, blockIdx.x, [&](uint32_t i) { return slices[i].hist_begin; });
  const Slice S = slices[sl];
  SelState* st = &L.s.state[sl];
  const uint32_t flags = st->flags;
  const bool fell_back = !(flags & FLAG_GENERAL) && !FUSE && pass == 0 && S.r < S.len && first_pass_missed(st, S);
  const bool counting = (flags & FLAG_GENERAL) ? st->stage == (uint32_t)pass : fell_back;
  const bool add_only = FUSE && S.r == S.len;      // nothing to select, but a = g + m is still due
  if (!counting && !add_only) return;
  const uint32_t prefix = st->prefix;
  const int bits = digit_bits(pass), shift = digit_shift(pass);
  for (uint32_t b = tid; b < (uint32_t)kBins; b += kThreads) hist_s[b] = 0;
  __syncthreads();
  const uint32_t nchunks = slice_chunks(S);
  const uint32_t hb = blockIdx.x - S.hist_begin;
  const uint32_t c0 = hb * kHistChunks, c1 = min(nchunks, c0 + kHistChunks);
  const uint32_t span = S.head + S.len;
  const int64_t base_g = S.g_off - S.head, base_m = S.m_off - S.head;
  for (uint32_t c = c0; c < c1; ++c) {
    const uint32_t e_w = c * (uint32_t)kChunk + warp * (uint32_t)kWarpSpan;
    float a[kIter][4];
    uint32_t valid[kIter];
#pragma unroll
    for (int it = 0; it < kIter; ++it)
      valid[it] = load_vec<GradT, FUSE>(L.grad, L.residual, base_g, base_m, e_w + it * 128u + lane * 4u,
                                        S.head, span, a[it]);
    if (counting) {
#pragma unroll
      for (int it = 0; it < kIter; ++it)
#pragma unroll
        for (int j = 0; j < 4; ++j) {
          const uint32_t key = mag_key(a[it][j]);
          if (((valid[it] >> j) & 1u) && (pass == 0 || (key >> (shift + bits)) == prefix))
            atomicAdd(&hist_s[(key >> shift) & ((1u << bits) - 1u)], 1u);
        }
    }
  }
  if (!counting) return;
  __syncthreads();
  uint32_t* gh = L.s.hist + (size_t)sl * kBins;
  for (uint32_t b = tid; b < (1u << bits); b += kThreads) {
    const uint32_t v = hist_s[b];
    if (v) atomicAdd(gh + b, v);
  }
  const uint32_t nblocks = (nchunks + kHistChunks - 1) / kHistChunks;
  if (is_last_block(&L.s.done[sl], nblocks)) finish_pass(L, sl, S, pass, true, fell_back, hist_s, scratch);
}

__device__ __forceinline__ uint32_t slice_ctiles(const Slice& S) {
  return (S.cand_cap + kCandTile - 1) / kCandTile;
}

// One digit of the radix select among the candidates of each slice.
__global__ void __launch_bounds__(kThreads) k_cand_hist(Launch L, int pass) {
  __shared__ uint32_t hist_s[kBins];
  __shared__ uint32_t scratch[kWarps + 2];
  const uint32_t tid = threadIdx.x;
  const Slice* slices = L.s.slices;
  const uint32_t sl = find_slice(L.n_slices, blockIdx.x, [&](uint32_t i) { return slices[i].ctile_begin; });
  const Slice S = slices[sl];
  SelState* st = &L.s.state[sl];
  if (st->resolved != (uint32_t)resolved_before(pass)) return;
  const uint32_t n_cand = st->n_cand;
  if (n_cand < S.r || n_cand > S.cand_cap) {       // cannot happen once the exact path has run
    if (tid == 0 && blockIdx.x == S.ctile_begin) atomicOr(L.s.error, ERR_CANDIDATE_OVERFLOW);
    return;
  }
  const uint32_t prefix = st->prefix;
  const int bits = digit_bits(pass), shift = digit_shift(pass);
  for (uint32_t b = tid; b < (uint32_t)kBins; b += kThreads) hist_s[b] = 0;
  __syncthreads();
  const uint32_t t0 = (blockIdx.x - S.ctile_begin) * (uint32_t)kCandTile;
  const float* cval = L.s.cand_val + S.cand_off;
#pragma unroll
  for (int q = 0; q < kCandPer; ++q) {
    const uint32_t i = t0 + q * kThreads + tid;
    if (i < n_cand) {
      const uint32_t key = mag_key(cval[i]);
      if (pass == 0 || (key >> (shift + bits)) == prefix) atomicAdd(&hist_s[(key >> shift) & ((1u << bits) - 1u)], 1u);
    }
  }
  __syncthreads();
  uint32_t* gh = L.s.hist + (size_t)sl * kBins;
  for (uint32_t b = tid; b < (1u << bits); b += kThreads) {
    const uint32_t v = hist_s[b];
    if (v) atomicAdd(gh + b, v);
  }
  if (is_last_block(&L.s.done[sl], slice_ctiles(S))) finish_pass(L, sl, S, pass, false, false, hist_s, scratch);
}

// ----------------------------------------------------------------------------- emit
// Position p of a top-r member = number of members with a lower index.  Members are the candidates
// with key > tau plus the first `quota` candidates with key == tau.  Position p is sent iff the
// sampler's bitmap has bit p; its place in the message is the number of selected positions below p.
__device__ __forceinline__ bool position_selected(const Launch& L, const Slice& S, uint32_t p, uint32_t& slot) {
  if (S.k == S.r) { slot = p; return true; }
  const uint32_t word = L.s.sel[S.sel_off + (p >> 5)];
  slot = L.s.sel_pre[S.sel_off + (p >> 5)] + __popc(word & ((1u << (p & 31u)) - 1u));
  return (word >> (p & 31u)) & 1u;
}

__global__ void __launch_bounds__(kThreads) k_emit(Launch L) {
  __shared__ uint32_t s_tile, s_wA[kWarps], s_wB[kWarps], s_ex[2];
  const uint32_t tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  if (tid == 0) s_tile = atomicAdd(&L.s.tickets[2], 1u);
  __syncthreads();
  const uint32_t tile = s_tile;
  const Slice* slices = L.s.slices;
  const uint32_t sl = find_slice(L.n_slices, tile, [&](uint32_t i) { return slices[i].ctile_begin; });
  const Slice S = slices[sl];
  const SelState* st = &L.s.state[sl];
  if (S.r == S.len || st->resolved != 31) return;
  const uint32_t n_cand = st->n_cand;
  if (n_cand < S.r || n_cand > S.cand_cap) return;
  const uint32_t tau = st->prefix, quota = st->need;
  const uint32_t ct = tile - S.ctile_begin;
  const uint32_t i_w = ct * (uint32_t)kCandTile + warp * (uint32_t)(kCandPer * 32);
  const uint32_t* cidx = L.s.cand_idx + S.cand_off;
  const float* cval = L.s.cand_val + S.cand_off;
  float val[kCandPer];
  uint32_t ballA[kCandPer], ballB[kCandPer];
  uint32_t wA = 0, wB = 0;
#pragma unroll
  for (int q = 0; q < kCandPer; ++q) {
    const uint32_t i = i_w + q * 32u + lane;
    bool isA = false, isB = false;
    val[q] = 0.f;
    if (i < n_cand) {
      val[q] = cval[i];
      const uint32_t key = mag_key(val[q]);
      isA = key > tau; isB = key == tau;
    }
    ballA[q] = __ballot_sync(0xFFFFFFFFu, isA);
    ballB[q] = __ballot_sync(0xFFFFFFFFu, isB);
    wA += __popc(ballA[q]); wB += __popc(ballB[q]);
  }
  if (lane == 0) { s_wA[warp] = wA; s_wB[warp] = wB; }
  __syncthreads();
  if (warp == 0) {
    uint32_t bA = 0, bB = 0;
#pragma unroll
    for (int w = 0; w < kWarps; ++w) { bA += s_wA[w]; bB += s_wB[w]; }
    uint32_t exA, exB;
    lookback_exclusive(L.s.look_e + S.ctile_begin, ct, bA, bB, exA, exB, L.s.error);
    if (lane == 0) { s_ex[0] = exA; s_ex[1] = exB; }
  }
  __syncthreads();
  uint32_t gt_before = s_ex[0], eq_before = s_ex[1];
  for (uint32_t w = 0; w < warp; ++w) { gt_before += s_wA[w]; eq_before += s_wB[w]; }
  const uint32_t lt = (1u << lane) - 1u;
#pragma unroll
  for (int q = 0; q < kCandPer; ++q) {
    const bool isA = (ballA[q] >> lane) & 1u, isB = (ballB[q] >> lane) & 1u;
    const uint32_t g = gt_before + __popc(ballA[q] & lt), e = eq_before + __popc(ballB[q] & lt);
    if (isA || (isB && e < quota)) {
      const uint32_t p = g + min(e, quota);
      uint32_t slot;
      if (p < S.r && position_selected(L, S, p, slot) && slot < S.k) {
        const uint32_t idx = cidx[i_w + q * 32u + lane];
        L.msg_idx[S.msg_off + slot] = S.idx_base + idx;
        L.msg_val[S.msg_off + slot] = val[q];
        L.residual[S.m_off + idx] = 0.0f;
      }
    }
    gt_before += __popc(ballA[q]); eq_before += __popc(ballB[q]);
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
      L.msg_idx[S.msg_off + pre] = S.idx_base + p;
      L.msg_val[S.msg_off + pre] = L.residual[S.m_off + p];
      L.residual[S.m_off + p] = 0.0f;
    }
    ++pre;
  }
}

}  // namespace rtopk
