// Finishing a slice straight from the runs of the streaming pass (Definition 1's top-r set, then the
// members Definition 3's subset chose), without laying the candidates out in index order first.
//
// The streaming pass leaves the candidates of a slice in one dense list: per chunk of 4096 coordinates
// a run of (index, value) entries in index order, the runs one behind the other in the order in which
// the chunks were finished, and per chunk where its run starts.  It also leaves the sampled or predicted
// bracket [tau_lo, tau_hi] of the r-th largest key and, counted while the candidates were written (f32
// gradients; k_run_hist below otherwise), their histogram over the bracket: 2047 equal buckets (the keys above
// the bracket are the rest of the list).
// The bucket that holds the r-th largest key splits the candidates: those above it are members of the
// top-r set for sure, those below it are not, and the few dozen inside it are decided exactly.  Two
// grid-wide launches over all slices at once; each walks the LIST in tiles of 2048 entries, eight
// consecutive entries per thread, so the work is spread evenly however unevenly the candidates are
// spread over the chunks:
//
//   k_run_count   every block picks the bucket for itself while its first tile is on its way.  The sure
//                 members are counted per chunk (a thread adds its eight entries to their
//                 chunks' counts, one addition per chunk it meets), the candidates inside the bucket go
//                 to a short list.  The last block of a slice finds the r-th element of the whole order
//                 -- larger magnitude first, then lower index -- on the list: its key is the exact
//                 threshold tau, its index the last one at which a key equal to tau still is a member.
//                 It adds the listed members to their chunks' counts and turns the counts into an
//                 exclusive prefix over the chunks.
//   k_run_emit    the position of a member in index order is the number of members before it: those of
//                 the chunks before (the prefix) plus those before it in its own run (a segmented prefix
//                 over the tile; for the one run that may reach back into earlier tiles, at most 4095
//                 entries, the block counts the members among them again).  The members the subset
//                 chose go through a per-warp queue and become messages; their residual slots are
//                 zeroed; in a step call the run table of the messages is kept for the aggregation.
// A block walks several tiles (k_run_count fetches the next one while it works on the current one):
// these kernels are chains of dependent memory round trips, and one wave of blocks pays the slice's
// set-up once.
//
// Whatever does not fit this scheme -- the first bracket missed (too few or too many candidates), the
// r-th largest key lies above the bracket, or more than kListMax candidates share the bucket (heavy
// ties) -- is left to k_finish, which handles every case; a slice finished here is skipped there.
#pragma once

#include "common.cuh"
#include "select.cuh"

namespace rtopk {

constexpr int kRunThreads = 256;
constexpr int kRunWarps = kRunThreads / 32;
constexpr int kRunPer = 8;                                   // consecutive list entries per thread
constexpr int kRunTile = kRunThreads * kRunPer;              // list entries per tile
constexpr int kScanPer = 16;                                 // loads in flight per thread of the prefix over the chunks
constexpr int kRankMax = 512;                                // lists up to this length are ranked by counting

// Exclusive prefix of v over the block's threads, and the block's total.  `s` holds kRunWarps words.
__device__ __forceinline__ uint32_t run_block_scan(uint32_t v, uint32_t* s, uint32_t& total) {
  const uint32_t lane = threadIdx.x & 31u, warp = threadIdx.x >> 5;
  const uint32_t incl = warp_incl_scan(v);
  __syncthreads();
  if (lane == 31) s[warp] = incl;
  __syncthreads();
  uint32_t off = 0, t = 0;
#pragma unroll
  for (uint32_t w = 0; w < (uint32_t)kRunWarps; ++w) { const uint32_t x = s[w]; if (w < warp) off += x; t += x; }
  total = t;
  return off + incl - v;
}

// The digit D of a complete kBins-bin histogram in shared memory with count(> D) < need <= count(>= D),
// and count(> D); D = 0xFFFFFFFF if the histogram holds fewer than `need` keys.  `s` holds 16 words.
__device__ __forceinline__ void run_pick(const uint32_t* hist, uint32_t need, uint32_t* s, uint32_t& D, uint32_t& above) {
  static_assert(kBins == 8 * kRunThreads, "eight bins per thread");
  const uint32_t tid = threadIdx.x, lane = tid & 31u, warp = tid >> 5;
  const int hi = kBins - 1 - 8 * (int)tid;                       // thread 0 holds the largest digits
  uint32_t h[8], mine = 0;
#pragma unroll
  for (int i = 0; i < 8; ++i) { h[i] = hist[hi - i]; mine += h[i]; }
  uint32_t incl = warp_incl_scan(mine);
  __syncthreads();
  if (lane == 31) s[warp] = incl;
  if (tid == 0) { s[8] = 0xFFFFFFFFu; s[9] = 0; }
  __syncthreads();
  for (uint32_t w = 0; w < warp; ++w) incl += s[w];
  const uint32_t excl = incl - mine;
  if (excl < need && need <= incl) {
    uint32_t run = excl;
#pragma unroll
    for (int i = 0; i < 8; ++i) {
      if (run + h[i] >= need) { s[8] = (uint32_t)(hi - i); s[9] = run; break; }
      run += h[i];
    }
  }
  __syncthreads();
  D = s[8]; above = s[9];
  __syncthreads();
}

// The histogram over the bracket where the streaming pass has not counted it (bf16 gradients: that pass is
// bound by instruction issue there, and the counting cost it more than this launch takes); also clears the
// chunks' member counts.  The keys above the bracket are not counted: their number is the rest of the list.
// grid: (blocks per slice, n_slices); a block takes tile after tile of kRunThreads * kHistPer candidates
constexpr int kHistPer = 8;
__global__ void __launch_bounds__(kRunThreads) k_run_hist(Launch L) {
  __shared__ uint32_t hist[kBins];
  const uint32_t sl = blockIdx.y, tid = threadIdx.x;
  const Slice S = L.s.slices[sl];
  const uint32_t n_cand = L.s.cursor[sl];
  const uint32_t tau_lo = L.s.state[sl].tau_lo, tau_hi = max(tau_lo, L.s.state[sl].tau_hi);
  if (S.r == S.len) return;
  if (n_cand < S.r || n_cand > S.cand_cap) return;               // the bracket missed: left to k_finish
  {
    uint32_t* cm = L.s.chunk_pre + S.chunk_begin;                  // members per chunk: counted by k_run_count
    const uint32_t nchunks = slice_chunks(S);
    for (uint32_t c = blockIdx.x * kRunThreads + tid; c < nchunks; c += gridDim.x * kRunThreads) cm[c] = 0;
  }
  constexpr uint32_t kTile = kRunThreads * kHistPer;
  const uint32_t nblocks = min(gridDim.x, (n_cand + kTile - 1u) / kTile);
  if (blockIdx.x >= nblocks) return;
  const uint32_t sh = bracket_shift(tau_lo, tau_hi);
  for (uint32_t b = tid; b < (uint32_t)kBins; b += kRunThreads) hist[b] = 0;
  __syncthreads();
  const float* rv = L.s.raw_val + S.cand_off;
  for (uint32_t i0 = blockIdx.x * kTile; i0 < n_cand; i0 += gridDim.x * kTile) {
    float v[kHistPer];
#pragma unroll
    for (int u = 0; u < kHistPer; ++u) { const uint32_t i = i0 + u * kRunThreads + tid; v[u] = i < n_cand ? rv[i] : 0.f; }
#pragma unroll
    for (int u = 0; u < kHistPer; ++u) {
      const uint32_t key = mag_key(v[u]);
      if (i0 + u * kRunThreads + tid < n_cand && key >= tau_lo && key <= tau_hi) atomicAdd(&hist[(key - tau_lo) >> sh], 1u);
    }
  }
  __syncthreads();
  uint32_t* gh = L.s.hist + (size_t)sl * kBins;
  for (uint32_t b = tid; b < (uint32_t)kBins; b += kRunThreads) { const uint32_t c = hist[b]; if (c) atomicAdd(gh + b, c); }
}

// Eight consecutive entries of a slice's candidate list, starting at entry i0 (a multiple of 8; the
// lists start on 128-byte boundaries and their capacities are multiples of 32 entries).
__device__ __forceinline__ void run_load8(const float* rv, const uint32_t* ri, uint32_t i0, uint32_t n_cand,
                                          float (&v)[kRunPer], uint32_t (&ix)[kRunPer]) {
  static_assert(kRunPer == 8, "two 16-byte vectors per array");
  if (i0 < n_cand) {
    const float4 a = *reinterpret_cast<const float4*>(rv + i0), b = *reinterpret_cast<const float4*>(rv + i0 + 4);
    const uint4 c = *reinterpret_cast<const uint4*>(ri + i0), e = *reinterpret_cast<const uint4*>(ri + i0 + 4);
    v[0] = a.x; v[1] = a.y; v[2] = a.z; v[3] = a.w; v[4] = b.x; v[5] = b.y; v[6] = b.z; v[7] = b.w;
    ix[0] = c.x; ix[1] = c.y; ix[2] = c.z; ix[3] = c.w; ix[4] = e.x; ix[5] = e.y; ix[6] = e.z; ix[7] = e.w;
  } else {
#pragma unroll
    for (int u = 0; u < kRunPer; ++u) { v[u] = 0.f; ix[u] = 0u; }
  }
}

constexpr uint32_t kNoChunk = 0xFFFFFFFFu;

// grid: (blocks per slice, n_slices); a block takes tile after tile of the slice's list
__global__ void __launch_bounds__(kRunThreads, 4) k_run_count(Launch L) {
  __shared__ uint32_t hist[kBins];                                 // (last block: rounds over the list)
  __shared__ uint32_t keys[kListMax];
  __shared__ uint32_t idxs[kListMax];
  __shared__ uint32_t s[16];
  const uint32_t sl = blockIdx.y, tid = threadIdx.x;
  const Slice S = L.s.slices[sl];
  const uint32_t n_cand = L.s.cursor[sl];
  const uint32_t tau_lo = L.s.state[sl].tau_lo, tau_hi = max(tau_lo, L.s.state[sl].tau_hi);
  Fin* F = L.s.fin + sl;
  if (S.r == S.len) return;
  if (n_cand < S.r || n_cand > S.cand_cap) return;               // the bracket missed: left to k_finish
  const uint32_t n_tiles = (n_cand + kRunTile - 1) / kRunTile;
  const uint32_t nblocks = min(gridDim.x, n_tiles);
  if (blockIdx.x >= nblocks) return;
  uint32_t* cm = L.s.chunk_pre + S.chunk_begin;
  const float* rv = L.s.raw_val + S.cand_off;
  const uint32_t* ri = L.s.raw_idx + S.cand_off;
  uint32_t* lkey = L.s.list + (size_t)sl * 2 * kListMax;
  uint32_t* lidx = lkey + kListMax;
  float v[kRunPer], vn[kRunPer];
  uint32_t ix[kRunPer], ixn[kRunPer];
  run_load8(rv, ri, blockIdx.x * (uint32_t)kRunTile + tid * (uint32_t)kRunPer, n_cand, v, ix);
  // While the first tile is on its way: the bucket of the bracket's histogram that holds the r-th largest
  // key.  Every block picks it for itself (8 KB of histogram and one block scan cost less than a launch, or
  // a last-block hand-over, of their own); the answer is the same in every block of the slice.
  const uint32_t* gh = L.s.hist + (size_t)sl * kBins;
  uint32_t part = 0, inside;
#pragma unroll
  for (int i = 0; i < kBins / kRunThreads; ++i) { const uint32_t h = __ldcg(gh + tid + i * kRunThreads); hist[tid + i * kRunThreads] = h; part += h; }
  run_block_scan(part, s, inside);
  if (tid == 0) hist[kBins - 1] = n_cand - inside;                 // the keys above the bracket: the rest of the list
  __syncthreads();
  uint32_t D, b_above;
  run_pick(hist, S.r, s, D, b_above);
  if (D >= (uint32_t)(kBins - 1)) return;                         // the r-th largest key lies above the bracket (or is missing)
  const uint32_t b_n = hist[D];
  if (b_n > (uint32_t)kListMax) return;                            // heavy ties
  const uint32_t sh = bracket_shift(tau_lo, tau_hi);
  const uint32_t b_lo = tau_lo + (D << sh), b_hi = min(tau_hi + 1u, b_lo + (1u << sh));
  const uint32_t width = b_hi - b_lo;
  __syncthreads();                                                 // (hist is used again by the last block)
  for (uint32_t tile = blockIdx.x; tile < n_tiles; tile += gridDim.x) {
    const uint32_t i0 = tile * (uint32_t)kRunTile + tid * (uint32_t)kRunPer;
    const uint32_t nx = tile + gridDim.x;                          // the next tile is under way while this one is counted
    run_load8(rv, ri, nx < n_tiles ? nx * (uint32_t)kRunTile + tid * (uint32_t)kRunPer : n_cand, n_cand, vn, ixn);
    uint32_t cur = kNoChunk, acc = 0;
#pragma unroll
    for (int u = 0; u < kRunPer; ++u) {
      const bool in = i0 + u < n_cand;
      const uint32_t key = mag_key(v[u]);
      const uint32_t chunk = in ? (ix[u] + S.head) / (uint32_t)kChunk : kNoChunk;
      if (chunk != cur) {
        if (acc) atomicAdd(cm + cur, acc);                         // (acc is zero while cur is no chunk)
        cur = chunk; acc = 0;
      }
      acc += in && key >= b_hi;
      if (in && key - b_lo < width) {                              // inside the bucket: a few dozen per slice
        const uint32_t at = atomicAdd(&F->list_n, 1u);
        if (at < (uint32_t)kListMax) { lkey[at] = key; lidx[at] = ix[u]; }
      }
    }
    if (acc) atomicAdd(cm + cur, acc);
#pragma unroll
    for (int u = 0; u < kRunPer; ++u) { v[u] = vn[u]; ix[u] = ixn[u]; }
  }
  __syncthreads();
  if (tid == 0) {
    __threadfence();
    s[15] = atomicAdd(&F->done2, 1u) == nblocks - 1u;
    if (s[15]) __threadfence();
  }
  __syncthreads();
  if (!s[15]) return;

  // ---- the last block of the slice: the r-th element on the list, the listed members, the prefix
  SelState* st = &L.s.state[sl];
  const uint32_t n = __ldcg(&F->list_n), need = S.r - b_above;   // rank of the target inside the bucket, from the top
  auto fail = [&]() {
    if (tid == 0) { atomicOr(L.s.error, ERR_SELECT_INCONSISTENT); st->resolved = 32; }
  };
  if (n != b_n || n < need) { fail(); return; }                   // cannot happen: the bucket was counted
  for (uint32_t t = tid; t < n; t += kRunThreads) { keys[t] = __ldcg(lkey + t); idxs[t] = __ldcg(lidx + t); }
  __syncthreads();
  if (tid == 0) { s[10] = 0; s[11] = 0; s[12] = 0; s[13] = 0xFFFFFFFFu; }
  __syncthreads();
  uint32_t tau, cut;
  if (n <= (uint32_t)kRankMax) {
    // rank by counting: how many listed candidates come before this one in the whole order
    for (uint32_t t = tid; t < n; t += kRunThreads) {
      const uint32_t k = keys[t], ix = idxs[t];
      uint32_t before = 0;
      for (uint32_t x = 0; x < n; ++x) before += keys[x] > k || (keys[x] == k && idxs[x] < ix);
      if (before == need - 1u) { s[10] = k; s[11] = ix; }
    }
    __syncthreads();
    tau = s[10]; cut = s[11];
  } else {
    // histogram rounds over the list alone (equal buckets over what is left of the interval) ...
    uint32_t found = b_lo, end = b_hi, rank = need;
    bool ok = true;
    while (end - found > 1u) {
      const uint32_t w = end - found;
      uint32_t s2 = 0;
      while (((w - 1u) >> s2) >= (uint32_t)kBins) ++s2;
      __syncthreads();
      for (uint32_t bk = tid; bk < (uint32_t)kBins; bk += kRunThreads) hist[bk] = 0;
      __syncthreads();
      for (uint32_t t = tid; t < n; t += kRunThreads) {
        const uint32_t rel = keys[t] - found;
        if (rel < w) atomicAdd(&hist[rel >> s2], 1u);
      }
      __syncthreads();
      uint32_t D, ab;
      run_pick(hist, rank, s, D, ab);
      if (D == 0xFFFFFFFFu) { ok = false; break; }
      rank -= ab;
      found += D << s2;
      end = min(end, found + (1u << s2));
    }
    if (!ok) { fail(); return; }
    tau = found;
    // ... then the rank-th lowest index among the keys equal to tau
    uint32_t* ties = hist;
    __syncthreads();
    if (tid == 0) s[12] = 0;
    __syncthreads();
    for (uint32_t t = tid; t < n; t += kRunThreads)
      if (keys[t] == tau) ties[atomicAdd(&s[12], 1u)] = idxs[t];
    __syncthreads();
    const uint32_t nt = s[12];
    for (uint32_t t = tid; t < nt; t += kRunThreads) {
      const uint32_t mine = ties[t];
      uint32_t lower = 0;
      for (uint32_t x = 0; x < nt; ++x) lower += ties[x] < mine;
      if (lower == rank - 1u) s[13] = mine;
    }
    __syncthreads();
    cut = s[13];
  }
  // the listed members join their chunks' counts
  uint32_t n_above = 0;
  for (uint32_t t = tid; t < n; t += kRunThreads) {
    n_above += keys[t] > tau;
    if (keys[t] > tau || (keys[t] == tau && idxs[t] <= cut)) atomicAdd(cm + (idxs[t] + S.head) / (uint32_t)kChunk, 1u);
  }
  uint32_t listed_above;
  (void)run_block_scan(n_above, s, listed_above);
  const uint32_t n_gt = b_above + listed_above, quota = need - listed_above;   // keys above tau; keys equal to tau inside the top-r set
  __threadfence();
  __syncthreads();
  // Exclusive prefix over the chunks' member counts.  A warp takes a contiguous span, 32 chunks at a time
  // (one line per load: a thread-contiguous split costs 32 memory transactions per load, and this one
  // block works alone): the spans' totals first, then the prefix inside each span.
  const uint32_t nchunks = slice_chunks(S);
  const uint32_t lane = tid & 31u, warp = tid >> 5;
  const uint32_t span = ((nchunks + kRunWarps * 32u - 1u) / (kRunWarps * 32u)) * 32u;
  const uint32_t w_lo = min(nchunks, warp * span), w_hi = min(nchunks, w_lo + span);
  uint32_t sum = 0;
  for (uint32_t c0 = w_lo; c0 < w_hi; c0 += 32u * kScanPer) {
#pragma unroll
    for (int u = 0; u < kScanPer; ++u) { const uint32_t c = c0 + u * 32u + lane; sum += c < w_hi ? __ldcg(cm + c) : 0u; }
  }
  sum = warp_sum(sum);
  __syncthreads();
  if (lane == 0) s[warp] = sum;
  __syncthreads();
  uint32_t off = 0, total = 0;
#pragma unroll
  for (uint32_t w = 0; w < (uint32_t)kRunWarps; ++w) { const uint32_t x = s[w]; if (w < warp) off += x; total += x; }
  if (total != S.r) { fail(); return; }                           // (block-uniform)
  for (uint32_t c0 = w_lo; c0 < w_hi; c0 += 32u * kScanPer) {
    uint32_t x[kScanPer];
#pragma unroll
    for (int u = 0; u < kScanPer; ++u) { const uint32_t c = c0 + u * 32u + lane; x[u] = c < w_hi ? __ldcg(cm + c) : 0u; }
#pragma unroll
    for (int u = 0; u < kScanPer; ++u) {
      const uint32_t c = c0 + u * 32u + lane, incl = warp_incl_scan(x[u]);
      if (c < w_hi) cm[c] = off + incl - x[u];
      off += __shfl_sync(0xFFFFFFFFu, incl, 31);
    }
  }
  if (tid != 0) return;
  Fin f = {};
  f.tau = tau; f.cut = cut; f.ok = 1;
  L.s.fin[sl] = f;
  // what rtopk_get_stats reports, and the threshold history
  st->prefix = tau; st->resolved = 31; st->n_gt = n_gt; st->need = quota;
  st->n_cand = L.s.cursor[sl]; st->n_cand_first = st->n_cand; st->flags |= FLAG_FINISHED;
  if (L.reuse) {
    TauHistory h = L.s.history[sl];
    const uint32_t pred = st->pred;
    if (pred != 0) {
      const float rel = fabsf(__uint_as_float(tau) / __uint_as_float(pred) - 1.0f);
      h.err = rel == rel ? fmaxf(rel, 0.7f * h.err) : 0.2f;
    } else if (h.valid == 0 && h.err == 0.0f) {
      h.err = 0.03f;                                               // nothing known yet about this slice
    }
    h.tau2 = h.valid >= 1 ? h.tau1 : 0u;
    h.tau1 = tau;
    h.valid = min(h.valid + 1u, 2u);
    L.s.history[sl] = h;
  }
}

// Inclusive segmented sum over the block's threads: every thread brings the count of its last segment
// (`val`) and whether a segment starts inside it (`flag`); returns, for the thread, the count carried
// into its first entry from the threads before -- the entries since the last segment start there.
// `s` holds kRunWarps words.  Counts stay below 2^31 (bit 31 carries the flag).
__device__ __forceinline__ uint32_t run_segmented_carry(uint32_t val, bool flag, uint32_t* s) {
  const uint32_t lane = threadIdx.x & 31u, warp = threadIdx.x >> 5;
  uint32_t x = val | (flag ? 0x80000000u : 0u);
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    const uint32_t y = __shfl_up_sync(0xFFFFFFFFu, x, o);
    if (lane >= (uint32_t)o) x = (x & 0x80000000u) ? x : ((x + (y & 0x7FFFFFFFu)) | (y & 0x80000000u));
  }
  __syncthreads();
  if (lane == 31) s[warp] = x;
  __syncthreads();
  uint32_t carry = 0;                                             // from the warps before
  for (uint32_t w = 0; w < warp; ++w) { const uint32_t y = s[w]; carry = (y & 0x80000000u) ? (y & 0x7FFFFFFFu) : carry + y; }
  uint32_t ex = __shfl_up_sync(0xFFFFFFFFu, x, 1);                // from the lanes before
  if (lane == 0) ex = 0;
  return (ex & 0x80000000u) ? (ex & 0x7FFFFFFFu) : carry + ex;
}

// grid: (blocks per slice, n_slices); a block takes tile after tile of the slice's list
__global__ void __launch_bounds__(kRunThreads, 5) k_run_emit(Launch L) {
  __shared__ uint32_t s[16];
  __shared__ uint32_t q_idx[kRunWarps][32 * kRunPer];              // per warp: the chosen members of its part of the tile
  __shared__ float q_val[kRunWarps][32 * kRunPer];
  __shared__ uint32_t q_pos[kRunWarps][32 * kRunPer];
  const uint32_t sl = blockIdx.y, tid = threadIdx.x, lane = tid & 31u, warp = tid >> 5;
  const Slice S = L.s.slices[sl];
  const uint32_t n_cand = L.s.cursor[sl];
  const uint32_t flags = L.s.state[sl].flags;
  const uint32_t tau = L.s.fin[sl].tau, cut = L.s.fin[sl].cut;
  if (S.r == S.len) return;
  if (!(flags & FLAG_FINISHED)) return;                          // left to k_finish
  const uint32_t n_tiles = (n_cand + kRunTile - 1) / kRunTile;
  if (blockIdx.x >= n_tiles) return;
  const uint32_t* cm = L.s.chunk_pre + S.chunk_begin;              // members in the chunks before
  const uint32_t* ri = L.s.raw_idx + S.cand_off;
  const float* rv = L.s.raw_val + S.cand_off;
  const uint32_t* sel = L.s.sel + S.sel_off;
  const uint32_t* sel_pre = L.s.sel_pre + S.sel_off;
  const bool sel_all = S.k == S.r;
  const uint32_t below = (1u << lane) - 1u;
  auto member = [&](uint32_t key, uint32_t idx) { return key > tau || (key == tau && idx <= cut); };
  for (uint32_t tile = blockIdx.x; tile < n_tiles; tile += gridDim.x) {
    const uint32_t base = tile * (uint32_t)kRunTile, i0 = base + tid * (uint32_t)kRunPer;
    // Besides its eight entries a thread fetches the entry in front of them (is its first entry the start
    // of a run?) and one of the 256 entries in front of the tile (the tile's first run may begin there).
    float v[kRunPer];
    uint32_t ix[kRunPer];
    run_load8(rv, ri, i0, n_cand, v, ix);
    const uint32_t prev = lane == 0 && tid != 0 && i0 < n_cand ? ri[i0 - 1] : 0u;
    const bool back = base > tid;
    const float bv = back ? rv[base - 1u - tid] : 0.f;
    const uint32_t bi = back ? ri[base - 1u - tid] : 0u;
    // segments: the runs' parts inside the tile.  The tile's first entry starts no segment here.
    uint32_t bits = 0, heads = 0, chunk_prev = 0;
#pragma unroll
    for (int u = 0; u < kRunPer; ++u) {
      const bool in = i0 + u < n_cand;
      const uint32_t chunk = in ? (ix[u] + S.head) / (uint32_t)kChunk : kNoChunk;
      if (in && member(mag_key(v[u]), ix[u])) bits |= 1u << u;
      if (u > 0 && chunk != chunk_prev) heads |= 1u << u;
      if (u == 0) {
        if (tid == 0) s[12] = chunk;
      }
      chunk_prev = chunk;
    }
    {
      uint32_t before = __shfl_up_sync(0xFFFFFFFFu, chunk_prev, 1);   // the last chunk of the thread in front
      if (lane == 0) before = (prev + S.head) / (uint32_t)kChunk;
      const uint32_t first = i0 < n_cand ? (ix[0] + S.head) / (uint32_t)kChunk : kNoChunk;
      if (tid != 0 && first != before) heads |= 1u;
    }
    // the members of the chunks before, for every member (neighbours ask for the same word)
    uint32_t p[kRunPer];
#pragma unroll
    for (int u = 0; u < kRunPer; ++u) p[u] = (bits >> u) & 1u ? cm[(ix[u] + S.head) / (uint32_t)kChunk] : 0u;
    // members of the thread's last segment, and the count carried in from the threads before
    const uint32_t last = heads ? 31u - (uint32_t)__clz(heads) : 0u;
    const uint32_t carry = run_segmented_carry((uint32_t)__popc(bits >> last), heads != 0u, s);
    // the tile's first run in front of the tile: its members are counted again.  Its entries there are the
    // ones next to the tile that lie in the same chunk; a run longer than the 256 fetched is walked on.
    const uint32_t c_first = s[12];
    const bool same = back && (bi + S.head) / (uint32_t)kChunk == c_first;
    uint32_t before = (uint32_t)__syncthreads_count(same && member(mag_key(bv), bi));
    uint32_t reach = (uint32_t)__syncthreads_count(same);
    for (uint32_t off = kRunThreads; reach == off && off < (uint32_t)kChunk; off += kRunThreads) {
      const bool in = base > off + tid;
      const uint32_t idx = in ? ri[base - 1u - off - tid] : 0u;
      const bool more = in && (idx + S.head) / (uint32_t)kChunk == c_first;
      before += (uint32_t)__syncthreads_count(more && member(mag_key(rv[base - 1u - off - tid]), idx));
      reach += (uint32_t)__syncthreads_count(more);
    }
    // positions, then which of them the subset chose
    uint32_t rank = carry, words[kRunPer];
#pragma unroll
    for (int u = 0; u < kRunPer; ++u) {
      if ((heads >> u) & 1u) rank = 0;
      if ((bits >> u) & 1u) {
        p[u] += rank + ((ix[u] + S.head) / (uint32_t)kChunk == c_first ? before : 0u);
        ++rank;
        if (p[u] >= S.r) bits &= ~(1u << u);                       // (cannot happen: exactly r members)
      }
    }
#pragma unroll
    for (int u = 0; u < kRunPer; ++u) words[u] = !sel_all && ((bits >> u) & 1u) ? sel[p[u] >> 5] : 0xFFFFFFFFu;
    uint32_t qn = 0;
#pragma unroll
    for (int u = 0; u < kRunPer; ++u) {
      const bool chosen = ((bits >> u) & 1u) && ((words[u] >> (p[u] & 31u)) & 1u);
      const uint32_t bal = __ballot_sync(0xFFFFFFFFu, chosen);
      if (chosen) {
        const uint32_t at = qn + (uint32_t)__popc(bal & below);
        q_idx[warp][at] = ix[u]; q_val[warp][at] = v[u]; q_pos[warp][at] = p[u];
      }
      qn += (uint32_t)__popc(bal);
    }
    __syncwarp();
    for (uint32_t q = lane; q < qn; q += 32u) {
      const uint32_t pos = q_pos[warp][q], idx = q_idx[warp][q];
      uint32_t slot = pos;
      if (!sel_all) slot = sel_pre[pos >> 5] + (uint32_t)__popc(sel[pos >> 5] & ((1u << (pos & 31u)) - 1u));
      if (slot < S.k) {
        L.msg_idx[(size_t)(S.msg_off + slot) * L.msg_stride] = S.idx_base + idx;
        L.msg_val[(size_t)(S.msg_off + slot) * L.msg_stride] = q_val[warp][q];
        L.residual[S.m_off + idx] = 0.0f;
        note_message(L, S, slot, S.idx_base + idx);
      }
    }
    __syncwarp();
  }
}

}  // namespace rtopk
