// Finishing a slice straight from the runs of the streaming pass (Definition 1's top-r set, then the
// members Definition 3's subset chose), without laying the candidates out in index order first.
//
// The streaming pass leaves, per chunk of 4096 coordinates, a run of candidates (index, value) in
// index order, and the sampled or predicted bracket [tau_lo, tau_hi] of the r-th largest key.  A
// histogram of the candidates over the bracket -- 2047 equal buckets plus one for the keys above --
// gives the bucket that holds the r-th largest key, and that bucket splits the candidates: those above
// it are members of the top-r set for sure, those below it are not, and the few dozen inside it are
// decided exactly.  Three grid-wide launches over all slices at once, each about one wave of blocks:
//
//   k_run_hist    the histogram (block-local first, the keys above the bracket counted in registers).
//   k_run_count   every block picks the bucket for itself (8 KB of histogram and one block scan cost
//                 less than a launch of its own).  Then eight lanes per chunk walk the chunk's run: the
//                 sure members are counted, the candidates inside the bucket go to a short list with
//                 their indices.  The last block of a slice finds the r-th element of the whole order --
//                 larger magnitude first, then lower index -- on the list: its key is the exact
//                 threshold tau, its index the last one at which a key equal to tau still is a member.
//                 It adds the listed members to their chunks' counts and turns the totals of the chunk
//                 groups into a prefix.
//   k_run_emit    eight lanes per chunk again: the position of a member in index order is the number of
//                 members before it (groups before, chunks before, rank in its run), so the members of a
//                 run take consecutive positions and their bits lie in two or three words of the
//                 subset's bitmap, fetched once per run; the chosen ones become messages and their
//                 residual slots are zeroed.
// A run holds about 1 % of a chunk, 40 to 50 candidates.  Eight lanes read it one 32-byte sector at a
// time, four runs per warp: a whole warp per run leaves a third of the lanes idle and costs several
// times the instructions (these kernels are bound by instruction issue, not by bytes), a thread per run
// scatters every load over 32 sectors.
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
constexpr int kRunChunks = 4;                                // chunks per group (one warp step): members are totalled per group, then per slice
constexpr int kRunBlockGroups = 32;                          // groups per block (four per warp)
constexpr int kHistPer = 8;                                  // candidates per thread and tile of k_run_hist
constexpr int kRunBatch = 8;                                 // entries of a run a thread reads at a time
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

// grid: (blocks per slice, n_slices); a block takes tile after tile of kRunThreads * kHistPer candidates
__global__ void __launch_bounds__(kRunThreads) k_run_hist(Launch L) {
  __shared__ uint32_t hist[kBins];
  const uint32_t sl = blockIdx.y, tid = threadIdx.x, lane = tid & 31u;
  const Slice S = L.s.slices[sl];
  if (S.r == S.len) return;
  const uint32_t n_cand = L.s.cursor[sl];
  if (n_cand < S.r || n_cand > S.cand_cap) return;               // the bracket missed: left to k_finish
  constexpr uint32_t kTile = kRunThreads * kHistPer;
  if (blockIdx.x * kTile >= n_cand) return;
  const uint32_t tau_lo = L.s.state[sl].tau_lo, tau_hi = max(tau_lo, L.s.state[sl].tau_hi);
  const uint32_t sh = bracket_shift(tau_lo, tau_hi);
  for (uint32_t b = tid; b < (uint32_t)kBins; b += kRunThreads) hist[b] = 0;
  __syncthreads();
  const float* rv = L.s.raw_val + S.cand_off;
  uint32_t n_hi = 0;                                               // the keys above the bracket share one bucket
  for (uint32_t i0 = blockIdx.x * kTile; i0 < n_cand; i0 += gridDim.x * kTile) {
    float v[kHistPer];
#pragma unroll
    for (int u = 0; u < kHistPer; ++u) { const uint32_t i = i0 + u * kRunThreads + tid; v[u] = i < n_cand ? rv[i] : 0.f; }
#pragma unroll
    for (int u = 0; u < kHistPer; ++u) {
      const uint32_t key = mag_key(v[u]);
      if (i0 + u * kRunThreads + tid < n_cand) {
        if (key > tau_hi) ++n_hi;
        else if (key >= tau_lo) atomicAdd(&hist[(key - tau_lo) >> sh], 1u);
      }
    }
  }
  n_hi = warp_sum(n_hi);
  if (lane == 0 && n_hi) atomicAdd(&hist[kBins - 1], n_hi);
  __syncthreads();
  uint32_t* gh = L.s.hist + (size_t)sl * kBins;
  for (uint32_t b = tid; b < (uint32_t)kBins; b += kRunThreads) { const uint32_t c = hist[b]; if (c) atomicAdd(gh + b, c); }
}

// The bucket of the bracket's histogram that holds the r-th largest key.  `ok` is false where the run
// kernels do not go on.
struct Bucket { uint32_t lo, hi, above, n; bool ok; };
__device__ __forceinline__ Bucket run_bucket(const Launch& L, uint32_t sl, const Slice& S, uint32_t* hist, uint32_t* s) {
  const uint32_t tid = threadIdx.x;
  const uint32_t n_cand = L.s.cursor[sl];
  const uint32_t tau_lo = L.s.state[sl].tau_lo, tau_hi = max(tau_lo, L.s.state[sl].tau_hi);
  const uint32_t* gh = L.s.hist + (size_t)sl * kBins;
#pragma unroll
  for (int i = 0; i < kBins / kRunThreads; ++i) hist[tid + i * kRunThreads] = gh[tid + i * kRunThreads];
  __syncthreads();
  uint32_t D, above;
  run_pick(hist, S.r, s, D, above);
  const uint32_t sh = bracket_shift(tau_lo, tau_hi);
  Bucket b;
  b.ok = n_cand >= S.r && n_cand <= S.cand_cap && D < (uint32_t)(kBins - 1);   // else: missed, or above the bracket
  b.n = b.ok ? hist[D] : 0u;
  b.ok = b.ok && b.n <= (uint32_t)kListMax;                                    // else: heavy ties
  b.lo = tau_lo + (D << sh);
  b.hi = min(tau_hi + 1u, b.lo + (1u << sh));
  b.above = above;
  return b;
}

// Sum over the four octets' leaders / over an octet (8 neighbouring lanes).
__device__ __forceinline__ uint32_t octet_sum(uint32_t v) {
  v += __shfl_xor_sync(0xFFFFFFFFu, v, 4); v += __shfl_xor_sync(0xFFFFFFFFu, v, 2); v += __shfl_xor_sync(0xFFFFFFFFu, v, 1);
  return v;
}
__device__ __forceinline__ uint32_t octets_max(uint32_t v) {     // v is the same on the lanes of an octet
  v = max(v, __shfl_xor_sync(0xFFFFFFFFu, v, 8)); v = max(v, __shfl_xor_sync(0xFFFFFFFFu, v, 16));
  return v;
}

// grid: (ceil(most groups of a slice / kRunBlockGroups), n_slices); a warp step is one group of four
// chunks, eight lanes per chunk
__global__ void __launch_bounds__(kRunThreads) k_run_count(Launch L) {
  __shared__ uint32_t keys[kListMax];
  __shared__ uint32_t idxs[kListMax];
  __shared__ uint32_t hist[kBins];
  __shared__ uint32_t s[16];
  const uint32_t sl = blockIdx.y, tid = threadIdx.x, lane = tid & 31u, warp = tid >> 5;
  const Slice S = L.s.slices[sl];
  if (S.r == S.len) return;
  const uint32_t nchunks = slice_chunks(S);
  const uint32_t ngroups = (nchunks + kRunChunks - 1) / kRunChunks;
  const uint32_t nblocks = (ngroups + kRunBlockGroups - 1) / kRunBlockGroups;
  if (blockIdx.x >= nblocks) return;
  const Bucket b = run_bucket(L, sl, S, hist, s);
  if (!b.ok) return;                                             // (the same in every block of the slice)
  Fin* F = L.s.fin + sl;
  const uint32_t* cs = L.s.chunk_start + S.chunk_begin;
  const uint32_t* cc = L.s.chunk_count + S.chunk_begin;
  uint32_t* cm = L.s.chunk_pre + S.chunk_begin;
  const float* rv = L.s.raw_val + S.cand_off;
  const uint32_t* ri = L.s.raw_idx + S.cand_off;
  uint32_t* lkey = L.s.list + (size_t)sl * 2 * kListMax;
  uint32_t* lidx = lkey + kListMax;
  uint32_t* pt = L.s.part_tot + S.part_begin;
  const uint32_t width = b.hi - b.lo;
  const uint32_t oct = lane >> 3, sub = lane & 7u;
  const uint32_t g_end = min(ngroups, (blockIdx.x + 1u) * (uint32_t)kRunBlockGroups);
  uint32_t g = blockIdx.x * (uint32_t)kRunBlockGroups + warp;
  // the place of the next run is fetched while the current one is walked
  uint32_t c = g * (uint32_t)kRunChunks + oct;
  uint32_t start = g < g_end && c < nchunks ? cs[c] : 0u, cnt = g < g_end && c < nchunks ? cc[c] : 0u;
  for (; g < g_end; g += kRunWarps) {
    const uint32_t start_c = start, cnt_c = cnt, c_c = c;
    c = (g + kRunWarps) * (uint32_t)kRunChunks + oct;
    const bool more = g + kRunWarps < g_end && c < nchunks;
    start = more ? cs[c] : 0u;
    cnt = more ? cc[c] : 0u;
    const uint32_t steps = (octets_max(cnt_c) + 7u) >> 3;
    uint32_t sure = 0;
    for (uint32_t st = 0; st < steps; st += 2) {                   // two sectors per lane in flight
      const uint32_t j0 = st * 8u + sub, j1 = j0 + 8u;
      const bool in0 = j0 < cnt_c, in1 = j1 < cnt_c;
      const float x0 = in0 ? rv[start_c + j0] : 0.f, x1 = in1 ? rv[start_c + j1] : 0.f;
      const uint32_t k0 = mag_key(x0), k1 = mag_key(x1);
      sure += (in0 && k0 >= b.hi) + (in1 && k1 >= b.hi);
      if (in0 && k0 - b.lo < width) {                              // inside the bucket: a few dozen per slice
        const uint32_t at = atomicAdd(&F->list_n, 1u);
        if (at < (uint32_t)kListMax) { lkey[at] = k0; lidx[at] = ri[start_c + j0]; }
      }
      if (in1 && k1 - b.lo < width) {
        const uint32_t at = atomicAdd(&F->list_n, 1u);
        if (at < (uint32_t)kListMax) { lkey[at] = k1; lidx[at] = ri[start_c + j1]; }
      }
    }
    sure = octet_sum(sure);
    if (sub == 0 && c_c < nchunks) cm[c_c] = sure;
    uint32_t tot = sure;                                           // over the four octets
    tot += __shfl_xor_sync(0xFFFFFFFFu, tot, 8); tot += __shfl_xor_sync(0xFFFFFFFFu, tot, 16);
    if (lane == 0) pt[g] = tot;
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
  const uint32_t n = __ldcg(&F->list_n), need = S.r - b.above;   // rank of the target inside the bucket, from the top
  auto fail = [&]() {
    if (tid == 0) { atomicOr(L.s.error, ERR_SELECT_INCONSISTENT); st->resolved = 32; }
  };
  if (n != b.n || n < need) { fail(); return; }                   // cannot happen: the bucket was counted
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
    uint32_t found = b.lo, end = b.hi, rank = need;
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
  // the listed members join their chunks' and groups' counts
  uint32_t n_above = 0;
  for (uint32_t t = tid; t < n; t += kRunThreads) {
    n_above += keys[t] > tau;
    if (keys[t] > tau || (keys[t] == tau && idxs[t] <= cut)) {
      const uint32_t chunk = (idxs[t] + S.head) / (uint32_t)kChunk;
      atomicAdd(cm + chunk, 1u);
      atomicAdd(pt + chunk / (uint32_t)kRunChunks, 1u);
    }
  }
  uint32_t dummy;
  (void)run_block_scan(n_above, s, dummy);
  const uint32_t n_gt = b.above + dummy, quota = need - dummy;    // keys above tau; keys equal to tau inside the top-r set
  __threadfence();
  __syncthreads();
  // exclusive prefix over the groups' totals, a window of 8 per thread at a time
  uint32_t carry = 0;
  for (uint32_t p0 = 0; p0 < ngroups; p0 += 8u * kRunThreads) {
    uint32_t mine[8], sum = 0;
#pragma unroll
    for (int u = 0; u < 8; ++u) { const uint32_t p = p0 + tid * 8u + u; mine[u] = p < ngroups ? __ldcg(pt + p) : 0u; sum += mine[u]; }
    uint32_t total;
    uint32_t ex = carry + run_block_scan(sum, s, total);
#pragma unroll
    for (int u = 0; u < 8; ++u) { const uint32_t p = p0 + tid * 8u + u; if (p < ngroups) pt[p] = ex; ex += mine[u]; }
    carry += total;
  }
  if (carry != S.r) { fail(); return; }                           // (block-uniform)
  if (tid != 0) return;
  Fin f;
  f.tau = tau; f.cut = cut; f.ok = 1; f.list_n = 0; f.done2 = 0;
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

// grid: as k_run_count
__global__ void __launch_bounds__(kRunThreads) k_run_emit(Launch L) {
  const uint32_t sl = blockIdx.y, tid = threadIdx.x, lane = tid & 31u, warp = tid >> 5;
  const Slice S = L.s.slices[sl];
  if (S.r == S.len) return;
  if (!(L.s.state[sl].flags & FLAG_FINISHED)) return;            // left to k_finish
  const uint32_t nchunks = slice_chunks(S);
  const uint32_t ngroups = (nchunks + kRunChunks - 1) / kRunChunks;
  if (blockIdx.x * (uint32_t)kRunBlockGroups >= ngroups) return;
  const uint32_t tau = L.s.fin[sl].tau, cut = L.s.fin[sl].cut;
  const uint32_t* cs = L.s.chunk_start + S.chunk_begin;
  const uint32_t* cc = L.s.chunk_count + S.chunk_begin;
  const uint32_t* cm = L.s.chunk_pre + S.chunk_begin;
  const uint32_t* ri = L.s.raw_idx + S.cand_off;
  const float* rv = L.s.raw_val + S.cand_off;
  const uint32_t* sel = L.s.sel + S.sel_off;
  const uint32_t* sel_pre = L.s.sel_pre + S.sel_off;
  const uint32_t* pt = L.s.part_tot + S.part_begin;
  const bool sel_all = S.k == S.r;
  const uint32_t sel_words = (S.r + 31u) >> 5;
  const uint32_t oct = lane >> 3, sub = lane & 7u, below = (1u << sub) - 1u;
  const uint32_t g_end = min(ngroups, (blockIdx.x + 1u) * (uint32_t)kRunBlockGroups);
  uint32_t g = blockIdx.x * (uint32_t)kRunBlockGroups + warp;
  // the place and the member counts of the next group are fetched while the current one is walked
  uint32_t c = g * (uint32_t)kRunChunks + oct;
  bool has = g < g_end && c < nchunks;
  uint32_t start = has ? cs[c] : 0u, cnt = has ? cc[c] : 0u, mem = has ? cm[c] : 0u, gbase = g < g_end ? pt[g] : 0u;
  for (; g < g_end; g += kRunWarps) {
    const uint32_t start_c = start, cnt_c = cnt, mem_c = mem, gbase_c = gbase;
    c = (g + kRunWarps) * (uint32_t)kRunChunks + oct;
    has = g + kRunWarps < g_end && c < nchunks;
    start = has ? cs[c] : 0u; cnt = has ? cc[c] : 0u; mem = has ? cm[c] : 0u;
    gbase = g + kRunWarps < g_end ? pt[g + kRunWarps] : 0u;
    // members before this run: the groups before, then the octets before it in the group
    const uint32_t m0 = __shfl_sync(0xFFFFFFFFu, mem_c, 0), m1 = __shfl_sync(0xFFFFFFFFu, mem_c, 8),
                   m2 = __shfl_sync(0xFFFFFFFFu, mem_c, 16);
    uint32_t p_run = gbase_c + (oct > 0 ? m0 : 0u) + (oct > 1 ? m1 : 0u) + (oct > 2 ? m2 : 0u);
    // The run's members take positions p_run, p_run + 1, ...: lanes 0..3 of the octet hold the bitmap words
    // that cover the first of them, lanes 4..7 those words' running popcounts (longer runs read on demand).
    const uint32_t w0 = p_run >> 5;
    uint32_t held = 0;
    if (!sel_all && mem_c) {
      const uint32_t w = w0 + (sub & 3u);
      if (w < sel_words) held = sub < 4u ? sel[w] : sel_pre[w];
    }
    const uint32_t steps = (octets_max(cnt_c) + 7u) >> 3;
    for (uint32_t st = 0; st < steps; ++st) {
      const uint32_t j = st * 8u + sub;
      const bool in = j < cnt_c;
      const float v = in ? rv[start_c + j] : 0.f;
      const uint32_t idx = in ? ri[start_c + j] : 0u;
      const uint32_t key = mag_key(v);
      const bool member = in && (key > tau || (key == tau && idx <= cut));
      const uint32_t bal = (__ballot_sync(0xFFFFFFFFu, member) >> (oct * 8u)) & 0xFFu;
      const uint32_t p = p_run + __popc(bal & below);
      p_run += __popc(bal);
      const uint32_t k = (p >> 5) - w0;                            // which of the held words (if below 4)
      uint32_t word = __shfl_sync(0xFFFFFFFFu, held, (oct << 3) + (k & 3u));
      uint32_t pre = __shfl_sync(0xFFFFFFFFu, held, (oct << 3) + 4u + (k & 3u));
      if (member && p < S.r) {
        uint32_t slot = p;
        bool chosen = true;
        if (!sel_all) {
          if (k >= 4u) { word = sel[p >> 5]; pre = sel_pre[p >> 5]; }
          chosen = (word >> (p & 31u)) & 1u;
          slot = pre + __popc(word & ((1u << (p & 31u)) - 1u));
        }
        if (chosen && slot < S.k) {
          L.msg_idx[(size_t)(S.msg_off + slot) * L.msg_stride] = S.idx_base + idx;
          L.msg_val[(size_t)(S.msg_off + slot) * L.msg_stride] = v;
          L.residual[S.m_off + idx] = 0.0f;
        }
      }
    }
  }
}

}  // namespace rtopk
