// Shared device-side definitions of the rTop-k library: slice descriptors, selection state,
// scans and Philox4x32-10.
#pragma once

#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

namespace rtopk {

// ----------------------------------------------------------------------------- geometry
constexpr int kThreads = 256;                 // threads per block of the streaming kernels
constexpr int kWarps = kThreads / 32;
constexpr int kIter = 4;                      // 4-element vectors per thread per chunk
constexpr int kWarpSpan = 32 * kIter * 4;     // 512 consecutive elements per warp
constexpr int kChunk = kWarps * kWarpSpan;    // 4096 elements per block of the collect kernels
constexpr int kHistChunks = 4;                // chunks per unit of work of the histogram pass (k_bracket)
constexpr int kGroupsMax = 2048;              // chunk groups per slice (two per thread of k_finish)

// radix digits of the 31-bit magnitude key, most significant first: 11 + 11 + 9 bits
constexpr int kBins = 2048;
__host__ __device__ constexpr int digit_bits(int pass) { return pass < 2 ? 11 : 9; }
__host__ __device__ constexpr int digit_shift(int pass) { return pass == 0 ? 20 : (pass == 1 ? 9 : 0); }
__host__ __device__ constexpr int resolved_before(int pass) { return pass == 0 ? 0 : (pass == 1 ? 11 : 22); }

constexpr uint32_t kNoQuota = 0xFFFFFFFFu;
constexpr int kSampleMax = 32768;             // sampled elements per slice (threshold estimate)
constexpr int kSampleThreads = 1024;

// stage of the full-vector radix select of one slice
enum : uint32_t { STAGE_PASS0 = 0, STAGE_PASS1 = 1, STAGE_PASS2 = 2, STAGE_COLLECT = 3, STAGE_DONE = 4 };
enum : uint32_t { FLAG_GENERAL = 1u, FLAG_FELL_BACK = 2u, FLAG_FINISHED = 4u /* finished by the run kernels (finish.cuh) */ };
enum : uint32_t { ERR_WAIT_TIMEOUT = 1u, ERR_CANDIDATE_OVERFLOW = 2u, ERR_SELECT_INCONSISTENT = 4u };

// One slice: a worker row, or one tensor of a worker row.  Offsets are in elements.
struct Slice {
  int64_t g_off;        // slice start relative to the gradient base pointer
  int64_t m_off;        // slice start relative to the residual base pointer
  uint32_t len;         // number of coordinates d_s
  uint32_t r, k;
  uint32_t row;         // local row (worker_base + row is the global worker id)
  uint32_t segment;
  uint32_t idx_base;    // index of the slice's first coordinate in the whole vector
  uint32_t head;        // (slice start) mod 4: elements of the first aligned vector before the slice
  uint32_t msg_off;     // start of the slice's k pairs in the flattened message arrays
  uint32_t cand_off, cand_cap;
  uint32_t chunk_begin; // first collect tile (all slices are numbered one after another)
  uint32_t hist_begin;  // first histogram block
  uint32_t group_begin; // first entry of the slice in the chunk-group totals
  uint32_t samp_off;    // start in the draw buffer (k entries)
  uint32_t first_off;   // start in the first-occurrence table
  uint32_t first_mask;  // 0: the table is dense (r entries); else it is a hash table of first_mask + 1 slots
  uint32_t sel_off;     // start in the selection bitmap / its prefix counts (32-bit words)
  uint32_t gshift;      // a chunk group is 2^gshift consecutive chunks (at most kGroupsMax groups per slice)
};

// Selection state of one slice, advanced kernel by kernel.
struct SelState {
  uint32_t tau_lo;      // collect threshold: keys above it are candidates ...
  uint32_t eq_quota;    // ... and the first eq_quota keys equal to it (kNoQuota = all)
  uint32_t prefix;      // resolved high bits of the r-th largest key
  uint32_t resolved;    // how many of the 31 bits are resolved
  uint32_t n_gt;        // keys strictly above the resolved prefix bucket
  uint32_t need;        // rank of the r-th largest inside the bucket (1-based)
  uint32_t n_cand;      // candidates written
  uint32_t stage;
  uint32_t flags;
  uint32_t n_cand_first;// candidates of the sampled-threshold pass (statistics)
  uint32_t tau_hi;      // sampled upper estimate of the r-th largest key (0x7FFFFFFF = none)
  uint32_t pred;        // predicted r-th largest key when the bracket came from the history (0: from the sample)
};

// What a slice remembers from call to call when thresholds are reused: the exact r-th largest keys
// of the last two calls, a running bound of the relative prediction error, and how many of the two
// keys may be used (0: the next call samples).
struct TauHistory { uint32_t tau1, tau2; float err; uint32_t valid; };

// Where the run kernels (finish.cuh) stand with one slice.
constexpr int kListMax = 2048;        // the histogram bucket that holds the r-th largest key is resolved on a list of up to this many candidates
struct alignas(32) Fin {
  uint32_t tau, cut;         // the exact r-th largest key; a key equal to it is a member up to this index
  uint32_t ok;
  uint32_t list_n;           // entries of the slice's short list
  uint32_t done2;            // blocks of k_run_count that have completed
  uint32_t pad[3];
};

struct Scratch {
  Slice* slices;
  SelState* state;
  uint32_t* hist;         // [slices][kBins]
  uint32_t* done;         // [slices] block-completion counters
  uint32_t* tickets;      // [3] chunk counter of k_stream ([0..2] unused)
  uint32_t* cursor;       // [slices] next free entry of the raw candidate buffer (= candidates so far)
  uint32_t* group_total;  // candidates per chunk group (summed by the stream pass)
  uint32_t* chunk_start;  // [chunks] where a chunk's run sits in the raw buffer ...
  uint32_t* chunk_count;  // ... its length ...
  uint32_t* chunk_pre;    // ... and how many marked coordinates (threshold encoder) or members of the top-r set (run kernels) precede it in the slice
  uint32_t* raw_idx;      // candidates in reservation order
  float* raw_val;
  uint32_t* cand_idx;     // candidates in index order
  float* cand_val;
  uint32_t* draws;        // t_j
  uint32_t* first;        // first-occurrence table F
  uint32_t* sel;          // selection bitmap over positions
  uint32_t* sel_pre;      // exclusive popcount prefix per bitmap word
  uint32_t* sel_blk;      // selected positions per chunk of bitmap words (scan scratch)
  uint32_t* error;        // device error flags
  TauHistory* history;    // [slices] threshold history across calls
  Fin* fin;               // [slices] state of the run kernels
  uint32_t* list;         // [slices][2 * kListMax]: keys, then indices, of the candidates inside the bucket
  uint32_t* tile_inv;     // run table of the messages (Launch::tile_inv / tile_cnt), in the zeroed region
  uint32_t* tile_cnt;
};

struct Launch {
  Scratch s;
  const void* grad;
  float* residual;
  uint32_t* msg_idx;
  float* msg_val;
  uint32_t msg_stride;        // words between consecutive entries of msg_idx / msg_val: 1 (two arrays) or 2 (pairs)
  uint32_t n_slices;
  uint32_t worker_base;
  uint32_t seed_lo, seed_hi;
  uint32_t step;
  const uint32_t* step_ptr;   // not null: the round number is read from this device word instead of `step`
  uint32_t reuse;             // 1: brackets may be predicted from the slices' threshold history
  // Run table of the messages, for the aggregation that follows in a step call (null otherwise): per local
  // worker row and tile of kRunTableTile coordinates, the first place in the row of a message of that tile,
  // kept as the maximum of its complement so that the table starts from zero, and how many there are.
  uint32_t* tile_inv;
  uint32_t* tile_cnt;
  uint32_t tiles_per_row;
  uint32_t K_row;             // messages per worker row
};
constexpr uint32_t kRunTableTile = 16384;

// Called by whoever writes message `slot` of slice S for coordinate `index` (counted in the whole vector).
__device__ __forceinline__ void note_message(const Launch& L, const Slice& S, uint32_t slot, uint32_t index) {
  if (L.tile_inv == nullptr) return;
  const uint32_t place = S.msg_off - S.row * L.K_row + slot;
  const size_t at = (size_t)S.row * L.tiles_per_row + index / kRunTableTile;
  atomicMax(L.tile_inv + at, ~place);
  atomicAdd(L.tile_cnt + at, 1u);
}

// ----------------------------------------------------------------------------- small helpers
__device__ __forceinline__ uint32_t lane_id() { return threadIdx.x & 31; }
__device__ __forceinline__ uint32_t mag_key(float x) { return __float_as_uint(x) & 0x7FFFFFFFu; }

__device__ __forceinline__ uint32_t warp_incl_scan(uint32_t v) {
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    uint32_t n = __shfl_up_sync(0xFFFFFFFFu, v, o);
    if (lane_id() >= (uint32_t)o) v += n;
  }
  return v;
}

__device__ __forceinline__ uint32_t warp_sum(uint32_t v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xFFFFFFFFu, v, o);
  return v;
}

// Bucket width (log2) of the histogram over a bracket [tau_lo, tau_hi] of the r-th largest key: 2047
// equal buckets hold the bracket, the last one the keys above it.
__device__ __forceinline__ uint32_t bracket_shift(uint32_t tau_lo, uint32_t tau_hi) {
  uint32_t sh = 0;
  while (((tau_hi - tau_lo) >> sh) >= (uint32_t)(kBins - 1)) ++sh;
  return sh;
}

// index of the slice that owns global tile `t`: the last s with begin(s) <= t
template <typename F>
__device__ __forceinline__ uint32_t find_slice(uint32_t n, uint32_t t, F begin) {
  uint32_t lo = 0, hi = n;
  while (hi - lo > 1) {
    uint32_t mid = (lo + hi) >> 1;
    if (begin(mid) <= t) lo = mid; else hi = mid;
  }
  return lo;
}

// ----------------------------------------------------------------------------- digit pick
// Given a complete histogram of one digit (bins [0, nbins)) in shared memory and the rank `need`
// (1-based, counted from the largest digit), finds the digit D with
//   count(digit > D) < need <= count(digit >= D)
// and returns D and count(digit > D).  Called by every thread of the block; `scratch` holds
// blockDim.x / 32 + 2 words.  Returns false if the histogram holds fewer than `need` keys.
__device__ __forceinline__ bool pick_digit(const uint32_t* hist, int nbins, uint32_t need, uint32_t* scratch,
                                           uint32_t& D, uint32_t& above) {
  const int nthreads = blockDim.x;
  const int per = (nbins + nthreads - 1) / nthreads;
  // thread t owns bins [hi - per + 1, hi] counted from the top: t = 0 holds the largest digits
  const int hi = nbins - 1 - (int)threadIdx.x * per;
  uint32_t mine = 0;
  for (int i = 0; i < per; ++i) {
    const int b = hi - i;
    if (b >= 0) mine += hist[b];
  }
  // inclusive scan over threads (from the top digits downwards)
  uint32_t incl = warp_incl_scan(mine);
  const uint32_t warp = threadIdx.x >> 5, nwarps = (nthreads + 31) >> 5;
  if (lane_id() == 31) scratch[warp] = incl;
  if (threadIdx.x == 0) {
    scratch[nwarps] = 0xFFFFFFFFu;      // result: digit
    scratch[nwarps + 1] = 0;            // result: above
  }
  __syncthreads();
  uint32_t woff = 0;
  for (uint32_t w = 0; w < warp; ++w) woff += scratch[w];
  incl += woff;
  const uint32_t excl = incl - mine;
  if (excl < need && need <= incl) {     // the crossing lies in this thread's bins
    uint32_t run = excl;
    for (int i = 0; i < per; ++i) {
      const int b = hi - i;
      if (b < 0) break;
      const uint32_t h = hist[b];
      if (run + h >= need) { scratch[nwarps] = (uint32_t)b; scratch[nwarps + 1] = run; break; }
      run += h;
    }
  }
  __syncthreads();
  D = scratch[nwarps];
  above = scratch[nwarps + 1];
  __syncthreads();
  return D != 0xFFFFFFFFu;
}

// ----------------------------------------------------------------------------- Philox4x32-10
// Salmon, Moraes, Dror, Shaw, "Parallel Random Numbers: As Easy as 1, 2, 3" (SC'11): ten rounds;
// each multiplies counter words 0 and 2 by the two round multipliers, XORs the high halves with
// words 1 and 3 and the round key, and bumps the key by the Weyl constants.
__device__ __forceinline__ uint2 philox4x32_10_lo(uint32_t c0, uint32_t c1, uint32_t c2, uint32_t c3,
                                                  uint32_t k0, uint32_t k1) {
#pragma unroll
  for (int i = 0; i < 10; ++i) {
    const uint32_t h0 = __umulhi(0xD2511F53u, c0), l0 = 0xD2511F53u * c0;
    const uint32_t h1 = __umulhi(0xCD9E8D57u, c2), l1 = 0xCD9E8D57u * c2;
    c0 = h1 ^ c1 ^ k0; c1 = l1;
    c2 = h0 ^ c3 ^ k1; c3 = l0;
    k0 += 0x9E3779B9u; k1 += 0xBB67AE85u;
  }
  return make_uint2(c0, c1);   // output words 0 and 1
}

// Floyd iteration j draws uniformly from {0..j}: floor(u64 * (j+1) / 2^64), u64 = (x1 << 32) | x0.
__device__ __forceinline__ uint32_t floyd_draw(uint32_t j, uint32_t worker, uint32_t segment, uint32_t step,
                                               uint32_t seed_lo, uint32_t seed_hi) {
  const uint2 x = philox4x32_10_lo(j, worker, segment, step, seed_lo, seed_hi);
  const unsigned long long u = ((unsigned long long)x.y << 32) | x.x;
  return (uint32_t)__umul64hi(u, (unsigned long long)j + 1ull);
}

}  // namespace rtopk
