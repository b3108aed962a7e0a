// k_stream: the one pass over the W x d gradient and residual matrices (Algorithm 1's g + m).
//
// Persistent blocks; each has one producer warp and eight consumer warps.  The producer takes chunk
// tickets from a global counter (blocks run at different speeds: a fixed assignment ends with the
// slowest block's share) and stages the chunk's residual and gradient bytes into shared
// memory with 1-D bulk async copies (TMA) that complete on an mbarrier; a ring of kStages buffers
// keeps loads in flight while the consumers work.  The consumers form a = g + m, store it back,
// flag the keys >= the sampled threshold, and append them -- in index order inside the chunk
// (packed prefix sums) -- to a run of the slice's raw candidate buffer reserved with one atomicAdd
// per chunk.  The run's start and length go into a per-chunk table and its length is also added to
// the total of its chunk group; the finishing kernels number the members of the top-r set by chunk and
// by place inside the run (finish.cuh) or lay the runs out in chunk order first (k_finish), so the
// result does not depend on the order in which chunks happened to reserve their runs.  No block
// ever waits on another block.
//
// The only waits are on the block's own mbarriers; they are bounded, and on expiry the error flag
// is raised and the block leaves through a path every consumer takes together.
#pragma once

#include "common.cuh"
#include "element.cuh"

namespace rtopk {

constexpr int kStages = 2;
constexpr int kConsumers = kThreads;             // 256 = 8 warps
constexpr int kStreamThreads = kConsumers + 32;  // + producer warp
constexpr int kWaitLimit = 1 << 24;

struct StageDesc { uint32_t slice, chunk, valid, pad; };

template <typename GradT>
struct alignas(128) StreamSmem {
  alignas(128) float m[kStages][kChunk];
  alignas(128) GradT g[kStages][kChunk];
  alignas(8) unsigned long long full[kStages];
  unsigned long long empty[kStages];
  StageDesc desc[kStages];
  uint32_t wA[2][kWarps];
  uint32_t ex[2];
};

__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }
__device__ __forceinline__ void mbar_init(unsigned long long* bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(bar)), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_arrive(unsigned long long* bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_u32(bar)) : "memory");
}
__device__ __forceinline__ void mbar_arrive_expect_tx(unsigned long long* bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_u32(bar)), "r"(bytes) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(unsigned long long* bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(ok) : "r"(smem_u32(bar)), "r"(parity) : "memory");
  return ok != 0;
}
// Bounded wait for the phase with the given parity to complete.
__device__ __forceinline__ bool mbar_wait(unsigned long long* bar, uint32_t parity, int limit = kWaitLimit) {
  for (int i = 0; i < limit; ++i)
    if (mbar_try_wait(bar, parity)) return true;
  return false;
}
// A last, shorter wait of a block that is giving up (see the consumers' exit in k_stream): if the phase
// was never armed it simply runs out.
constexpr int kDrainLimit = 1 << 16;
__device__ __forceinline__ void mbar_drain(unsigned long long* bar, uint32_t parity) {
  for (int i = 0; i < kDrainLimit; ++i)
    if (mbar_try_wait(bar, parity)) return;
}
// L2 eviction policy of the candidate runs: they are small and k_finish reads them back, so they
// should outlive the gradient / residual traffic (which is loaded and stored with streaming hints).
__device__ __forceinline__ unsigned long long l2_policy_evict_last() {
  unsigned long long p;
  asm volatile("createpolicy.fractional.L2::evict_last.b64 %0, 1.0;" : "=l"(p));
  return p;
}
__device__ __forceinline__ void st_hint(uint32_t* ptr, uint32_t v, unsigned long long policy) {
  asm volatile("st.global.L2::cache_hint.u32 [%0], %1, %2;" ::"l"(ptr), "r"(v), "l"(policy) : "memory");
}
// 1-D bulk async copy global -> shared (TMA); src, dst 16-byte aligned, bytes a multiple of 16.
__device__ __forceinline__ void bulk_load(void* dst, const void* src, uint32_t bytes, unsigned long long* bar) {
  asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
               ::"r"(smem_u32(dst)), "l"(src), "r"(bytes), "r"(smem_u32(bar)) : "memory");
}
// Barrier over the consumer threads only (the producer warp never joins it).
__device__ __forceinline__ void consumer_sync() {
  asm volatile("bar.sync 1, %0;" ::"n"(kConsumers) : "memory");
}
// ... with an OR-reduction of a predicate: every consumer learns whether any of them failed.
__device__ __forceinline__ bool consumer_any(bool flag) {
  uint32_t out;
  asm volatile(
      "{\n\t.reg .pred p, q;\n\t"
      "setp.ne.u32 q, %1, 0;\n\t"
      "bar.red.or.pred p, 2, %2, q;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(out) : "r"((uint32_t)flag), "n"(kConsumers) : "memory");
  return out != 0;
}

template <typename GradT> struct SmemGrad;
template <> struct SmemGrad<float> {
  static __device__ __forceinline__ float4 ld4(const float* p) { return *reinterpret_cast<const float4*>(p); }
  static __device__ __forceinline__ float ld1(const float* p) { return *p; }
};
template <> struct SmemGrad<__nv_bfloat16> {
  static __device__ __forceinline__ float4 ld4(const __nv_bfloat16* p) {
    const uint2 v = *reinterpret_cast<const uint2*>(p);
    float4 f;
    f.x = __uint_as_float(v.x << 16); f.y = __uint_as_float(v.x & 0xFFFF0000u);
    f.z = __uint_as_float(v.y << 16); f.w = __uint_as_float(v.y & 0xFFFF0000u);
    return f;
  }
  static __device__ __forceinline__ float ld1(const __nv_bfloat16* p) {
    return __uint_as_float((uint32_t)(*reinterpret_cast<const uint16_t*>(p)) << 16);
  }
};

// GIVEUP is the instance the test of the give-up path runs (RTOPK_OPT_TEST_STREAM_GIVEUP): its consumers
// treat their first wait as run out and its producer waits only briefly for them, so every block takes the
// exit a real expiry would take -- error flag, a last bounded wait for the bulk copies still on their way
// into the block's shared memory, return -- while all copies do arrive.
// HIST (f32 gradients): the call is finished by the run kernels (finish.cuh).  Every candidate inside the bracket
// [tau_lo, tau_hi] is then also counted in the slice's histogram over the bracket (one reduction into
// global memory per such candidate: a third of the candidates, 0.4 % of the coordinates; the keys above
// the bracket need no counting, their number is the rest of the list), and the chunk's member count is
// cleared for k_run_count.  The table was cleared by the kernel in front of this one.
template <typename GradT, bool GIVEUP, bool HIST>
__global__ void __launch_bounds__(kStreamThreads, 3) k_stream(Launch L, uint32_t total_tiles, uint32_t uniform_chunks) {
  extern __shared__ __align__(128) unsigned char smem_raw[];
  StreamSmem<GradT>& sm = *reinterpret_cast<StreamSmem<GradT>*>(smem_raw);
  const uint32_t tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  if (tid == 0) {
    for (int s = 0; s < kStages; ++s) { mbar_init(&sm.full[s], 1); mbar_init(&sm.empty[s], kWarps); }
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  __syncthreads();
  const Slice* slices = L.s.slices;

  if (warp == kWarps) {
    // ------------------------------------------------------------------ producer (one lane)
    if (lane != 0) return;
    const char* grad = static_cast<const char*>(L.grad);
    // The first chunk of a block is its own number; the following ones are tickets drawn from a
    // global counter, so that blocks that run ahead take more chunks and all blocks end together.
    // The next ticket is drawn while the current stage is still in use (its latency is hidden).
    uint32_t tile = blockIdx.x;
    for (uint32_t i = 0;; ++i) {
      const uint32_t stage = i % kStages, phase = (i / kStages) & 1u;
      const uint32_t next_tile = tile < total_tiles ? gridDim.x + atomicAdd(&L.s.tickets[3], 1u) : tile;
      if (!mbar_wait(&sm.empty[stage], phase ^ 1u, GIVEUP ? kDrainLimit : kWaitLimit)) {
        // the consumers never freed the stage: give up, but not before the copies issued into the two stages
        // (iterations i - 1 and i - 2) have landed in this block's shared memory
        atomicOr(L.s.error, ERR_WAIT_TIMEOUT);
        if (i >= 1) mbar_drain(&sm.full[(i - 1) % kStages], ((i - 1) / kStages) & 1u);
        if (i >= 2) mbar_drain(&sm.full[(i - 2) % kStages], ((i - 2) / kStages) & 1u);
        return;
      }
      if (tile >= total_tiles) {
        sm.desc[stage].valid = 0;
        mbar_arrive(&sm.full[stage]);
        return;
      }
      const uint32_t sl = uniform_chunks ? tile / uniform_chunks
                                         : find_slice(L.n_slices, tile, [&](uint32_t s) { return slices[s].chunk_begin; });
      const Slice* S = slices + sl;
      const uint32_t head = S->head, span = head + S->len;
      const uint32_t c = tile - S->chunk_begin;
      const uint32_t e0 = c * (uint32_t)kChunk;
      const uint32_t n_el = min((uint32_t)kChunk, span - e0);
      const uint32_t bytes_m = (n_el * 4u + 15u) & ~15u;
      const uint32_t bytes_g = (n_el * (uint32_t)sizeof(GradT) + 15u) & ~15u;
      sm.desc[stage].slice = sl; sm.desc[stage].chunk = c; sm.desc[stage].valid = 1;
      mbar_arrive_expect_tx(&sm.full[stage], bytes_m + bytes_g);
      bulk_load(sm.m[stage], L.residual + (S->m_off - head) + e0, bytes_m, &sm.full[stage]);
      bulk_load(sm.g[stage], grad + ((S->g_off - head) + (int64_t)e0) * (int64_t)sizeof(GradT), bytes_g, &sm.full[stage]);
      tile = next_tile;
    }
  }

  // -------------------------------------------------------------------- consumers
  const unsigned long long keep = l2_policy_evict_last();
  uint32_t cur_slice = 0xFFFFFFFFu;
  Slice S;
  uint32_t tau = 0x80000000u, tau_hi = 0x80000000u, sh = 0;
  for (uint32_t i = 0;; ++i) {
    const uint32_t stage = i % kStages, phase = (i / kStages) & 1u, buf = i & 1u;
    const bool arrived = GIVEUP ? false : mbar_wait(&sm.full[stage], phase);
    if (consumer_any(!arrived)) {                 // every consumer leaves together
      if (tid == 0) atomicOr(L.s.error, ERR_WAIT_TIMEOUT);
      // ... but not while a bulk copy into this block's shared memory may still be on its way: the copies
      // the producer has issued into both stages get one more (bounded) wait before the block ends
      mbar_drain(&sm.full[stage], phase);
      mbar_drain(&sm.full[(i + 1) % kStages], ((i + 1) / kStages) & 1u);
      return;
    }
    const StageDesc d = sm.desc[stage];
    if (!d.valid) return;
    if (d.slice != cur_slice) {
      cur_slice = d.slice;
      S = slices[cur_slice];
      tau = L.s.state[cur_slice].tau_lo;
      if (HIST) { tau_hi = max(tau, L.s.state[cur_slice].tau_hi); sh = bracket_shift(tau, tau_hi); }
    }
    const uint32_t head = S.head, span = head + S.len;
    const uint32_t e_w = d.chunk * (uint32_t)kChunk + warp * (uint32_t)kWarpSpan;   // element on the slice's grid
    const uint32_t l_w = warp * (uint32_t)kWarpSpan;                                 // same, inside the chunk
    float a[kIter][4];
#pragma unroll
    for (int it = 0; it < kIter; ++it) {
      const uint32_t l = l_w + it * 128u + lane * 4u;
      const float4 m4 = *reinterpret_cast<const float4*>(&sm.m[stage][l]);
      const float4 g4 = SmemGrad<GradT>::ld4(&sm.g[stage][l]);
      a[it][0] = ef_add(g4.x, m4.x); a[it][1] = ef_add(g4.y, m4.y);
      a[it][2] = ef_add(g4.z, m4.z); a[it][3] = ef_add(g4.w, m4.w);
    }
    __syncwarp();
    if (lane == 0) mbar_arrive(&sm.empty[stage]);      // the stage may be refilled from here on
    float* res = L.residual + (S.m_off - head);
    uint32_t maskA = 0;
#pragma unroll
    for (int it = 0; it < kIter; ++it) {
      const uint32_t e = e_w + it * 128u + lane * 4u;
      uint32_t valid;
      if (e >= head && e + 4u <= span) {
        valid = 0xFu;
        __stcs(reinterpret_cast<float4*>(res + e), make_float4(a[it][0], a[it][1], a[it][2], a[it][3]));
      } else {
        valid = 0;
#pragma unroll
        for (int j = 0; j < 4; ++j)
          if (e + j >= head && e + j < span) { valid |= 1u << j; res[e + j] = a[it][j]; }
      }
#pragma unroll
      for (int j = 0; j < 4; ++j)
        maskA |= (uint32_t)(((valid >> j) & 1u) && mag_key(a[it][j]) >= tau) << (it * 4 + j);
    }
    uint32_t packA = 0;
#pragma unroll
    for (int it = 0; it < kIter; ++it) packA |= (uint32_t)__popc((maskA >> (it * 4)) & 0xFu) << (it * 8);
    const uint32_t inclA = warp_incl_scan(packA);
    const uint32_t totA = __shfl_sync(0xFFFFFFFFu, inclA, 31);
    const uint32_t exLaneA = inclA - packA;
    uint32_t wA = 0;
#pragma unroll
    for (int it = 0; it < kIter; ++it) wA += (totA >> (it * 8)) & 0xFFu;
    if (lane == 0) sm.wA[buf][warp] = wA;
    consumer_sync();
    if (tid == 0) {
      uint32_t bA = 0;
#pragma unroll
      for (int w = 0; w < kWarps; ++w) bA += sm.wA[buf][w];
      uint32_t start = 0;
      if (bA) {
        start = atomicAdd(&L.s.cursor[cur_slice], bA);
        atomicAdd(&L.s.group_total[S.group_begin + (d.chunk >> S.gshift)], bA);
      }
      const uint32_t tile = S.chunk_begin + d.chunk;
      L.s.chunk_start[tile] = start;
      L.s.chunk_count[tile] = bA;
      if (HIST) L.s.chunk_pre[tile] = 0;
      sm.ex[buf] = start;
    }
    consumer_sync();
    if (maskA) {
      uint32_t before = sm.ex[buf];
      for (uint32_t w = 0; w < warp; ++w) before += sm.wA[buf][w];
      uint32_t* cidx = L.s.raw_idx + S.cand_off;
      float* cval = L.s.raw_val + S.cand_off;
      uint32_t* gh = L.s.hist + (size_t)cur_slice * kBins;
#pragma unroll
      for (int it = 0; it < kIter; ++it) {
        uint32_t bits = (maskA >> (it * 4)) & 0xFu;
        uint32_t pos = before + ((exLaneA >> (it * 8)) & 0xFFu);
        const uint32_t e = e_w + it * 128u + lane * 4u - head;
        while (bits) {                                             // (a candidate or two per warp and vector)
          const uint32_t j = (uint32_t)__ffs(bits) - 1u;
          bits &= bits - 1u;
          const float lo2 = j & 1u ? a[it][1] : a[it][0], hi2 = j & 1u ? a[it][3] : a[it][2];
          const uint32_t vb = __float_as_uint(j & 2u ? hi2 : lo2);
          if (pos < S.cand_cap) { st_hint(cidx + pos, e + j, keep); st_hint(reinterpret_cast<uint32_t*>(cval) + pos, vb, keep); }
          ++pos;
          if (HIST) {
            const uint32_t key = vb & 0x7FFFFFFFu;
            if (key <= tau_hi) atomicAdd(gh + ((key - tau) >> sh), 1u);
          }
        }
        before += (totA >> (it * 8)) & 0xFFu;
      }
    }
  }
}

}  // namespace rtopk
