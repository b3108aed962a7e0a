// Host side of the rTop-k library: argument checks, scratch layout, and the launch sequence of
// one round of Algorithm 1's communication path (node body for W workers, then the master's
// average).  All device work is enqueued on the caller's stream; nothing here synchronises
// except the explicitly documented status / statistics reads.
#include "../../include/rtopk.h"

#include <cuda_runtime.h>

#include <algorithm>
#include <cmath>
#include <cstdio>
#include <cstring>
#include <mutex>
#include <new>
#include <type_traits>
#include <vector>

#include "aggregate.cuh"
#include "codec.cuh"
#include "common.cuh"
#include "finish.cuh"
#include "sampler.cuh"
#include "select.cuh"
#include "stream.cuh"
#include "threshold.cuh"

using namespace rtopk;

struct rtopk_ctx {
  int device = 0;
  int64_t d_max = 0, r_max = 0, k_max = 0;
  int32_t W_max = 0, S_max = 0;
  int select_path = 0;
  int finish_path = 0;                // RTOPK_OPT_FINISH_PATH
  int test_giveup = 0;                // RTOPK_OPT_TEST_STREAM_GIVEUP
  int last_cuda_error = 0;
  // device scratch (one allocation each)
  Slice* d_slices = nullptr;
  SelState* d_state = nullptr;
  char* d_zero = nullptr;        // counters, histograms, bitmaps: cleared per call
  size_t zero_bytes = 0;
  uint32_t* d_first = nullptr;   // first-occurrence tables: all 0xFF before the subset kernels run
  size_t first_clean = 0;        // leading entries that a call has left at 0xFF for the next one
  const uint32_t* run_inv = nullptr;   // run table of the messages of the last sparsify call that kept one
  const uint32_t* run_cnt = nullptr;
  size_t first_entries = 0;
  uint32_t* d_cand_idx = nullptr;
  float* d_cand_val = nullptr;
  uint32_t* d_raw_idx = nullptr;
  float* d_raw_val = nullptr;
  uint32_t* d_sent = nullptr;        // one bit per coordinate: updated by the sparse aggregation under momentum
  uint32_t* d_chunk_tab = nullptr;   // chunk_start | chunk_count | chunk_pre
  size_t chunk_tab_entries = 0;
  size_t cand_entries = 0;
  uint32_t* d_draws = nullptr;
  uint32_t* d_sel_pre = nullptr;
  uint32_t* d_sel_blk = nullptr;
  size_t sel_blk_entries = 0;
  size_t sel_words = 0;
  uint32_t* d_error = nullptr;
  Fin* d_fin = nullptr;              // per-slice state of the run kernels
  uint32_t* d_list = nullptr;        // per-slice short lists (keys, indices)
  TauHistory* d_history = nullptr;   // per-slice threshold history (RTOPK_OPT_REUSE_THRESHOLD)
  int reuse = 0;
  int threshold_signs = 0;            // RTOPK_OPT_THRESHOLD_SIGNS
  int device_step = 0;                // RTOPK_OPT_DEVICE_STEP
  uint32_t* d_step = nullptr;         // the round counter on the device
  bool history_stale = true;         // cleared before the next call that may use it
  const float* history_residual = nullptr;
  uint32_t* d_agg_starts = nullptr;
  size_t agg_start_entries = 0;
  void* d_stage = nullptr;       // host-call staging: two gradient buffers, messages, update
  size_t stage_bytes = 0;
  size_t stage_g_bytes = 0, stage_mi_bytes = 0;   // the layout the staging buffer is currently carved with
  // rtopk_step_host moves data on two copy streams of its own, so that the upload of the next call's
  // gradient and the download of the last call's results overlap the step between them
  cudaStream_t copy_in = nullptr, copy_out = nullptr;
  cudaEvent_t ev_uploaded[2] = {nullptr, nullptr};   // gradient buffer b holds this call's gradient
  cudaEvent_t ev_consumed[2] = {nullptr, nullptr};   // the step that read gradient buffer b has ended
  bool consumed_valid[2] = {false, false};
  cudaEvent_t ev_downloaded = nullptr;               // the results of the last call are in host memory
  int stage_next = 0;
  std::vector<Slice> cached_slices;   // what d_slices currently holds
  Slice* h_slices = nullptr;          // pinned copy of the table: the source of an upload that is captured into a graph
  size_t slices_max = 0;
  uint32_t last_n_slices = 0;
  // optional per-phase timing (RTOPK_OPT_PROFILE): events recorded on the caller's stream
  int sms = 0;
  uint64_t launches = 0;                          // kernels launched by this context so far
  int finish_max_clusters[kMaxCluster + 1] = {};  // [cs]: co-resident k_finish clusters of size cs (1..16)
  int stream_blocks[2] = {0, 0};      // persistent grid of k_stream per gradient dtype
  // work that does not depend on the data (the k-of-r subset, clearing the dense update) runs on a
  // side stream next to the streaming pass
  cudaStream_t side = nullptr;
  cudaEvent_t ev_fork = nullptr, ev_join = nullptr;
  cudaEvent_t ev_streamed = nullptr, ev_cleared = nullptr;   // the dense update is cleared beside the finishing kernels
  cudaEvent_t ev_zeroed = nullptr;                           // the side stream has cleared the late part of the zeroed region
  int profile = 0;
  cudaEvent_t ev[RTOPK_N_PHASES + 1] = {};
  bool ev_valid[RTOPK_N_PHASES + 1] = {};
};

namespace {

constexpr int kVersion = 100;
constexpr size_t kSampleSmemBytes = (size_t)(kSampleMax + 2 * kBins + 64) * sizeof(uint32_t);

size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }

int cuda_fail(rtopk_ctx* ctx, cudaError_t e) {
  if (ctx) ctx->last_cuda_error = (int)e;
  return RTOPK_ERR_CUDA;
}
#define RTOPK_CUDA(ctx, call)                                   \
  do {                                                          \
    cudaError_t e__ = (call);                                   \
    if (e__ != cudaSuccess) return cuda_fail((ctx), e__);       \
  } while (0)

// Marks the boundary before phase `i` (i = RTOPK_N_PHASES: the end of the last phase).
void mark(rtopk_ctx* ctx, int i, cudaStream_t st) {
  if (!ctx->profile) return;
  ctx->ev_valid[i] = cudaEventRecord(ctx->ev[i], st) == cudaSuccess;
}

struct DeviceGuard {
  int prev = -1;
  bool ok = true;
  explicit DeviceGuard(int dev) {
    if (cudaGetDevice(&prev) != cudaSuccess) { ok = false; return; }
    if (prev != dev && cudaSetDevice(dev) != cudaSuccess) ok = false;
  }
  ~DeviceGuard() { if (prev >= 0) cudaSetDevice(prev); }
};

uint32_t cand_capacity(uint64_t len, uint64_t r) {
  const uint64_t c = 3 * r + 4096;   // room for the sampled bracket's margin at small r / d
  return (uint32_t)(((c < len ? c : len) + 31u) & ~31ull);     // multiples of 32 keep every list 128-byte aligned
}

// First-occurrence table of the k-of-r subset: dense (r entries) while r <= 16 k, else a hash table of
// at least 2 k slots (keys | firsts).  Returns the entries it takes and sets the slice's mask.
uint64_t first_table_entries(Slice& sl) {
  if ((uint64_t)sl.r <= 16ull * sl.k) { sl.first_mask = 0; return sl.r; }
  uint32_t slots = 64;
  while (slots < 2u * sl.k) slots <<= 1;
  sl.first_mask = slots - 1;
  return 2ull * slots;
}

// Layout of one call: the slice table plus every per-call scratch offset.
struct Plan {
  std::vector<Slice> slices;
  uint32_t n_chunks = 0, n_hist_blocks = 0, n_groups = 0;
  size_t cand_entries = 0, draw_entries = 0, first_entries = 0, sel_words = 0;
  size_t table_words = 0;             // rows x tiles of the messages' run table
  uint32_t tiles_per_row = 0;
  uint32_t k_draw_max = 0, words_all_max = 0, cap_max = 0, chunks_max = 0, sel_words_max = 0;
  bool any_select = false, any_sampler = false, any_all = false;
  bool uniform = false;               // every slice has the same number of chunks (plain calls)
  uint32_t K_row = 0;
};

// `always_gather`: every slice gets a candidate list, also when r equals its length (the threshold
// encoder's r is only an upper bound of the marked set).
int make_plan(const rtopk_ctx* ctx, int64_t ld_g, int64_t ld_m, int64_t d, int32_t W, int32_t S,
              const int64_t* seg_off, const int64_t* seg_r, const int64_t* seg_k, Plan& P,
              bool always_gather = false) {
  uint64_t K = 0, R = 0;
  for (int s = 0; s < S; ++s) {
    const int64_t len = seg_off[s + 1] - seg_off[s];
    if (len < 1 || seg_k[s] < 1 || seg_k[s] > seg_r[s] || seg_r[s] > len) return RTOPK_ERR_INVALID_ARG;
    K += (uint64_t)seg_k[s];
    R += (uint64_t)seg_r[s];
  }
  if (seg_off[0] != 0 || seg_off[S] != d) return RTOPK_ERR_INVALID_ARG;
  if ((int64_t)K > ctx->k_max || (int64_t)R > ctx->r_max) return RTOPK_ERR_INVALID_ARG;
  if (K * (uint64_t)W >= (1ull << 32)) return RTOPK_ERR_INVALID_ARG;
  P.K_row = (uint32_t)K;
  P.tiles_per_row = (uint32_t)((d + kRunTableTile - 1) / kRunTableTile);
  P.table_words = (size_t)W * P.tiles_per_row;
  P.uniform = (S == 1);
  P.slices.resize((size_t)W * (size_t)S);
  uint64_t chunks = 0, hblocks = 0, groups = 0, cand = 0, draws = 0, first = 0, selw = 0;
  for (int w = 0; w < W; ++w) {
    uint64_t msg_at = (uint64_t)w * K;
    for (int s = 0; s < S; ++s) {
      Slice& sl = P.slices[(size_t)w * S + s];
      std::memset(&sl, 0, sizeof(sl));
      const int64_t lo = seg_off[s], len = seg_off[s + 1] - lo;
      sl.g_off = (int64_t)w * ld_g + lo;
      sl.m_off = (int64_t)w * ld_m + lo;
      sl.len = (uint32_t)len;
      sl.r = (uint32_t)seg_r[s];
      sl.k = (uint32_t)seg_k[s];
      sl.row = (uint32_t)w;
      sl.segment = (uint32_t)s;
      sl.idx_base = (uint32_t)lo;
      sl.head = (uint32_t)(lo & 7);   // slices sit on an 8-element grid: 16-byte bulk copies for both dtypes
      sl.msg_off = (uint32_t)msg_at;
      msg_at += sl.k;
      const uint32_t nchunks = (uint32_t)((sl.head + (uint64_t)sl.len + kChunk - 1) / kChunk);
      sl.chunk_begin = (uint32_t)chunks;
      sl.hist_begin = (uint32_t)hblocks;
      chunks += nchunks;
      if (nchunks > P.chunks_max) P.chunks_max = nchunks;
      hblocks += (nchunks + kHistChunks - 1) / kHistChunks;
      // chunk groups: the stream pass sums the candidates of 2^gshift consecutive chunks, which lets
      // k_finish place every run without a pass over the whole chunk table
      sl.gshift = 5;
      while (((nchunks + (1u << sl.gshift) - 1) >> sl.gshift) > (uint32_t)kGroupsMax) ++sl.gshift;
      sl.group_begin = (uint32_t)groups;
      groups += (nchunks + (1u << sl.gshift) - 1) >> sl.gshift;
      sl.cand_off = (uint32_t)cand;
      if (sl.r < sl.len || always_gather) {
        sl.cand_cap = cand_capacity(sl.len, sl.r);
        cand += sl.cand_cap;
        if (sl.cand_cap > P.cap_max) P.cap_max = sl.cand_cap;
        P.any_select = true;
      } else {
        sl.cand_cap = 0;
        P.any_all = true;
        const uint32_t nw = (sl.r + 31) / 32;
        if (nw > P.words_all_max) P.words_all_max = nw;
      }
      sl.samp_off = (uint32_t)draws;
      sl.first_off = (uint32_t)first;
      sl.sel_off = (uint32_t)selw;
      if (sl.k < sl.r) {
        draws += sl.k;
        first += first_table_entries(sl);
        selw += (sl.r + 31) / 32;
        if ((sl.r + 31) / 32 > P.sel_words_max) P.sel_words_max = (sl.r + 31) / 32;
        P.any_sampler = true;
        if (sl.k > P.k_draw_max) P.k_draw_max = sl.k;
      }
    }
  }
  if (chunks >= (1ull << 31) || cand >= (1ull << 32) || first >= (1ull << 32)) return RTOPK_ERR_INVALID_ARG;
  P.n_chunks = (uint32_t)chunks; P.n_hist_blocks = (uint32_t)hblocks; P.n_groups = (uint32_t)groups;
  P.cand_entries = cand; P.draw_entries = draws; P.first_entries = first; P.sel_words = selw;
  return RTOPK_OK;
}

// Carves the per-call zeroed region.  Returns the bytes used; *early_bytes is the leading part that
// holds the counters the sampling kernels clear themselves (the rest is cleared by a memset).
size_t carve_zero(const rtopk_ctx* ctx, const Plan& P, Scratch& s, size_t* early_bytes = nullptr) {
  char* p = ctx->d_zero;
  size_t at = 0;
  auto take = [&](size_t bytes) { char* q = p + at; at = align_up(at + bytes, 256); return q; };
  s.tickets = (uint32_t*)take(4 * sizeof(uint32_t));
  s.done = (uint32_t*)take(P.slices.size() * sizeof(uint32_t));
  s.cursor = (uint32_t*)take(P.slices.size() * sizeof(uint32_t));
  s.group_total = (uint32_t*)take((size_t)P.n_groups * sizeof(uint32_t));
  s.hist = (uint32_t*)take(P.slices.size() * kBins * sizeof(uint32_t));
  if (early_bytes) *early_bytes = at;
  s.sel = (uint32_t*)take(P.sel_words * sizeof(uint32_t));
  s.tile_inv = (uint32_t*)take(P.table_words * sizeof(uint32_t));
  s.tile_cnt = (uint32_t*)take(P.table_words * sizeof(uint32_t));
  return at;
}

size_t zero_region_bytes(size_t slices, size_t chunks, size_t groups, size_t sel_words, size_t table_words) {
  size_t at = 0;
  auto take = [&](size_t bytes) { at = align_up(at + bytes, 256); };
  take(16); take(slices * 4); take(slices * 4); take(groups * 4);
  take(slices * kBins * 4); take(sel_words * 4); take(table_words * 4); take(table_words * 4);
  (void)chunks;
  return at;
}

int check_common(const rtopk_ctx* ctx, const void* grad, int grad_dtype, int64_t ld_g, const float* residual,
                 int64_t ld_m, int64_t d, int32_t W, int32_t worker_base, const uint32_t* msg_idx,
                 const float* msg_val) {
  if (!ctx || !grad || !residual || !msg_idx || !msg_val) return RTOPK_ERR_INVALID_ARG;
  if (grad_dtype != RTOPK_F32 && grad_dtype != RTOPK_BF16) return RTOPK_ERR_INVALID_ARG;
  if (d < 1 || d > ctx->d_max || W < 1 || W > ctx->W_max || worker_base < 0) return RTOPK_ERR_INVALID_ARG;
  const int64_t g_mult = grad_dtype == RTOPK_F32 ? 4 : 8;
  if (ld_g < d || ld_m < d || (ld_g % g_mult) != 0 || (ld_m % 4) != 0) return RTOPK_ERR_INVALID_ARG;
  if (((uintptr_t)grad & 15u) || ((uintptr_t)residual & 15u) || ((uintptr_t)msg_idx & 3u) ||
      ((uintptr_t)msg_val & 3u))
    return RTOPK_ERR_INVALID_ARG;
  return RTOPK_OK;
}

int run_sampler(rtopk_ctx* ctx, const Plan& P, const Launch& L, cudaStream_t st, bool clear_first);

// `late.on`: the side stream draws the k-of-r subset only once the streaming pass has ended (see
// sparsify_impl); the stream does not wait for it here.  `late.hist`: the run kernels follow, so the
// streaming pass also counts the candidates' histogram over the bracket.
struct LateSide { bool on, hist; };

template <typename GradT>
int launch_select(rtopk_ctx* ctx, const Plan& P, const Launch& L, cudaStream_t st, cudaEvent_t join, LateSide late) {
  const uint32_t n = (uint32_t)P.slices.size();
  int rc = RTOPK_OK;
  auto stream_pass = [&]() -> int {
    mark(ctx, RTOPK_PHASE_STREAM, st);
    const uint32_t per = (uint32_t)((P.slices[0].head + (uint64_t)P.slices[0].len + kChunk - 1) / kChunk);
    const uint32_t uniform = P.uniform ? per : 0u;
    const int blocks = ctx->stream_blocks[sizeof(GradT) == 4 ? 0 : 1];
    if (ctx->test_giveup) k_stream<GradT, true, false><<<blocks, kStreamThreads, sizeof(StreamSmem<GradT>), st>>>(L, P.n_chunks, uniform);
    else if (sizeof(GradT) == 4 && late.hist) k_stream<float, false, true><<<blocks, kStreamThreads, sizeof(StreamSmem<float>), st>>>(L, P.n_chunks, uniform);
    else k_stream<GradT, false, false><<<blocks, kStreamThreads, sizeof(StreamSmem<GradT>), st>>>(L, P.n_chunks, uniform);
    ++ctx->launches;
    if (late.on) {
      // the streaming pass saturates the memory system and fills every SM, the kernels after it do neither:
      // what does not depend on the data runs on the side stream once the pass has ended
      RTOPK_CUDA(ctx, cudaEventRecord(ctx->ev_streamed, st));
      RTOPK_CUDA(ctx, cudaStreamWaitEvent(ctx->side, ctx->ev_streamed, 0));
      {
        RTOPK_CUDA(ctx, cudaStreamWaitEvent(st, ctx->ev_zeroed, 0));      // (recorded long ago: see sparsify_impl)
        const int rs = run_sampler(ctx, P, L, ctx->side, true);
        if (rs) return rs;
        RTOPK_CUDA(ctx, cudaEventRecord(ctx->ev_join, ctx->side));
        // behind the subset, off the path of the kernel that waits for it: the round counter, and the
        // first-occurrence tables put back to 0xFF for the next call
        if (ctx->device_step) { k_step_bump<<<1, 32, 0, ctx->side>>>(ctx->d_step); ++ctx->launches; }
        RTOPK_CUDA(ctx, cudaMemsetAsync(ctx->d_first, 0xFF, P.first_entries * sizeof(uint32_t), ctx->side));
        ctx->first_clean = P.first_entries;
      }
      RTOPK_CUDA(ctx, cudaEventRecord(ctx->ev_cleared, ctx->side));
    }
    mark(ctx, RTOPK_PHASE_ORDER, st);
    mark(ctx, RTOPK_PHASE_EXACT, st);
    return RTOPK_OK;
  };
  if (ctx->select_path == 0) {
    mark(ctx, RTOPK_PHASE_THRESHOLD, st);
    k_sample<GradT><<<n, kSampleThreads, kSampleSmemBytes, st>>>(L);
    ++ctx->launches;
    rc = stream_pass();
    if (rc) return rc;
    // k_finish needs the subset (side stream); a slice whose bracket missed is selected exactly inside
    // its k_finish cluster, so no kernel of the exact path is launched here
    if (join) RTOPK_CUDA(ctx, cudaStreamWaitEvent(st, join, 0));
  } else {
    // the bracket from a histogram over the full vector; from there on as above
    mark(ctx, RTOPK_PHASE_THRESHOLD, st);
    k_init_state<<<(n + 127) / 128, 128, 0, st>>>(L, 0u);
    ++ctx->launches;
    if (P.any_select) {
      const uint32_t hgrid = std::min<uint32_t>(P.n_hist_blocks, (uint32_t)ctx->sms * 8u);
      k_bracket<GradT><<<hgrid, kThreads, 0, st>>>(L, P.n_hist_blocks);
      ++ctx->launches;
    }
    rc = stream_pass();
    if (rc) return rc;
    if (join) RTOPK_CUDA(ctx, cudaStreamWaitEvent(st, join, 0));
  }
  return RTOPK_OK;
}

int upload_slices(rtopk_ctx* ctx, const Plan& P, cudaStream_t st) {
  const size_t bytes = P.slices.size() * sizeof(Slice);
  if (ctx->cached_slices.size() == P.slices.size() &&
      std::memcmp(ctx->cached_slices.data(), P.slices.data(), bytes) == 0)
    return RTOPK_OK;
  // An eager copy from pageable memory has left the source when the call returns; a captured one reads
  // its source at every replay, so it gets a buffer that lives as long as the context.
  cudaStreamCaptureStatus cap = cudaStreamCaptureStatusNone;
  if (st != nullptr) RTOPK_CUDA(ctx, cudaStreamIsCapturing(st, &cap));
  const Slice* src = P.slices.data();
  if (cap != cudaStreamCaptureStatusNone) {
    if (P.slices.size() > ctx->slices_max) return RTOPK_ERR_INVALID_ARG;
    std::memcpy(ctx->h_slices, P.slices.data(), bytes);
    src = ctx->h_slices;
  }
  RTOPK_CUDA(ctx, cudaMemcpyAsync(ctx->d_slices, src, bytes, cudaMemcpyHostToDevice, st));
  ctx->cached_slices = P.slices;
  ctx->history_stale = true;          // other slices: what was learnt about the old ones does not apply
  return RTOPK_OK;
}

int run_sampler(rtopk_ctx* ctx, const Plan& P, const Launch& L, cudaStream_t st, bool clear_first) {
  if (!P.any_sampler) return RTOPK_OK;
  const uint32_t n = (uint32_t)P.slices.size();
  if (clear_first && P.first_entries > ctx->first_clean)
    RTOPK_CUDA(ctx, cudaMemsetAsync(ctx->d_first, 0xFF, P.first_entries * sizeof(uint32_t), st));
  ctx->first_clean = 0;                                // used from here on
  const dim3 grid((P.k_draw_max + kDrawThreads - 1) / kDrawThreads, n);
  k_draw<<<grid, kDrawThreads, 0, st>>>(L);
  ++ctx->launches;
  k_resolve<<<grid, kDrawThreads, 0, st>>>(L);
  ++ctx->launches;
  const dim3 sgrid((P.sel_words_max + kSelChunk - 1) / kSelChunk, n);
  if ((size_t)sgrid.x * n > ctx->sel_blk_entries) return RTOPK_ERR_INVALID_ARG;
  if (sgrid.x > 1) {                                   // (a bitmap of one chunk has no chunks before it to add up)
    k_sel_count<<<sgrid, kScanThreads, 0, st>>>(L);
    ++ctx->launches;
  }
  k_sel_scan<<<sgrid, kScanThreads, 0, st>>>(L);
  ++ctx->launches;
  return RTOPK_OK;
}

// Points a launch descriptor at the context's scratch for plan P and fills in the call's arguments.
int bind_launch(rtopk_ctx* ctx, const Plan& P, const void* grad, float* residual, int32_t worker_base, uint64_t seed,
                uint32_t step, uint32_t* msg_idx, float* msg_val, Launch& L, size_t* early_bytes, size_t* zbytes) {
  std::memset(&L, 0, sizeof(L));
  *zbytes = carve_zero(ctx, P, L.s, early_bytes);
  if (*zbytes > ctx->zero_bytes) return RTOPK_ERR_INVALID_ARG;
  L.s.slices = ctx->d_slices; L.s.state = ctx->d_state;
  L.s.cand_idx = ctx->d_cand_idx; L.s.cand_val = ctx->d_cand_val;
  L.s.raw_idx = ctx->d_raw_idx; L.s.raw_val = ctx->d_raw_val;
  if ((size_t)P.n_chunks > ctx->chunk_tab_entries) return RTOPK_ERR_INVALID_ARG;
  L.s.chunk_start = ctx->d_chunk_tab;
  L.s.chunk_count = ctx->d_chunk_tab + ctx->chunk_tab_entries;
  L.s.chunk_pre = ctx->d_chunk_tab + 2 * ctx->chunk_tab_entries;
  L.s.draws = ctx->d_draws; L.s.first = ctx->d_first; L.s.sel_pre = ctx->d_sel_pre; L.s.sel_blk = ctx->d_sel_blk;
  L.s.error = ctx->d_error;
  L.s.fin = ctx->d_fin; L.s.list = ctx->d_list;
  L.grad = grad; L.residual = residual; L.msg_idx = msg_idx; L.msg_val = msg_val;
  L.msg_stride = 1;
  L.tile_inv = nullptr; L.tile_cnt = nullptr;            // set by the step calls (sparsify_impl)
  L.tiles_per_row = P.tiles_per_row; L.K_row = P.K_row;
  L.n_slices = (uint32_t)P.slices.size();
  L.worker_base = (uint32_t)worker_base;
  L.seed_lo = (uint32_t)seed; L.seed_hi = (uint32_t)(seed >> 32);
  L.step = step;
  L.step_ptr = ctx->device_step ? ctx->d_step : nullptr;
  return RTOPK_OK;
}

int sparsify_impl(rtopk_ctx* ctx, const void* grad, int grad_dtype, int64_t ld_g, float* residual, int64_t ld_m,
                  int64_t d, int32_t W, int32_t worker_base, int32_t S, const int64_t* seg_off,
                  const int64_t* seg_r, const int64_t* seg_k, uint64_t seed, uint32_t step, uint32_t* msg_idx,
                  float* msg_val, cudaStream_t st, uint32_t* K_out, uint32_t msg_stride = 1,
                  bool keep_run_table = false) {
  int rc = check_common(ctx, grad, grad_dtype, ld_g, residual, ld_m, d, W, worker_base, msg_idx, msg_val);
  if (rc) return rc;
  if (S < 1 || S > ctx->S_max || !seg_off || !seg_r || !seg_k) return RTOPK_ERR_INVALID_ARG;
  Plan P;
  rc = make_plan(ctx, ld_g, ld_m, d, W, S, seg_off, seg_r, seg_k, P);
  if (rc) return rc;
  if (P.cand_entries > ctx->cand_entries || P.first_entries > ctx->first_entries ||
      P.sel_words > ctx->sel_words)
    return RTOPK_ERR_INVALID_ARG;
  DeviceGuard guard(ctx->device);
  if (!guard.ok) return RTOPK_ERR_CUDA;
  Launch L;
  size_t early_bytes = 0, zbytes = 0;
  rc = bind_launch(ctx, P, grad, residual, worker_base, seed, step, msg_idx, msg_val, L, &early_bytes, &zbytes);
  if (rc) return rc;

  L.msg_stride = msg_stride;
  ctx->run_inv = nullptr; ctx->run_cnt = nullptr;
  if (keep_run_table) {
    // the aggregation of a step call finds every worker's entries of an output tile without searching
    L.tile_inv = L.s.tile_inv; L.tile_cnt = L.s.tile_cnt;
    ctx->run_inv = L.s.tile_inv; ctx->run_cnt = L.s.tile_cnt;
  }
  rc = upload_slices(ctx, P, st);
  if (rc) return rc;
  ctx->last_n_slices = L.n_slices;
  L.s.history = ctx->d_history;
  L.reuse = (ctx->reuse && ctx->select_path == 0) ? 1u : 0u;
  if (L.reuse) {
    // the history follows one residual buffer through consecutive calls of one shape
    if (ctx->history_stale || ctx->history_residual != residual) {
      RTOPK_CUDA(ctx, cudaMemsetAsync(ctx->d_history, 0, P.slices.size() * sizeof(TauHistory), st));
      ctx->history_stale = false;
      ctx->history_residual = residual;
    }
  } else {
    ctx->history_stale = true;
  }
  mark(ctx, RTOPK_PHASE_SUBSET, st);
  // k_sample clears the leading counters of the zeroed region itself; with the bracket from the histogram
  // pass there is no such kernel and the whole region is cleared here.  The rest (the histograms, the
  // selection bitmap, the run table of the messages) is first touched behind the streaming pass or by the
  // subset kernels: it is cleared on the side stream.
  const bool late_on_side = ctx->select_path == 0;
  if (!late_on_side) RTOPK_CUDA(ctx, cudaMemsetAsync(ctx->d_zero, 0, zbytes, st));
  // Calls that are finished by the run kernels need the subset only for the last of them, and those kernels
  // leave most of every SM idle, whereas the streaming pass wants all of it from its first microsecond: there
  // the subset is drawn beside the run kernels, not beside the start of the pass.
  const bool from_runs = P.any_select && L.n_slices <= 65535u && ctx->finish_path != 1;
  const bool sampler_late = from_runs && late_on_side && P.any_sampler;
  const bool forked = P.any_sampler && !sampler_late;
  if (forked) {
    // work that does not depend on the data runs beside the streaming pass: the k-of-r subset
    RTOPK_CUDA(ctx, cudaEventRecord(ctx->ev_fork, st));
    RTOPK_CUDA(ctx, cudaStreamWaitEvent(ctx->side, ctx->ev_fork, 0));
    if (late_on_side) RTOPK_CUDA(ctx, cudaMemsetAsync(ctx->d_zero + early_bytes, 0, zbytes - early_bytes, ctx->side));
    rc = run_sampler(ctx, P, L, ctx->side, true);
    if (rc) return rc;
    // the subset kernels are the only readers of the round counter: it advances right behind them
    if (ctx->device_step) { k_step_bump<<<1, 32, 0, ctx->side>>>(ctx->d_step); ++ctx->launches; }
    RTOPK_CUDA(ctx, cudaEventRecord(ctx->ev_join, ctx->side));
  } else if (sampler_late) {
    // the rest of the zeroed region (a few hundred KB) is cleared beside the start of the streaming pass, so
    // that nothing stands between the end of the pass and the first run kernel
    RTOPK_CUDA(ctx, cudaEventRecord(ctx->ev_fork, st));
    RTOPK_CUDA(ctx, cudaStreamWaitEvent(ctx->side, ctx->ev_fork, 0));
    RTOPK_CUDA(ctx, cudaMemsetAsync(ctx->d_zero + early_bytes, 0, zbytes - early_bytes, ctx->side));
    RTOPK_CUDA(ctx, cudaEventRecord(ctx->ev_zeroed, ctx->side));
  } else if (late_on_side) {
    RTOPK_CUDA(ctx, cudaMemsetAsync(ctx->d_zero + early_bytes, 0, zbytes - early_bytes, st));
  }
  cudaEvent_t join = forked ? ctx->ev_join : nullptr;
  // (f32 gradients: the streaming pass counts the candidates' histogram itself; bf16: k_run_hist does)
  const bool hist_in_stream = from_runs && grad_dtype == RTOPK_F32 && !ctx->test_giveup;
  const LateSide late = {sampler_late, hist_in_stream};
  rc = grad_dtype == RTOPK_F32 ? launch_select<float>(ctx, P, L, st, join, late)
                               : launch_select<__nv_bfloat16>(ctx, P, L, st, join, late);
  if (rc) return rc;
  // (a subset drawn beside the streaming pass has been waited for by launch_select; one drawn beside the run
  // kernels is waited for in front of the emission below)
  mark(ctx, RTOPK_PHASE_FINISH, st);
  if (from_runs) {
    // the usual case is finished straight from the streaming pass's runs, all slices side by side; what
    // these kernels leave (a missed bracket, heavy ties) is flagged for k_finish
    if (!hist_in_stream) {
      const uint32_t per_slice = std::max<uint32_t>(1u, ((uint32_t)ctx->sms * 8u + L.n_slices - 1u) / L.n_slices);
      const uint32_t tiles = (P.cap_max + kRunThreads * kHistPer - 1) / (kRunThreads * kHistPer);
      k_run_hist<<<dim3(std::min(tiles, per_slice), L.n_slices), kRunThreads, 0, st>>>(L);
      ++ctx->launches;
    }
    const uint32_t per_slice_run = std::max<uint32_t>(1u, ((uint32_t)ctx->sms * 4u + L.n_slices - 1u) / L.n_slices);
    const dim3 rgrid(std::min((P.cap_max + kRunTile - 1) / (uint32_t)kRunTile, per_slice_run), L.n_slices);
    k_run_count<<<rgrid, kRunThreads, 0, st>>>(L);
    if (sampler_late) RTOPK_CUDA(ctx, cudaStreamWaitEvent(st, ctx->ev_join, 0));   // the emission needs the subset
    const uint32_t per_slice_emit = std::max<uint32_t>(1u, ((uint32_t)ctx->sms * 5u + L.n_slices - 1u) / L.n_slices);
    const dim3 egrid(std::min((P.cap_max + kRunTile - 1) / (uint32_t)kRunTile, per_slice_emit), L.n_slices);
    k_run_emit<<<egrid, kRunThreads, 0, st>>>(L);
    ctx->launches += 2;
  }
  if (P.any_select) {
    // the largest cluster size that still lets every slice's cluster be resident at once
    int cs = 1;
    for (int c = kMaxCluster; c >= 1; --c)
      if ((int)L.n_slices <= ctx->finish_max_clusters[c]) { cs = c; break; }
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)cs * L.n_slices, 1, 1);
    cfg.blockDim = dim3(kFinishThreads, 1, 1);
    cfg.dynamicSmemBytes = kFinishSmemBytes;
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = (unsigned)cs; attr[0].val.clusterDim.y = 1; attr[0].val.clusterDim.z = 1;
    cfg.attrs = attr; cfg.numAttrs = 1;
    RTOPK_CUDA(ctx, cudaLaunchKernelEx(&cfg, k_finish, L));
    ++ctx->launches;
  }
  if (P.any_all) {
    const dim3 grid((P.words_all_max + kThreads - 1) / kThreads, L.n_slices);
    k_emit_all<<<grid, kThreads, 0, st>>>(L, P.words_all_max);
    ++ctx->launches;
  }
  if (sampler_late) RTOPK_CUDA(ctx, cudaStreamWaitEvent(st, ctx->ev_cleared, 0));   // the side stream's last work
  if (ctx->device_step && !forked && !sampler_late) { k_step_bump<<<1, 32, 0, st>>>(ctx->d_step); ++ctx->launches; }
  mark(ctx, RTOPK_PHASE_AGGREGATE, st);
  ctx->ev_valid[RTOPK_N_PHASES] = false;   // closed by the aggregate of a step call, if any
  RTOPK_CUDA(ctx, cudaGetLastError());
  if (K_out) *K_out = P.K_row;
  return RTOPK_OK;
}


// The threshold-then-subsample encoder (proof of Theorem 1) for W rows: the streaming pass gathers
// the coordinates above theta, then the sizes, the subset and the messages follow on the device.
int threshold_impl(rtopk_ctx* ctx, const void* grad, int grad_dtype, int64_t ld_g, float* residual, int64_t ld_m,
                   int64_t d, int32_t W, int32_t worker_base, float theta, int64_t k, uint64_t seed, uint32_t step,
                   uint32_t* msg_idx, float* msg_val, uint32_t* msg_count, uint32_t* msg_ones, cudaStream_t st) {
  int rc = check_common(ctx, grad, grad_dtype, ld_g, residual, ld_m, d, W, worker_base, msg_idx, msg_val);
  if (rc) return rc;
  if (!msg_count || !msg_ones || ((uintptr_t)msg_count & 3u) || ((uintptr_t)msg_ones & 3u)) return RTOPK_ERR_INVALID_ARG;
  if (!(theta >= 0.0f) || theta > 3.4028234e38f) return RTOPK_ERR_INVALID_ARG;        // finite, not NaN
  const float M = theta + theta;                                                       // the model's scale
  if (ctx->threshold_signs && M > 3.4028234e38f) return RTOPK_ERR_INVALID_ARG;
  if (k < 1 || k > d || k > ctx->k_max) return RTOPK_ERR_INVALID_ARG;
  if (ctx->select_path != 0) return RTOPK_ERR_UNSUPPORTED;
  const int64_t limit = std::min<int64_t>(ctx->r_max, d);      // the largest marked set the scratch holds
  if (k > limit) return RTOPK_ERR_INVALID_ARG;
  const int64_t off[2] = {0, d};
  Plan P;
  rc = make_plan(ctx, ld_g, ld_m, d, W, 1, off, &limit, &k, P, true);
  if (rc) return rc;
  if (P.cand_entries > ctx->cand_entries || P.first_entries > ctx->first_entries || P.sel_words > ctx->sel_words)
    return RTOPK_ERR_INVALID_ARG;
  DeviceGuard guard(ctx->device);
  if (!guard.ok) return RTOPK_ERR_CUDA;
  Launch L;
  size_t early_bytes = 0, zbytes = 0;
  rc = bind_launch(ctx, P, grad, residual, worker_base, seed, step, msg_idx, msg_val, L, &early_bytes, &zbytes);
  if (rc) return rc;
  rc = upload_slices(ctx, P, st);
  if (rc) return rc;
  // k_thr_sizes rewrites (r, k) of the device table: the next call uploads its slices afresh
  ctx->cached_slices.clear();
  ctx->history_stale = true;
  ctx->last_n_slices = L.n_slices;
  L.s.history = ctx->d_history;
  uint32_t theta_key;
  std::memcpy(&theta_key, &theta, 4);
  theta_key &= 0x7FFFFFFFu;
  mark(ctx, RTOPK_PHASE_SUBSET, st);
  mark(ctx, RTOPK_PHASE_THRESHOLD, st);
  k_thr_init<<<L.n_slices, kThrThreads, 0, st>>>(L, theta_key + 1u);
  ++ctx->launches;
  // the subset's tables are cleared beside the streaming pass
  RTOPK_CUDA(ctx, cudaEventRecord(ctx->ev_fork, st));
  RTOPK_CUDA(ctx, cudaStreamWaitEvent(ctx->side, ctx->ev_fork, 0));
  RTOPK_CUDA(ctx, cudaMemsetAsync(ctx->d_zero + early_bytes, 0, zbytes - early_bytes, ctx->side));
  if (P.any_sampler) RTOPK_CUDA(ctx, cudaMemsetAsync(ctx->d_first, 0xFF, P.first_entries * sizeof(uint32_t), ctx->side));
  RTOPK_CUDA(ctx, cudaEventRecord(ctx->ev_join, ctx->side));
  mark(ctx, RTOPK_PHASE_STREAM, st);
  const uint32_t per = (uint32_t)((P.slices[0].head + (uint64_t)P.slices[0].len + kChunk - 1) / kChunk);
  if (grad_dtype == RTOPK_F32)
    k_stream<float, false, false><<<ctx->stream_blocks[0], kStreamThreads, sizeof(StreamSmem<float>), st>>>(L, P.n_chunks, per);
  else
    k_stream<__nv_bfloat16, false, false><<<ctx->stream_blocks[1], kStreamThreads, sizeof(StreamSmem<__nv_bfloat16>), st>>>(L, P.n_chunks, per);
  ++ctx->launches;
  mark(ctx, RTOPK_PHASE_ORDER, st);
  k_thr_sizes<<<L.n_slices, kThrSizeThreads, 0, st>>>(L, (uint32_t)limit, (uint32_t)k, msg_count, msg_ones);
  ++ctx->launches;
  mark(ctx, RTOPK_PHASE_EXACT, st);
  RTOPK_CUDA(ctx, cudaStreamWaitEvent(st, ctx->ev_join, 0));
  rc = run_sampler(ctx, P, L, st, false);
  if (rc) return rc;
  mark(ctx, RTOPK_PHASE_FINISH, st);
  const dim3 egrid((P.chunks_max + kThrThreads / 32 - 1) / (kThrThreads / 32), L.n_slices);
  k_thr_emit<<<egrid, kThrThreads, 0, st>>>(L, ctx->threshold_signs ? 1u : 0u, M);
  ++ctx->launches;
  if (ctx->device_step) { k_step_bump<<<1, 32, 0, st>>>(ctx->d_step); ++ctx->launches; }
  mark(ctx, RTOPK_PHASE_AGGREGATE, st);
  ctx->ev_valid[RTOPK_N_PHASES] = false;
  RTOPK_CUDA(ctx, cudaGetLastError());
  return RTOPK_OK;
}

int aggregate_threshold_impl(rtopk_ctx* ctx, const uint32_t* msg_idx, const float* msg_val, const uint32_t* msg_count,
                             const uint32_t* msg_ones, int64_t d, int32_t W, int64_t k, float* out, cudaStream_t st);

bool scale_mode_known(int m) {
  return m == RTOPK_SCALE_MEAN || m == RTOPK_SCALE_SUM || m == RTOPK_SCALE_UNBIASED || m == RTOPK_SCALE_COUNT;
}

bool aggregate_is_sparse(int64_t d, int32_t W, int64_t k) {
  return W <= kAggMaxW && (uint64_t)W * (uint64_t)k * 16ull <= (uint64_t)d;   // <= 1024 entries per tile on average
}

// eta < 0: `out` receives the average.  eta >= 0: `out` holds weights and receives w - eta * average
// (only the coordinates some worker sent change, so nothing is cleared).
// Whether a step call keeps the run table of its messages: the table costs two reductions per message and
// saves the aggregation one search per worker and output tile, so it pays while a tile holds few messages of
// a worker (at most 64), and it is only read by the sparse kernel.
bool run_table_pays(int64_t d, int32_t W, int64_t k) {
  return W >= 1 && k >= 1 && aggregate_is_sparse(d, W, k) && (uint64_t)k * 256ull <= (uint64_t)d;
}

// `velocity` not null: heavy-ball momentum, `out` holds the weights (eta >= 0), every coordinate changes.
template <typename M>
int aggregate_launch(rtopk_ctx* ctx, const M& msgs, int64_t d, int32_t W, int64_t k, int scale_mode, float* out,
                     cudaStream_t st, float eta, int64_t r, float mu = 0.0f,
                     float* velocity = nullptr, const uint32_t* run_inv = nullptr, const uint32_t* run_cnt = nullptr) {
  if (!ctx || !out) return RTOPK_ERR_INVALID_ARG;
  if (d < 1 || d > ctx->d_max || W < 1 || W > ctx->W_max || k < 1 || k > d) return RTOPK_ERR_INVALID_ARG;
  if (!scale_mode_known(scale_mode)) return RTOPK_ERR_INVALID_ARG;
  if (scale_mode == RTOPK_SCALE_UNBIASED && (r < k || r > d)) return RTOPK_ERR_INVALID_ARG;   // needs the call's r
  if (scale_mode == RTOPK_SCALE_COUNT && W > 65535) return RTOPK_ERR_UNSUPPORTED;
  if ((uintptr_t)out & 15u) return RTOPK_ERR_INVALID_ARG;
  if ((uint64_t)k * (uint64_t)W >= (1ull << 32)) return RTOPK_ERR_INVALID_ARG;
  // Three regimes.  Up to 1024 entries per 16384 coordinates on average (the paper's densities): the sparse
  // kernel.  Beyond: the same kernel on tiles of 4096 while such a tile holds at most 1536 entries and a worker
  // sends at most d / 64 of them -- the dense kernel, which adds the workers' runs one after the other into a
  // tile of sums, pays one block barrier per worker and tile (about 1.3 ns x tiles x W in all) but then
  // takes 120 entries per ns against the sparse kernel's 45, so it wins once the rows are denser than that.
  const bool sparse16 = aggregate_is_sparse(d, W, k);
  const bool sparse4 = !sparse16 && W <= kAggMaxW && (uint64_t)W * (uint64_t)k * 8ull <= 3ull * (uint64_t)d &&
                       (uint64_t)k * 64ull <= (uint64_t)d;
  const bool sparse = sparse16 || sparse4;
  const uint32_t tile = sparse16 ? (uint32_t)kAggSparseTile : (uint32_t)kAggTile;
  const uint32_t ntiles = (uint32_t)((d + tile - 1) / tile);
  // the span-table format brings the sparse kernel's table of run starts along
  static_assert(kAggSparseTile == (int)kTiledSpan, "the spans of the format are the sparse kernel's tiles");
  const uint32_t* starts = ctx->d_agg_starts;
  bool have_starts = false;
  if constexpr (std::is_same<M, TiledMsgs>::value) {
    if (sparse16) { starts = msgs.tab; have_starts = true; }
  }
  if (!sparse16) run_cnt = nullptr;
  if (run_cnt) { starts = run_inv; have_starts = true; }     // kept by the sparsifier while it wrote the messages
  if (!have_starts && (size_t)W * (ntiles + 1) > ctx->agg_start_entries) return RTOPK_ERR_INVALID_ARG;
  DeviceGuard guard(ctx->device);
  if (!guard.ok) return RTOPK_ERR_CUDA;
  // with few workers and tiles the sparse kernel finds every tile's runs itself (one launch fewer);
  // otherwise a table of run starts is built first, all searches side by side
  const bool own_search = !have_starts && sparse16 && W <= kAggSearchW && (uint64_t)ntiles * (uint64_t)((W + 7) / 8) <= 4096u;
  if (!own_search && !have_starts) {
    const dim3 sgrid((ntiles + 1 + kAggThreads - 1) / kAggThreads, (uint32_t)W);
    k_agg_starts<M><<<sgrid, kAggThreads, 0, st>>>(msgs, (uint32_t)W, (uint32_t)k, ntiles, tile, ctx->d_agg_starts);
    ++ctx->launches;
  }
  AggScale sc = {1.0, 1.0, 0};
  if (scale_mode == RTOPK_SCALE_MEAN) sc.den = (double)W;
  else if (scale_mode == RTOPK_SCALE_UNBIASED) { sc.num = (double)r; sc.den = (double)W * (double)k; }
  else if (scale_mode == RTOPK_SCALE_COUNT) sc.by_count = 1;
  if (sparse) {
    // few coordinates are touched: every block clears its tile of the update and computes only what was sent
    const uint32_t clear = (eta < 0.0f && velocity == nullptr) ? 1u : 0u;
    // momentum: the sent coordinates are updated here and marked, the others by a plain pass behind it
    if (velocity) RTOPK_CUDA(ctx, cudaMemsetAsync(ctx->d_sent, 0, ((size_t)d + 31) / 32 * sizeof(uint32_t), st));
    if (sparse16)
      k_aggregate_sparse<M, kAggSparseTile><<<ntiles, kAggSparseThreads, 0, st>>>(msgs, own_search ? nullptr : starts, (uint32_t)d,
                                                                            (uint32_t)W, (uint32_t)k, sc, eta, out, mu,
                                                                            velocity, ctx->d_sent, clear, run_cnt);
    else
      k_aggregate_sparse<M, kAggTile><<<ntiles, kAggSparseThreads, 0, st>>>(msgs, starts, (uint32_t)d, (uint32_t)W, (uint32_t)k,
                                                                      sc, eta, out, mu, velocity, ctx->d_sent, clear,
                                                                      nullptr);
    ++ctx->launches;
    if (velocity) {
      const uint32_t groups = (uint32_t)((d + 3) / 4);
      const uint32_t blocks = std::min<uint32_t>((groups + 255u) / 256u, (uint32_t)ctx->sms * 16u);
      k_momentum_rest<<<blocks, 256, 0, st>>>((uint32_t)d, mu, eta, ctx->d_sent, velocity, out);
      ++ctx->launches;
    }
  } else {
    if (sc.by_count)
      k_aggregate<M, true><<<ntiles, kAggThreads, 0, st>>>(msgs, ctx->d_agg_starts, (uint32_t)d, (uint32_t)W,
                                                           (uint32_t)k, sc, eta, out, mu, velocity);
    else
      k_aggregate<M, false><<<ntiles, kAggThreads, 0, st>>>(msgs, ctx->d_agg_starts, (uint32_t)d, (uint32_t)W,
                                                            (uint32_t)k, sc, eta, out, mu, velocity);
    ++ctx->launches;
  }
  mark(ctx, RTOPK_N_PHASES, st);
  RTOPK_CUDA(ctx, cudaGetLastError());
  return RTOPK_OK;
}

int aggregate_impl(rtopk_ctx* ctx, const uint32_t* msg_idx, const float* msg_val, int64_t d, int32_t W, int64_t k,
                   int scale_mode, float* out, cudaStream_t st, float eta = -1.0f,
                   int64_t r = 0, uint32_t msg_stride = 1, float mu = 0.0f, float* velocity = nullptr,
                   bool from_step = false) {
  if (!msg_idx || !msg_val || ((uintptr_t)msg_idx & 3u) || ((uintptr_t)msg_val & 3u)) return RTOPK_ERR_INVALID_ARG;
  if (k < 1 || k > 0xFFFFFFFFll) return RTOPK_ERR_INVALID_ARG;
  const PlainMsgs msgs = {msg_idx, msg_val, (uint32_t)k, msg_stride};
  // `from_step`: the messages are the ones the context's last sparsify call wrote, with their run table
  const bool tab = from_step && ctx && ctx->run_cnt != nullptr;
  return aggregate_launch(ctx, msgs, d, W, k, scale_mode, out, st, eta, r, mu, velocity, tab ? ctx->run_inv : nullptr,
                          tab ? ctx->run_cnt : nullptr);
}

int aggregate_threshold_impl(rtopk_ctx* ctx, const uint32_t* msg_idx, const float* msg_val, const uint32_t* msg_count,
                             const uint32_t* msg_ones, int64_t d, int32_t W, int64_t k, float* out, cudaStream_t st) {
  if (!msg_idx || !msg_val || !msg_count || !msg_ones) return RTOPK_ERR_INVALID_ARG;
  if (((uintptr_t)msg_idx & 3u) || ((uintptr_t)msg_val & 3u) || ((uintptr_t)msg_count & 3u) || ((uintptr_t)msg_ones & 3u))
    return RTOPK_ERR_INVALID_ARG;
  if (k < 1 || k > 0xFFFFFFFFll) return RTOPK_ERR_INVALID_ARG;
  const ThresholdMsgs msgs = {msg_idx, msg_val, (uint32_t)k, msg_count, msg_ones};
  return aggregate_launch(ctx, msgs, d, W, k, RTOPK_SCALE_MEAN, out, st, -1.0f, 0);
}

// ceil(log2 d) index bits (at least 1) and the smallest row strides of the packed format: index
// words rounded up to 4 (16 bytes), value halves rounded up to 8 (16 bytes).
int packed_layout(int64_t d, int64_t k, int32_t* bits, int64_t* ld_words, int64_t* ld_halves) {
  if (d < 1 || d > 0xFFFFFFFFll || k < 1 || k > d) return RTOPK_ERR_INVALID_ARG;
  int b = 1;
  while (((int64_t)1 << b) < d) ++b;
  if (bits) *bits = b;
  if (ld_words) *ld_words = (((k * b + 31) / 32) + 3) / 4 * 4;
  if (ld_halves) *ld_halves = (k + 7) / 8 * 8;
  return RTOPK_OK;
}

}  // namespace

extern "C" {

int rtopk_version(void) { return kVersion; }

const char* rtopk_status_string(int status) {
  switch (status) {
    case RTOPK_OK: return "ok";
    case RTOPK_ERR_INVALID_ARG: return "invalid argument";
    case RTOPK_ERR_ALLOC: return "allocation failed";
    case RTOPK_ERR_CUDA: return "CUDA runtime error";
    case RTOPK_ERR_UNSUPPORTED: return "unsupported";
    case RTOPK_ERR_INTERNAL: return "internal error (device-side wait expired or invariant broken)";
    default: return "unknown status";
  }
}

int rtopk_last_cuda_error(const rtopk_ctx* ctx) { return ctx ? ctx->last_cuda_error : 0; }

int rtopk_create(rtopk_ctx** out, int device, int64_t d_max, int32_t W_max, int64_t r_max, int64_t k_max,
                 int32_t segments_max) {
  if (!out) return RTOPK_ERR_INVALID_ARG;
  *out = nullptr;
  if (d_max < 1 || d_max >= (1ll << 31) || W_max < 1 || W_max > 65535 || r_max < 1 || r_max > d_max ||
      k_max < 1 || k_max > r_max || segments_max < 1 || segments_max > 65535)
    return RTOPK_ERR_INVALID_ARG;
  int ndev = 0;
  if (cudaGetDeviceCount(&ndev) != cudaSuccess || device < 0 || device >= ndev) return RTOPK_ERR_CUDA;
  rtopk_ctx* ctx = new (std::nothrow) rtopk_ctx();
  if (!ctx) return RTOPK_ERR_ALLOC;
  ctx->device = device; ctx->d_max = d_max; ctx->W_max = W_max; ctx->r_max = r_max; ctx->k_max = k_max;
  ctx->S_max = segments_max;
  DeviceGuard guard(device);
  if (!guard.ok) { delete ctx; return RTOPK_ERR_CUDA; }
  const size_t W = (size_t)W_max, S = (size_t)segments_max, slices = W * S;
  const size_t chunks = W * ((size_t)d_max / kChunk + 2 * S + 1);
  // Candidate lists: a slice with r below its length gathers up to 3 r + 4096 candidates; a slice with
  // r equal to its length (Definition 2, random-k) gathers none.  A context made with r_max = d_max whose
  // full lists would take 2^30 entries or more is taken to be made for the latter: its lists are sized
  // for selections up to r = d_max / 32 only.
  size_t cand_row = std::min<size_t>((size_t)d_max, 3 * (size_t)r_max + 4096 * S) + 32 * S;
  if (r_max == d_max && W * cand_row >= ((size_t)1 << 30))
    cand_row = std::min<size_t>((size_t)d_max, 3 * ((size_t)d_max / 32) + 4096 * S) + 32 * S;
  const size_t groups = W * ((size_t)d_max / kChunk / 32 + 2 * S + 1);
  ctx->cand_entries = W * cand_row;
  ctx->first_entries = W * (std::min<size_t>((size_t)r_max, 16 * (size_t)k_max) + 128 * S);
  ctx->sel_words = W * ((size_t)r_max / 32 + S + 1);
  ctx->zero_bytes = zero_region_bytes(slices, chunks, groups, ctx->sel_words, W * (((size_t)d_max + kRunTableTile - 1) / kRunTableTile));
  ctx->agg_start_entries = W * ((size_t)(d_max + kAggTile - 1) / kAggTile + 2);
  if (ctx->cand_entries >= (1ull << 32) || ctx->first_entries >= (1ull << 32)) { delete ctx; return RTOPK_ERR_INVALID_ARG; }
  cudaError_t e = cudaSuccess;
  auto alloc = [&](void** p, size_t bytes) { if (e == cudaSuccess) e = cudaMalloc(p, bytes ? bytes : 16); };
  alloc((void**)&ctx->d_slices, slices * sizeof(Slice));
  ctx->slices_max = slices;
  if (e == cudaSuccess) e = cudaMallocHost((void**)&ctx->h_slices, slices * sizeof(Slice));
  alloc((void**)&ctx->d_state, slices * sizeof(SelState));
  alloc((void**)&ctx->d_zero, ctx->zero_bytes);
  alloc((void**)&ctx->d_first, ctx->first_entries * sizeof(uint32_t));
  alloc((void**)&ctx->d_cand_idx, ctx->cand_entries * sizeof(uint32_t));
  alloc((void**)&ctx->d_cand_val, ctx->cand_entries * sizeof(float));
  alloc((void**)&ctx->d_raw_idx, ctx->cand_entries * sizeof(uint32_t));
  alloc((void**)&ctx->d_raw_val, ctx->cand_entries * sizeof(float));
  ctx->chunk_tab_entries = chunks;
  alloc((void**)&ctx->d_chunk_tab, 3 * chunks * sizeof(uint32_t));
  alloc((void**)&ctx->d_draws, W * (size_t)k_max * sizeof(uint32_t));
  alloc((void**)&ctx->d_sel_pre, ctx->sel_words * sizeof(uint32_t));
  ctx->sel_blk_entries = slices * ((size_t)r_max / 32 / kSelChunk + 2);
  alloc((void**)&ctx->d_sel_blk, ctx->sel_blk_entries * sizeof(uint32_t));
  alloc((void**)&ctx->d_error, 16);
  alloc((void**)&ctx->d_fin, slices * sizeof(Fin));
  alloc((void**)&ctx->d_list, slices * 2 * kListMax * sizeof(uint32_t));
  alloc((void**)&ctx->d_step, 16);
  alloc((void**)&ctx->d_history, slices * sizeof(TauHistory));
  alloc((void**)&ctx->d_agg_starts, ctx->agg_start_entries * sizeof(uint32_t));
  alloc((void**)&ctx->d_sent, ((size_t)d_max + 31) / 32 * sizeof(uint32_t) + 16);
  if (e == cudaSuccess) e = cudaFuncSetAttribute(k_sample<float>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kSampleSmemBytes);
  if (e == cudaSuccess) e = cudaFuncSetAttribute(k_sample<__nv_bfloat16>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kSampleSmemBytes);
  for (int i = 0; i <= RTOPK_N_PHASES && e == cudaSuccess; ++i) e = cudaEventCreate(&ctx->ev[i]);
  if (e == cudaSuccess) e = cudaStreamCreateWithFlags(&ctx->side, cudaStreamNonBlocking);
  if (e == cudaSuccess) e = cudaEventCreateWithFlags(&ctx->ev_fork, cudaEventDisableTiming);
  if (e == cudaSuccess) e = cudaEventCreateWithFlags(&ctx->ev_join, cudaEventDisableTiming);
  if (e == cudaSuccess) e = cudaEventCreateWithFlags(&ctx->ev_streamed, cudaEventDisableTiming);
  if (e == cudaSuccess) e = cudaEventCreateWithFlags(&ctx->ev_cleared, cudaEventDisableTiming);
  if (e == cudaSuccess) e = cudaEventCreateWithFlags(&ctx->ev_zeroed, cudaEventDisableTiming);
  if (e == cudaSuccess) e = cudaFuncSetAttribute(k_finish, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kFinishSmemBytes);
  if (e == cudaSuccess) e = cudaFuncSetAttribute(k_finish, cudaFuncAttributeNonPortableClusterSizeAllowed, 1);
  for (int c = 1; c <= kMaxCluster && e == cudaSuccess; ++c) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)c, 1, 1);
    cfg.blockDim = dim3(kFinishThreads, 1, 1);
    cfg.dynamicSmemBytes = kFinishSmemBytes;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = (unsigned)c; attr[0].val.clusterDim.y = 1; attr[0].val.clusterDim.z = 1;
    cfg.attrs = attr; cfg.numAttrs = 1;
    int n = 0;
    if (cudaOccupancyMaxActiveClusters(&n, k_finish, &cfg) == cudaSuccess) ctx->finish_max_clusters[c] = n;
    else cudaGetLastError();
  }
  if (e == cudaSuccess && ctx->finish_max_clusters[1] < 1) e = cudaErrorLaunchOutOfResources;
  if (e == cudaSuccess) {
    int sms = 0, per_f32 = 0, per_bf16 = 0;
    e = cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, device);
    if (e == cudaSuccess) e = cudaFuncSetAttribute(k_stream<float, true, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)sizeof(StreamSmem<float>));
    if (e == cudaSuccess) e = cudaFuncSetAttribute(k_stream<float, false, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)sizeof(StreamSmem<float>));
    if (e == cudaSuccess) e = cudaFuncSetAttribute(k_stream<float, false, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)sizeof(StreamSmem<float>));
    if (e == cudaSuccess) e = cudaFuncSetAttribute(k_stream<__nv_bfloat16, true, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)sizeof(StreamSmem<__nv_bfloat16>));
    if (e == cudaSuccess) e = cudaFuncSetAttribute(k_stream<__nv_bfloat16, false, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)sizeof(StreamSmem<__nv_bfloat16>));
    if (e == cudaSuccess) e = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_f32, k_stream<float, false, true>, kStreamThreads, sizeof(StreamSmem<float>));
    if (e == cudaSuccess) e = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_bf16, k_stream<__nv_bfloat16, false, false>, kStreamThreads, sizeof(StreamSmem<__nv_bfloat16>));
    if (e == cudaSuccess && (per_f32 < 1 || per_bf16 < 1)) e = cudaErrorLaunchOutOfResources;
    ctx->sms = sms;
    ctx->stream_blocks[0] = sms * per_f32;
    ctx->stream_blocks[1] = sms * per_bf16;
  }
  if (e == cudaSuccess) e = cudaMemset(ctx->d_error, 0, 16);
  if (e == cudaSuccess) e = cudaMemset(ctx->d_step, 0, 16);
  if (e == cudaSuccess) e = cudaMemset(ctx->d_state, 0, slices * sizeof(SelState));
  if (e != cudaSuccess) {
    const int rc = e == cudaErrorMemoryAllocation ? RTOPK_ERR_ALLOC : RTOPK_ERR_CUDA;
    cudaGetLastError();
    rtopk_destroy(ctx);
    return rc;
  }
  *out = ctx;
  return RTOPK_OK;
}

int rtopk_destroy(rtopk_ctx* ctx) {
  if (!ctx) return RTOPK_ERR_INVALID_ARG;
  DeviceGuard guard(ctx->device);
  void* ptrs[] = {ctx->d_slices, ctx->d_state, ctx->d_zero, ctx->d_first, ctx->d_cand_idx, ctx->d_cand_val,
                  ctx->d_raw_idx, ctx->d_raw_val, ctx->d_chunk_tab,
                  ctx->d_draws, ctx->d_sel_pre, ctx->d_sel_blk, ctx->d_error, ctx->d_agg_starts, ctx->d_stage, ctx->d_history,
                  ctx->d_step, ctx->d_fin, ctx->d_list, ctx->d_sent};
  for (void* p : ptrs) if (p) cudaFree(p);
  if (ctx->h_slices) cudaFreeHost(ctx->h_slices);
  for (cudaEvent_t ev : ctx->ev) if (ev) cudaEventDestroy(ev);
  if (ctx->ev_fork) cudaEventDestroy(ctx->ev_fork);
  if (ctx->ev_join) cudaEventDestroy(ctx->ev_join);
  if (ctx->ev_streamed) cudaEventDestroy(ctx->ev_streamed);
  if (ctx->ev_cleared) cudaEventDestroy(ctx->ev_cleared);
  if (ctx->ev_zeroed) cudaEventDestroy(ctx->ev_zeroed);
  if (ctx->side) cudaStreamDestroy(ctx->side);
  if (ctx->copy_in) { cudaStreamSynchronize(ctx->copy_in); cudaStreamDestroy(ctx->copy_in); }
  if (ctx->copy_out) { cudaStreamSynchronize(ctx->copy_out); cudaStreamDestroy(ctx->copy_out); }
  for (int b = 0; b < 2; ++b) {
    if (ctx->ev_uploaded[b]) cudaEventDestroy(ctx->ev_uploaded[b]);
    if (ctx->ev_consumed[b]) cudaEventDestroy(ctx->ev_consumed[b]);
  }
  if (ctx->ev_downloaded) cudaEventDestroy(ctx->ev_downloaded);
  delete ctx;
  return RTOPK_OK;
}

int rtopk_set_option(rtopk_ctx* ctx, int option, int64_t value) {
  if (!ctx) return RTOPK_ERR_INVALID_ARG;
  if (option == RTOPK_OPT_SELECT_PATH && (value == 0 || value == 1)) { ctx->select_path = (int)value; return RTOPK_OK; }
  if (option == RTOPK_OPT_REUSE_THRESHOLD && (value == 0 || value == 1)) {
    ctx->reuse = (int)value;
    ctx->history_stale = true;
    return RTOPK_OK;
  }
  if (option == RTOPK_OPT_DEVICE_STEP && (value == 0 || value == 1)) { ctx->device_step = (int)value; return RTOPK_OK; }
  if (option == RTOPK_OPT_FINISH_PATH && value >= 0 && value <= 2) { ctx->finish_path = (int)value; return RTOPK_OK; }
  if (option == RTOPK_OPT_TEST_STREAM_GIVEUP && (value == 0 || value == 1)) { ctx->test_giveup = (int)value; return RTOPK_OK; }
  if (option == RTOPK_OPT_THRESHOLD_SIGNS && (value == 0 || value == 1)) { ctx->threshold_signs = (int)value; return RTOPK_OK; }
  if (option == RTOPK_OPT_PROFILE && (value == 0 || value == 1)) {
    ctx->profile = (int)value;
    for (bool& v : ctx->ev_valid) v = false;
    return RTOPK_OK;
  }
  return RTOPK_ERR_INVALID_ARG;
}

int rtopk_sparsify(rtopk_ctx* ctx, const void* grad, int grad_dtype, int64_t ld_g, float* residual, int64_t ld_m,
                   int64_t d, int32_t W, int32_t worker_base, int64_t r, int64_t k, uint64_t seed, uint32_t step,
                   uint32_t* msg_idx, float* msg_val, void* stream) {
  const int64_t off[2] = {0, d};
  return sparsify_impl(ctx, grad, grad_dtype, ld_g, residual, ld_m, d, W, worker_base, 1, off, &r, &k, seed, step,
                       msg_idx, msg_val, (cudaStream_t)stream, nullptr);
}

int rtopk_sparsify_segmented(rtopk_ctx* ctx, const void* grad, int grad_dtype, int64_t ld_g, float* residual,
                             int64_t ld_m, int64_t d, int32_t W, int32_t worker_base, int32_t S,
                             const int64_t* seg_off, const int64_t* seg_r, const int64_t* seg_k, uint64_t seed,
                             uint32_t step, uint32_t* msg_idx, float* msg_val, void* stream) {
  return sparsify_impl(ctx, grad, grad_dtype, ld_g, residual, ld_m, d, W, worker_base, S, seg_off, seg_r, seg_k,
                       seed, step, msg_idx, msg_val, (cudaStream_t)stream, nullptr);
}

int rtopk_aggregate(rtopk_ctx* ctx, const uint32_t* msg_idx, const float* msg_val, int64_t d, int32_t W, int64_t k,
                    int scale_mode, float* out, void* stream) {
  return aggregate_impl(ctx, msg_idx, msg_val, d, W, k, scale_mode, out, (cudaStream_t)stream);
}

int rtopk_sparsify_pairs(rtopk_ctx* ctx, const void* grad, int grad_dtype, int64_t ld_g, float* residual, int64_t ld_m,
                         int64_t d, int32_t W, int32_t worker_base, int64_t r, int64_t k, uint64_t seed, uint32_t step,
                         uint64_t* msg_pairs, void* stream) {
  if (!msg_pairs || ((uintptr_t)msg_pairs & 7u)) return RTOPK_ERR_INVALID_ARG;
  const int64_t off[2] = {0, d};
  uint32_t* words = reinterpret_cast<uint32_t*>(msg_pairs);
  return sparsify_impl(ctx, grad, grad_dtype, ld_g, residual, ld_m, d, W, worker_base, 1, off, &r, &k, seed, step,
                       words, reinterpret_cast<float*>(words + 1), (cudaStream_t)stream, nullptr, 2);
}

int rtopk_aggregate_pairs(rtopk_ctx* ctx, const uint64_t* msg_pairs, int64_t d, int32_t W, int64_t k, int scale_mode,
                          float* out, void* stream) {
  if (!msg_pairs || ((uintptr_t)msg_pairs & 7u)) return RTOPK_ERR_INVALID_ARG;
  const uint32_t* words = reinterpret_cast<const uint32_t*>(msg_pairs);
  return aggregate_impl(ctx, words, reinterpret_cast<const float*>(words + 1), d, W, k, scale_mode, out,
                        (cudaStream_t)stream, -1.0f, 0, 2);
}

int rtopk_aggregate_unbiased(rtopk_ctx* ctx, const uint32_t* msg_idx, const float* msg_val, int64_t d, int32_t W,
                             int64_t k, int64_t r, float* out, void* stream) {
  return aggregate_impl(ctx, msg_idx, msg_val, d, W, k, RTOPK_SCALE_UNBIASED, out, (cudaStream_t)stream, -1.0f, r);
}

int rtopk_warmup_sizes(int64_t d, int32_t n_workers, double initial_density, double final_density,
                       int64_t warmup_steps, int64_t step, int64_t* r, int64_t* k) {
  if (d < 1 || n_workers < 1 || step < 0 || warmup_steps < 0 || !r || !k) return RTOPK_ERR_INVALID_ARG;
  if (!(final_density > 0.0) || !(initial_density >= final_density) || !(initial_density <= 1.0))
    return RTOPK_ERR_INVALID_ARG;
  double density = final_density;
  if (step < warmup_steps)
    density = initial_density * std::pow(final_density / initial_density, (double)step / (double)warmup_steps);
  int64_t kk = (int64_t)std::floor(density * (double)d);
  if (kk < 1) kk = 1;
  if (kk > d) kk = d;
  *k = kk;
  *r = kk > d / n_workers ? d : kk * (int64_t)n_workers;        // k / r = 1 / n, capped at d
  return RTOPK_OK;
}

int rtopk_packed_layout(int64_t d, int64_t k, int32_t* index_bits, int64_t* ld_words, int64_t* ld_halves) {
  return packed_layout(d, k, index_bits, ld_words, ld_halves);
}

int rtopk_encode(rtopk_ctx* ctx, const uint32_t* msg_idx, const float* msg_val, int64_t d, int32_t W, int64_t k,
                 float* residual, int64_t ld_m, uint32_t* packed_idx, int64_t ld_words, uint16_t* packed_val,
                 int64_t ld_halves, void* stream) {
  if (!ctx || !msg_idx || !msg_val || !packed_idx || !packed_val) return RTOPK_ERR_INVALID_ARG;
  if (W < 1 || W > ctx->W_max || d > ctx->d_max) return RTOPK_ERR_INVALID_ARG;
  int32_t bits = 0;
  int64_t min_words = 0, min_halves = 0;
  if (packed_layout(d, k, &bits, &min_words, &min_halves)) return RTOPK_ERR_INVALID_ARG;
  if (ld_words < min_words || ld_halves < min_halves || ld_words > 0xFFFFFFFFll || ld_halves > 0xFFFFFFFFll ||
      (ld_words % 4) || (ld_halves % 8))
    return RTOPK_ERR_INVALID_ARG;
  if (((uintptr_t)msg_idx & 3u) || ((uintptr_t)msg_val & 3u) || ((uintptr_t)packed_idx & 15u) || ((uintptr_t)packed_val & 15u))
    return RTOPK_ERR_INVALID_ARG;
  if (residual && (ld_m < d || ((uintptr_t)residual & 3u))) return RTOPK_ERR_INVALID_ARG;
  DeviceGuard guard(ctx->device);
  if (!guard.ok) return RTOPK_ERR_CUDA;
  const uint32_t span = (uint32_t)std::max(ld_words, ld_halves);
  const dim3 grid((span + kCodecThreads - 1) / kCodecThreads, (uint32_t)W);
  k_encode<<<grid, kCodecThreads, 0, (cudaStream_t)stream>>>(msg_idx, msg_val, (uint32_t)k, (uint32_t)bits, residual, ld_m,
                                                             packed_idx, (uint32_t)ld_words, packed_val,
                                                             (uint32_t)ld_halves);
  ++ctx->launches;
  RTOPK_CUDA(ctx, cudaGetLastError());
  return RTOPK_OK;
}

int rtopk_aggregate_packed(rtopk_ctx* ctx, const uint32_t* packed_idx, int64_t ld_words, const uint16_t* packed_val,
                           int64_t ld_halves, int64_t d, int32_t W, int64_t k, int scale_mode, float* out,
                           void* stream) {
  if (!packed_idx || !packed_val || ((uintptr_t)packed_idx & 3u) || ((uintptr_t)packed_val & 1u))
    return RTOPK_ERR_INVALID_ARG;
  int32_t bits = 0;
  int64_t min_words = 0, min_halves = 0;
  if (packed_layout(d, k, &bits, &min_words, &min_halves)) return RTOPK_ERR_INVALID_ARG;
  if (ld_words < (k * bits + 31) / 32 || ld_halves < k || ld_words > 0xFFFFFFFFll || ld_halves > 0xFFFFFFFFll)
    return RTOPK_ERR_INVALID_ARG;
  if (scale_mode == RTOPK_SCALE_UNBIASED) return RTOPK_ERR_INVALID_ARG;   // needs r: scale the result by r / k instead
  const PackedMsgs msgs = {packed_idx, packed_val, (uint32_t)ld_words, (uint32_t)ld_halves, (uint32_t)bits};
  return aggregate_launch(ctx, msgs, d, W, k, scale_mode, out, (cudaStream_t)stream, -1.0f, 0);
}

int rtopk_tiled_layout(int64_t d, int64_t k, int64_t* spans, int64_t* ld_low, int64_t* ld_halves) {
  if (d < 1 || d > 0xFFFFFFFFll || k < 1 || k > d) return RTOPK_ERR_INVALID_ARG;
  if (spans) *spans = (d + kTiledSpan - 1) / kTiledSpan;
  if (ld_low) *ld_low = (k + 7) / 8 * 8;
  if (ld_halves) *ld_halves = (k + 7) / 8 * 8;
  return RTOPK_OK;
}

int rtopk_encode_tiled(rtopk_ctx* ctx, const uint32_t* msg_idx, const float* msg_val, int64_t d, int32_t W, int64_t k,
                       float* residual, int64_t ld_m, uint32_t* span_tab, uint16_t* low_idx, int64_t ld_low,
                       uint16_t* packed_val, int64_t ld_halves, void* stream) {
  if (!ctx || !msg_idx || !msg_val || !span_tab || !low_idx || !packed_val) return RTOPK_ERR_INVALID_ARG;
  if (W < 1 || W > ctx->W_max || d > ctx->d_max) return RTOPK_ERR_INVALID_ARG;
  int64_t spans = 0, min_low = 0, min_halves = 0;
  if (rtopk_tiled_layout(d, k, &spans, &min_low, &min_halves)) return RTOPK_ERR_INVALID_ARG;
  if (ld_low < min_low || ld_halves < min_halves || ld_low > 0xFFFFFFFFll || ld_halves > 0xFFFFFFFFll || (ld_low % 8) ||
      (ld_halves % 8))
    return RTOPK_ERR_INVALID_ARG;
  if (((uintptr_t)msg_idx & 3u) || ((uintptr_t)msg_val & 3u) || ((uintptr_t)span_tab & 3u) || ((uintptr_t)low_idx & 15u) ||
      ((uintptr_t)packed_val & 15u))
    return RTOPK_ERR_INVALID_ARG;
  if (residual && (ld_m < d || ((uintptr_t)residual & 3u))) return RTOPK_ERR_INVALID_ARG;
  DeviceGuard guard(ctx->device);
  if (!guard.ok) return RTOPK_ERR_CUDA;
  const uint32_t span = (uint32_t)std::max(ld_low, ld_halves);
  const dim3 grid((span + kCodecThreads - 1) / kCodecThreads, (uint32_t)W);
  k_encode_tiled<<<grid, kCodecThreads, 0, (cudaStream_t)stream>>>(msg_idx, msg_val, (uint32_t)k, (uint32_t)d, kTiledSpan,
                                                                   (uint32_t)spans, residual, ld_m, span_tab, low_idx,
                                                                   (uint32_t)ld_low, packed_val, (uint32_t)ld_halves);
  ++ctx->launches;
  RTOPK_CUDA(ctx, cudaGetLastError());
  return RTOPK_OK;
}

int rtopk_aggregate_tiled(rtopk_ctx* ctx, const uint32_t* span_tab, const uint16_t* low_idx, int64_t ld_low,
                          const uint16_t* packed_val, int64_t ld_halves, int64_t d, int32_t W, int64_t k,
                          int scale_mode, float* out, void* stream) {
  if (!span_tab || !low_idx || !packed_val || ((uintptr_t)span_tab & 3u) || ((uintptr_t)low_idx & 1u) ||
      ((uintptr_t)packed_val & 1u))
    return RTOPK_ERR_INVALID_ARG;
  int64_t spans = 0;
  if (rtopk_tiled_layout(d, k, &spans, nullptr, nullptr)) return RTOPK_ERR_INVALID_ARG;
  if (ld_low < k || ld_halves < k || ld_low > 0xFFFFFFFFll || ld_halves > 0xFFFFFFFFll) return RTOPK_ERR_INVALID_ARG;
  if (scale_mode == RTOPK_SCALE_UNBIASED) return RTOPK_ERR_INVALID_ARG;   // needs r: scale the result by r / k instead
  const TiledMsgs msgs = {span_tab, low_idx, packed_val, (uint32_t)spans, (uint32_t)ld_low, (uint32_t)ld_halves};
  return aggregate_launch(ctx, msgs, d, W, k, scale_mode, out, (cudaStream_t)stream, -1.0f, 0);
}

namespace {
bool momentum_args_ok(float eta, float mu, const float* velocity, const float* weights) {
  return (eta >= 0.0f) && eta <= 3.0e38f && (mu >= 0.0f) && (mu < 1.0f) && velocity && weights &&
         !((uintptr_t)velocity & 15u) && !((uintptr_t)weights & 15u) && velocity != weights;
}
}  // namespace

int rtopk_apply_momentum(rtopk_ctx* ctx, const uint32_t* msg_idx, const float* msg_val, int64_t d, int32_t W,
                         int64_t k, int scale_mode, int64_t r, float eta, float mu, float* velocity, float* weights,
                         void* stream) {
  if (!momentum_args_ok(eta, mu, velocity, weights)) return RTOPK_ERR_INVALID_ARG;
  return aggregate_impl(ctx, msg_idx, msg_val, d, W, k, scale_mode, weights, (cudaStream_t)stream, eta, r, 1, mu,
                        velocity);
}

int rtopk_step_momentum(rtopk_ctx* ctx, const void* grad, int grad_dtype, int64_t ld_g, float* residual, int64_t ld_m,
                        int64_t d, int32_t W, int32_t worker_base, int64_t r, int64_t k, uint64_t seed, uint32_t step,
                        int scale_mode, float eta, float mu, uint32_t* msg_idx, float* msg_val, float* velocity,
                        float* weights, void* stream) {
  if (!momentum_args_ok(eta, mu, velocity, weights) || !scale_mode_known(scale_mode)) return RTOPK_ERR_INVALID_ARG;
  if (!ctx || d < 1 || d > ctx->d_max) return RTOPK_ERR_INVALID_ARG;
  const int64_t off[2] = {0, d};
  const int rc = sparsify_impl(ctx, grad, grad_dtype, ld_g, residual, ld_m, d, W, worker_base, 1, off, &r, &k, seed,
                               step, msg_idx, msg_val, (cudaStream_t)stream, nullptr, 1,
                               run_table_pays(d, W, k));
  if (rc) return rc;
  return aggregate_impl(ctx, msg_idx, msg_val, d, W, k, scale_mode, weights, (cudaStream_t)stream, eta, r, 1, mu,
                        velocity, true);
}

int rtopk_apply_update(rtopk_ctx* ctx, const uint32_t* msg_idx, const float* msg_val, int64_t d, int32_t W,
                       int64_t k, int scale_mode, float eta, float* weights, void* stream) {
  if (!(eta >= 0.0f) || eta > 3.0e38f) return RTOPK_ERR_INVALID_ARG;
  return aggregate_impl(ctx, msg_idx, msg_val, d, W, k, scale_mode, weights, (cudaStream_t)stream, eta);
}

int rtopk_step_apply(rtopk_ctx* ctx, const void* grad, int grad_dtype, int64_t ld_g, float* residual, int64_t ld_m,
                     int64_t d, int32_t W, int32_t worker_base, int64_t r, int64_t k, uint64_t seed,
                     uint32_t step, int scale_mode, float eta, uint32_t* msg_idx, float* msg_val, float* weights,
                     void* stream) {
  if (!weights || ((uintptr_t)weights & 15u) || !scale_mode_known(scale_mode)) return RTOPK_ERR_INVALID_ARG;
  if (!(eta >= 0.0f) || eta > 3.0e38f) return RTOPK_ERR_INVALID_ARG;
  if (!ctx || d < 1 || d > ctx->d_max) return RTOPK_ERR_INVALID_ARG;
  const int64_t off[2] = {0, d};
  const int rc = sparsify_impl(ctx, grad, grad_dtype, ld_g, residual, ld_m, d, W, worker_base, 1, off, &r, &k, seed,
                               step, msg_idx, msg_val, (cudaStream_t)stream, nullptr, 1,
                               run_table_pays(d, W, k));
  if (rc) return rc;
  return aggregate_impl(ctx, msg_idx, msg_val, d, W, k, scale_mode, weights, (cudaStream_t)stream, eta, r, 1, 0.0f,
                        nullptr, true);
}

int rtopk_step(rtopk_ctx* ctx, const void* grad, int grad_dtype, int64_t ld_g, float* residual, int64_t ld_m,
               int64_t d, int32_t W, int32_t worker_base, int64_t r, int64_t k, uint64_t seed, uint32_t step,
               int scale_mode, uint32_t* msg_idx, float* msg_val, float* out, void* stream) {
  if (!out || ((uintptr_t)out & 15u) || !scale_mode_known(scale_mode)) return RTOPK_ERR_INVALID_ARG;
  if (!ctx || d < 1 || d > ctx->d_max) return RTOPK_ERR_INVALID_ARG;
  const int64_t off[2] = {0, d};
  const int rc = sparsify_impl(ctx, grad, grad_dtype, ld_g, residual, ld_m, d, W, worker_base, 1, off, &r, &k, seed,
                               step, msg_idx, msg_val, (cudaStream_t)stream, nullptr, 1,
                               run_table_pays(d, W, k));
  if (rc) return rc;
  return aggregate_impl(ctx, msg_idx, msg_val, d, W, k, scale_mode, out, (cudaStream_t)stream, -1.0f, r, 1, 0.0f,
                        nullptr, true);
}

int rtopk_step_segmented(rtopk_ctx* ctx, const void* grad, int grad_dtype, int64_t ld_g, float* residual,
                         int64_t ld_m, int64_t d, int32_t W, int32_t worker_base, int32_t S, const int64_t* seg_off,
                         const int64_t* seg_r, const int64_t* seg_k, uint64_t seed, uint32_t step, int scale_mode,
                         uint32_t* msg_idx, float* msg_val, float* out, void* stream) {
  if (!out || ((uintptr_t)out & 15u) || !scale_mode_known(scale_mode)) return RTOPK_ERR_INVALID_ARG;
  if (scale_mode == RTOPK_SCALE_UNBIASED) return RTOPK_ERR_UNSUPPORTED;   // r / k differs from tensor to tensor
  if (!ctx || d < 1 || d > ctx->d_max || S < 1 || S > ctx->S_max || !seg_k) return RTOPK_ERR_INVALID_ARG;
  int64_t Ksum = 0;
  for (int s = 0; s < S; ++s) Ksum += seg_k[s] > 0 ? seg_k[s] : 0;
  uint32_t K = 0;
  const int rc = sparsify_impl(ctx, grad, grad_dtype, ld_g, residual, ld_m, d, W, worker_base, S, seg_off, seg_r,
                               seg_k, seed, step, msg_idx, msg_val, (cudaStream_t)stream, &K, 1,
                               run_table_pays(d, W, Ksum));
  if (rc) return rc;
  return aggregate_impl(ctx, msg_idx, msg_val, d, W, K, scale_mode, out, (cudaStream_t)stream, -1.0f, 0, 1, 0.0f,
                        nullptr, true);
}

int rtopk_sparsify_threshold(rtopk_ctx* ctx, const void* grad, int grad_dtype, int64_t ld_g, float* residual,
                             int64_t ld_m, int64_t d, int32_t W, int32_t worker_base, float theta, int64_t k,
                             uint64_t seed, uint32_t step, uint32_t* msg_idx, float* msg_val, uint32_t* msg_count,
                             uint32_t* msg_ones, void* stream) {
  return threshold_impl(ctx, grad, grad_dtype, ld_g, residual, ld_m, d, W, worker_base, theta, k, seed, step, msg_idx,
                        msg_val, msg_count, msg_ones, (cudaStream_t)stream);
}

int rtopk_aggregate_threshold(rtopk_ctx* ctx, const uint32_t* msg_idx, const float* msg_val, const uint32_t* msg_count,
                              const uint32_t* msg_ones, int64_t d, int32_t W, int64_t k, float* out, void* stream) {
  return aggregate_threshold_impl(ctx, msg_idx, msg_val, msg_count, msg_ones, d, W, k, out, (cudaStream_t)stream);
}

int rtopk_step_threshold(rtopk_ctx* ctx, const void* grad, int grad_dtype, int64_t ld_g, float* residual, int64_t ld_m,
                         int64_t d, int32_t W, int32_t worker_base, float theta, int64_t k, uint64_t seed,
                         uint32_t step, uint32_t* msg_idx, float* msg_val, uint32_t* msg_count, uint32_t* msg_ones,
                         float* out, void* stream) {
  if (!out || ((uintptr_t)out & 15u)) return RTOPK_ERR_INVALID_ARG;
  if (!ctx || d < 1 || d > ctx->d_max) return RTOPK_ERR_INVALID_ARG;
  const int rc = threshold_impl(ctx, grad, grad_dtype, ld_g, residual, ld_m, d, W, worker_base, theta, k, seed, step,
                                msg_idx, msg_val, msg_count, msg_ones, (cudaStream_t)stream);
  if (rc) return rc;
  return aggregate_threshold_impl(ctx, msg_idx, msg_val, msg_count, msg_ones, d, W, k, out, (cudaStream_t)stream);
}

int rtopk_step_host(rtopk_ctx* ctx, const void* h_grad, int grad_dtype, int64_t ld_g, float* residual, int64_t ld_m,
                    int64_t d, int32_t W, int32_t worker_base, int64_t r, int64_t k, uint64_t seed, uint32_t step,
                    int scale_mode, uint32_t* h_msg_idx, float* h_msg_val, float* h_out, void* stream) {
  if (!ctx || !h_grad || !h_msg_idx || !h_msg_val || !h_out) return RTOPK_ERR_INVALID_ARG;
  if (grad_dtype != RTOPK_F32 && grad_dtype != RTOPK_BF16) return RTOPK_ERR_INVALID_ARG;
  if (d < 1 || d > ctx->d_max || W < 1 || W > ctx->W_max || k < 1 || k > r || r > d || ld_g < d)
    return RTOPK_ERR_INVALID_ARG;
  cudaStream_t st = (cudaStream_t)stream;
  DeviceGuard guard(ctx->device);
  if (!guard.ok) return RTOPK_ERR_CUDA;
  const size_t gsz = grad_dtype == RTOPK_F32 ? 4 : 2;
  const size_t g_bytes = align_up((size_t)W * (size_t)ld_g * gsz, 256);
  const size_t mi_bytes = align_up((size_t)W * (size_t)k * 4, 256);
  const size_t out_bytes = align_up((size_t)d * 4, 256);
  const size_t total = 2 * g_bytes + 2 * mi_bytes + out_bytes;
  if (!ctx->copy_in) {
    // first use: the copy streams and their events
    RTOPK_CUDA(ctx, cudaStreamCreateWithFlags(&ctx->copy_in, cudaStreamNonBlocking));
    RTOPK_CUDA(ctx, cudaStreamCreateWithFlags(&ctx->copy_out, cudaStreamNonBlocking));
    for (int b = 0; b < 2; ++b) {
      RTOPK_CUDA(ctx, cudaEventCreateWithFlags(&ctx->ev_uploaded[b], cudaEventDisableTiming));
      RTOPK_CUDA(ctx, cudaEventCreateWithFlags(&ctx->ev_consumed[b], cudaEventDisableTiming));
    }
    RTOPK_CUDA(ctx, cudaEventCreateWithFlags(&ctx->ev_downloaded, cudaEventDisableTiming));
  }
  if (total > ctx->stage_bytes) {
    // first use (or a larger shape): the one place a call allocates, and therefore waits
    RTOPK_CUDA(ctx, cudaStreamSynchronize(st));
    RTOPK_CUDA(ctx, cudaStreamSynchronize(ctx->copy_in));
    RTOPK_CUDA(ctx, cudaStreamSynchronize(ctx->copy_out));
    if (ctx->d_stage) { cudaFree(ctx->d_stage); ctx->d_stage = nullptr; ctx->stage_bytes = 0; }
    const cudaError_t e = cudaMalloc(&ctx->d_stage, total);
    if (e != cudaSuccess) { cudaGetLastError(); ctx->last_cuda_error = (int)e; return RTOPK_ERR_ALLOC; }
    ctx->stage_bytes = total;
    ctx->stage_g_bytes = g_bytes; ctx->stage_mi_bytes = mi_bytes;
    ctx->consumed_valid[0] = ctx->consumed_valid[1] = false;
  } else if (g_bytes != ctx->stage_g_bytes || mi_bytes != ctx->stage_mi_bytes) {
    // another shape carves the same allocation differently: the earlier calls' steps and copies may
    // still be using the old offsets, so everything in flight ends before the new ones are used
    RTOPK_CUDA(ctx, cudaStreamSynchronize(st));
    RTOPK_CUDA(ctx, cudaStreamSynchronize(ctx->copy_in));
    RTOPK_CUDA(ctx, cudaStreamSynchronize(ctx->copy_out));
    ctx->stage_g_bytes = g_bytes; ctx->stage_mi_bytes = mi_bytes;
    ctx->consumed_valid[0] = ctx->consumed_valid[1] = false;
  }
  const int b = ctx->stage_next;
  ctx->stage_next ^= 1;
  char* base = (char*)ctx->d_stage;
  void* d_grad = base + (size_t)b * g_bytes;
  uint32_t* d_idx = (uint32_t*)(base + 2 * g_bytes);
  float* d_val = (float*)(base + 2 * g_bytes + mi_bytes);
  float* d_out = (float*)(base + 2 * g_bytes + 2 * mi_bytes);
  // upload: as soon as the step that last read this gradient buffer (two calls ago) has ended -- it does
  // not wait for the caller's stream, so it runs beside the previous call's step and download
  if (ctx->consumed_valid[b]) RTOPK_CUDA(ctx, cudaStreamWaitEvent(ctx->copy_in, ctx->ev_consumed[b], 0));
  RTOPK_CUDA(ctx, cudaMemcpyAsync(d_grad, h_grad, (size_t)W * (size_t)ld_g * gsz, cudaMemcpyHostToDevice, ctx->copy_in));
  RTOPK_CUDA(ctx, cudaEventRecord(ctx->ev_uploaded[b], ctx->copy_in));
  // step: on the caller's stream, once the gradient is there
  RTOPK_CUDA(ctx, cudaStreamWaitEvent(st, ctx->ev_uploaded[b], 0));
  const int rc = rtopk_step(ctx, d_grad, grad_dtype, ld_g, residual, ld_m, d, W, worker_base, r, k, seed, step,
                            scale_mode, d_idx, d_val, d_out, stream);
  if (rc) return rc;
  RTOPK_CUDA(ctx, cudaEventRecord(ctx->ev_consumed[b], st));
  ctx->consumed_valid[b] = true;
  // download: behind the step; the caller's stream waits for it, so that whatever follows on that
  // stream (or a synchronisation of it) sees the results, and the next step does not overwrite them early
  RTOPK_CUDA(ctx, cudaStreamWaitEvent(ctx->copy_out, ctx->ev_consumed[b], 0));
  RTOPK_CUDA(ctx, cudaMemcpyAsync(h_msg_idx, d_idx, (size_t)W * (size_t)k * 4, cudaMemcpyDeviceToHost, ctx->copy_out));
  RTOPK_CUDA(ctx, cudaMemcpyAsync(h_msg_val, d_val, (size_t)W * (size_t)k * 4, cudaMemcpyDeviceToHost, ctx->copy_out));
  RTOPK_CUDA(ctx, cudaMemcpyAsync(h_out, d_out, (size_t)d * 4, cudaMemcpyDeviceToHost, ctx->copy_out));
  RTOPK_CUDA(ctx, cudaEventRecord(ctx->ev_downloaded, ctx->copy_out));
  RTOPK_CUDA(ctx, cudaStreamWaitEvent(st, ctx->ev_downloaded, 0));
  return RTOPK_OK;
}

int rtopk_sample_positions(rtopk_ctx* ctx, int64_t r, int64_t k, uint64_t seed, uint32_t step, uint32_t worker,
                           uint32_t segment, uint32_t* pos, void* stream) {
  if (!ctx || !pos || k < 1 || k > r || r > ctx->r_max || k > ctx->k_max) return RTOPK_ERR_INVALID_ARG;
  cudaStream_t st = (cudaStream_t)stream;
  DeviceGuard guard(ctx->device);
  if (!guard.ok) return RTOPK_ERR_CUDA;
  Plan P;
  P.slices.resize(1);
  Slice& sl = P.slices[0];
  std::memset(&sl, 0, sizeof(sl));
  sl.len = (uint32_t)r; sl.r = (uint32_t)r; sl.k = (uint32_t)k; sl.row = 0; sl.segment = segment;
  P.any_sampler = k < r;
  P.k_draw_max = (uint32_t)k;
  P.first_entries = k < r ? (size_t)first_table_entries(sl) : 0;
  if (P.first_entries > ctx->first_entries) return RTOPK_ERR_INVALID_ARG;
  P.sel_words = ((size_t)r + 31) / 32;
  P.sel_words_max = (uint32_t)P.sel_words;
  Launch L;
  std::memset(&L, 0, sizeof(L));
  const size_t zbytes = carve_zero(ctx, P, L.s);
  if (zbytes > ctx->zero_bytes) return RTOPK_ERR_INVALID_ARG;
  L.s.slices = ctx->d_slices; L.s.state = ctx->d_state; L.s.draws = ctx->d_draws; L.s.first = ctx->d_first;
  L.s.sel_pre = ctx->d_sel_pre; L.s.sel_blk = ctx->d_sel_blk; L.s.error = ctx->d_error;
  L.n_slices = 1; L.worker_base = worker; L.seed_lo = (uint32_t)seed; L.seed_hi = (uint32_t)(seed >> 32);
  L.step = step;
  int rc = upload_slices(ctx, P, st);
  if (rc) return rc;
  RTOPK_CUDA(ctx, cudaMemsetAsync(ctx->d_zero, 0, zbytes, st));
  rc = run_sampler(ctx, P, L, st, true);
  if (rc) return rc;
  const uint32_t nwords = (uint32_t)((r + 31) / 32);
  k_positions<<<(nwords + kThreads - 1) / kThreads, kThreads, 0, st>>>(L, pos);
  ++ctx->launches;
  RTOPK_CUDA(ctx, cudaGetLastError());
  return RTOPK_OK;
}

int rtopk_set_device_step(rtopk_ctx* ctx, uint32_t step, void* stream) {
  if (!ctx) return RTOPK_ERR_INVALID_ARG;
  DeviceGuard guard(ctx->device);
  if (!guard.ok) return RTOPK_ERR_CUDA;
  k_step_set<<<1, 32, 0, (cudaStream_t)stream>>>(ctx->d_step, step);
  ++ctx->launches;
  RTOPK_CUDA(ctx, cudaGetLastError());
  return RTOPK_OK;
}

int rtopk_poll_status(rtopk_ctx* ctx, void* stream) {
  if (!ctx) return RTOPK_ERR_INVALID_ARG;
  cudaStream_t st = (cudaStream_t)stream;
  DeviceGuard guard(ctx->device);
  if (!guard.ok) return RTOPK_ERR_CUDA;
  uint32_t flags = 0;
  RTOPK_CUDA(ctx, cudaMemcpyAsync(&flags, ctx->d_error, sizeof(flags), cudaMemcpyDeviceToHost, st));
  RTOPK_CUDA(ctx, cudaStreamSynchronize(st));
  if (flags) {
    RTOPK_CUDA(ctx, cudaMemsetAsync(ctx->d_error, 0, sizeof(flags), st));
    return RTOPK_ERR_INTERNAL;
  }
  return RTOPK_OK;
}

int rtopk_get_phase_times(rtopk_ctx* ctx, float* ms, void* stream) {
  if (!ctx || !ms) return RTOPK_ERR_INVALID_ARG;
  DeviceGuard guard(ctx->device);
  if (!guard.ok) return RTOPK_ERR_CUDA;
  RTOPK_CUDA(ctx, cudaStreamSynchronize((cudaStream_t)stream));
  for (int i = 0; i < RTOPK_N_PHASES; ++i) {
    ms[i] = -1.0f;
    if (ctx->profile && ctx->ev_valid[i] && ctx->ev_valid[i + 1]) {
      float t = 0.f;
      if (cudaEventElapsedTime(&t, ctx->ev[i], ctx->ev[i + 1]) == cudaSuccess) ms[i] = t;
      else cudaGetLastError();
    }
  }
  return RTOPK_OK;
}

int rtopk_get_stats(rtopk_ctx* ctx, int32_t slice, rtopk_stats* out, void* stream) {
  if (!ctx || !out || slice < 0 || (uint32_t)slice >= ctx->last_n_slices) return RTOPK_ERR_INVALID_ARG;
  cudaStream_t st = (cudaStream_t)stream;
  DeviceGuard guard(ctx->device);
  if (!guard.ok) return RTOPK_ERR_CUDA;
  SelState s;
  RTOPK_CUDA(ctx, cudaMemcpyAsync(&s, ctx->d_state + slice, sizeof(s), cudaMemcpyDeviceToHost, st));
  RTOPK_CUDA(ctx, cudaStreamSynchronize(st));
  std::memset(out, 0, sizeof(*out));
  out->tau_key = s.prefix;
  out->tie_quota = s.need;
  out->n_greater = s.n_gt;
  out->n_candidates = s.n_cand;
  out->used_fallback = (s.flags & FLAG_FELL_BACK) ? 1u : 0u;
  out->bracket_predicted = s.pred != 0 ? 1u : 0u;
  return RTOPK_OK;
}

int rtopk_get_launch_count(const rtopk_ctx* ctx, uint64_t* out) {
  if (!ctx || !out) return RTOPK_ERR_INVALID_ARG;
  *out = ctx->launches;
  return RTOPK_OK;
}

// ----------------------------------------------------------------------------- no-allocation call
// Scratch of rtopk_sample_positions_static: one slice descriptor, then the draw buffer, the
// first-occurrence table, the position bitmap and its prefix, each sized for RTOPK_STATIC_MAX_R.
// The array lives in the device image; its name below is only a host-side handle, the device
// address comes from cudaGetSymbolAddress (once per device).
namespace {
constexpr size_t kStaticR = (size_t)RTOPK_STATIC_MAX_R;
constexpr size_t kStaticSliceBytes = 256;
constexpr size_t kStaticDrawsOff = kStaticSliceBytes;
constexpr size_t kStaticFirstOff = kStaticDrawsOff + kStaticR * 4;
constexpr size_t kStaticSelOff = kStaticFirstOff + kStaticR * 4;
constexpr size_t kStaticPreOff = kStaticSelOff + (kStaticR / 32 + 8) * 4;
constexpr size_t kStaticBlkOff = kStaticPreOff + (kStaticR / 32 + 8) * 4;
constexpr size_t kStaticBytes = kStaticBlkOff + 256;
static_assert(sizeof(Slice) <= kStaticSliceBytes, "slice descriptor must fit its slot");
}  // namespace

static __device__ __align__(256) unsigned char g_static_scratch[kStaticBytes];

namespace {
constexpr int kStaticMaxDevices = 64;
std::mutex g_static_mutex;
unsigned char* g_static_ptr[kStaticMaxDevices] = {};

// Writes the one-slice table the subset kernels read (no host-to-device copy needed).
__global__ void k_static_slice(Slice* slot, uint32_t r, uint32_t k, uint32_t segment) {
  if (blockIdx.x != 0 || threadIdx.x != 0) return;
  Slice s;
  s.g_off = 0; s.m_off = 0; s.len = r; s.r = r; s.k = k; s.row = 0; s.segment = segment; s.idx_base = 0;
  s.head = 0; s.msg_off = 0; s.cand_off = 0; s.cand_cap = 0; s.chunk_begin = 0; s.hist_begin = 0;
  s.group_begin = 0; s.samp_off = 0; s.first_off = 0; s.first_mask = 0; s.sel_off = 0; s.gshift = 5;
  *slot = s;
}
}  // namespace

int rtopk_sample_positions_static(int64_t r, int64_t k, uint64_t seed, uint32_t step, uint32_t worker,
                                  uint32_t segment, uint32_t* pos, void* stream) {
  if (!pos || k < 1 || k > r) return RTOPK_ERR_INVALID_ARG;
  if (r > (int64_t)RTOPK_STATIC_MAX_R) return RTOPK_ERR_UNSUPPORTED;
  cudaStream_t st = (cudaStream_t)stream;
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kStaticMaxDevices) return RTOPK_ERR_CUDA;
  unsigned char* base = nullptr;
  {
    // set-up, once per device, with that device current: the symbol's device address
    std::lock_guard<std::mutex> lock(g_static_mutex);
    if (!g_static_ptr[dev]) {
      void* p = nullptr;
      if (cudaGetSymbolAddress(&p, g_static_scratch) != cudaSuccess || !p) { cudaGetLastError(); return RTOPK_ERR_CUDA; }
      g_static_ptr[dev] = static_cast<unsigned char*>(p);
    }
    base = g_static_ptr[dev];
  }
  Launch L;
  std::memset(&L, 0, sizeof(L));
  L.s.slices = reinterpret_cast<Slice*>(base);
  L.s.draws = reinterpret_cast<uint32_t*>(base + kStaticDrawsOff);
  L.s.first = reinterpret_cast<uint32_t*>(base + kStaticFirstOff);
  L.s.sel = reinterpret_cast<uint32_t*>(base + kStaticSelOff);
  L.s.sel_pre = reinterpret_cast<uint32_t*>(base + kStaticPreOff);
  L.s.sel_blk = reinterpret_cast<uint32_t*>(base + kStaticBlkOff);
  L.n_slices = 1; L.worker_base = worker; L.seed_lo = (uint32_t)seed; L.seed_hi = (uint32_t)(seed >> 32);
  L.step = step;
  const uint32_t nwords = (uint32_t)((r + 31) / 32);
  k_static_slice<<<1, 32, 0, st>>>(L.s.slices, (uint32_t)r, (uint32_t)k, segment);
  if (k < r) {
    // the array keeps the previous call's contents: the table starts at "never drawn", the bitmap at zero
    if (cudaMemsetAsync(L.s.first, 0xFF, (size_t)r * sizeof(uint32_t), st) != cudaSuccess) return RTOPK_ERR_CUDA;
    if (cudaMemsetAsync(L.s.sel, 0, (size_t)nwords * sizeof(uint32_t), st) != cudaSuccess) return RTOPK_ERR_CUDA;
    const dim3 grid(((uint32_t)k + kDrawThreads - 1) / kDrawThreads, 1);
    k_draw<<<grid, kDrawThreads, 0, st>>>(L);
    k_resolve<<<grid, kDrawThreads, 0, st>>>(L);
    const dim3 sgrid((nwords + kSelChunk - 1) / kSelChunk, 1);   // at most 4 chunks at the largest r
    k_sel_count<<<sgrid, kScanThreads, 0, st>>>(L);
    k_sel_scan<<<sgrid, kScanThreads, 0, st>>>(L);
  }
  k_positions<<<(nwords + kThreads - 1) / kThreads, kThreads, 0, st>>>(L, pos);
  return cudaGetLastError() == cudaSuccess ? RTOPK_OK : RTOPK_ERR_CUDA;
}

}  // extern "C"
