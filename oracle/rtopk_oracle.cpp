// rTop-k CPU oracle -- TEST INFRASTRUCTURE, not a product path.
//
// A plain, slow, single-pass-per-definition restatement of the data-parallel
// hot path of rTop-k (Barnes, Inan, Isik, Ozgur: "rTop-k: A Statistical
// Estimation Approach to Distributed SGD"):
//
//   Algorithm 1, node body:   a = g + m ; ghat = rTop_k(a) ; m' = a - ghat ; send ghat
//   Algorithm 1, master:      ghat = (1/n) * sum_i ghat_i ; w' = w - eta * ghat
//   Definition 1 (top-r), Definition 2 (random-k), Definition 3 (rTop-k).
//
// Only the tests, the smoke check and the benchmark's cpu_baseline leg may call
// this file.  It shares no code, header, table or constant generator with the
// CUDA library.  Nothing here is blocked, fused or reordered: the top-r set is
// a full sort, the k-subset is the sequential Floyd loop, the aggregate is a
// dense double-precision accumulation in worker order.
//
// Readings where the paper is silent (fixed by the library's contract):
//   * ties in |a| (Def. 1 says "a permutation"): larger magnitude first, then
//     the lower index;
//   * "uniformly at random" (Def. 3): Floyd's subset algorithm on positions
//     0..r-1 of the top-r set numbered by ascending index, driven by
//     Philox4x32-10 (Salmon, Moraes, Dror, Shaw, SC'11) with
//     counter = (j, worker, segment, step), key = (seed lo, seed hi);
//   * a, m, message values and the update are IEEE binary32; the add is one
//     round-to-nearest add; magnitudes are compared through the bit pattern
//     with the sign cleared (so NaN > Inf > finite, and -0 ties with +0);
//   * IEEE 754 leaves the payload of a NaN result to the implementation, so a NaN sum is stored as
//     the default quiet NaN (bit pattern 0x7FC00000);
//   * m' is a bit copy of a outside the sent set and +0.0f inside it;
//   * messages are listed by ascending index;
//   * the master update rounds once: w' = fp32(double(w) - double(eta) * double(ghat)) with ghat
//     the binary32 average (the product of two binary32 numbers is exact in binary64).
//
// Pins (tests/test_oracle_*.py): Philox against published known answers; the
// draw scaling against big-integer arithmetic; Floyd against exhaustive
// enumeration (every k-subset equally often); top-r against brute force and
// library sorts; the whole operator against the closed form in the proof of
// Proposition 1 and the limits k = r (Def. 1) and r = d (Def. 2); the
// threshold-then-subsample encoder (proof of Theorem 1) against a library
// comparison of magnitudes, exhaustive enumeration of the kept subsets, the
// exact unbiasedness of its estimator and the identity sum(X~ / S) = ||X||_1;
// the momentum form of the master update against worked steps in exact binary
// fractions, its mu = 0 limit, a library optimizer run in binary64 and the
// geometric series; the span-table message format against a hand-worked row, a
// library lower-bound search, the bit-packed format and bfloat16 of a library.

#include <algorithm>
#include <cmath>
#include <cstdint>
#include <cstring>
#include <thread>
#include <vector>

namespace {

enum { ORACLE_OK = 0, ORACLE_BAD_ARG = 1 };
enum { GRAD_F32 = 0, GRAD_BF16 = 1 };
enum { SCALE_MEAN = 0, SCALE_SUM = 1, SCALE_UNBIASED = 2, SCALE_COUNT = 3 };

int g_threads = 1;

// ---- Philox4x32-10, from the published definition (SC'11, Section 3.3) ------
// One round: two 32x32->64 products of counter words 0 and 2 with the two
// round multipliers; the high halves are XORed with counter words 1 and 3 and
// with the key and cross over; the low halves pass through.  Between rounds
// the key words are bumped by the two Weyl constants (golden ratio, sqrt(3)-1).
void philox4x32_10(const uint32_t c_in[4], const uint32_t k_in[2], uint32_t out[4]) {
  const uint64_t MUL_A = 0xD2511F53u;  // multiplies counter word 0
  const uint64_t MUL_B = 0xCD9E8D57u;  // multiplies counter word 2
  const uint32_t WEYL_0 = 0x9E3779B9u;
  const uint32_t WEYL_1 = 0xBB67AE85u;
  uint32_t c0 = c_in[0], c1 = c_in[1], c2 = c_in[2], c3 = c_in[3];
  uint32_t k0 = k_in[0], k1 = k_in[1];
  for (int round = 0; round < 10; ++round) {
    const uint64_t pa = MUL_A * (uint64_t)c0;
    const uint64_t pb = MUL_B * (uint64_t)c2;
    const uint32_t n0 = (uint32_t)(pb >> 32) ^ c1 ^ k0;
    const uint32_t n1 = (uint32_t)pb;
    const uint32_t n2 = (uint32_t)(pa >> 32) ^ c3 ^ k1;
    const uint32_t n3 = (uint32_t)pa;
    c0 = n0; c1 = n1; c2 = n2; c3 = n3;
    k0 += WEYL_0;
    k1 += WEYL_1;
  }
  out[0] = c0; out[1] = c1; out[2] = c2; out[3] = c3;
}

// floor(u * n / 2^64): maps a 64-bit uniform word onto {0, ..., n-1}.
uint32_t scale_draw(uint64_t u, uint32_t n) {
  return (uint32_t)(((unsigned __int128)u * (unsigned __int128)n) >> 64);
}

// The draw Floyd's loop makes at iteration j: uniform on {0, ..., j}.
uint32_t draw_t(uint64_t seed, uint32_t step, uint32_t worker, uint32_t segment, uint32_t j) {
  const uint32_t ctr[4] = {j, worker, segment, step};
  const uint32_t key[2] = {(uint32_t)seed, (uint32_t)(seed >> 32)};
  uint32_t x[4];
  philox4x32_10(ctr, key, x);
  const uint64_t u = ((uint64_t)x[1] << 32) | (uint64_t)x[0];
  return scale_draw(u, j + 1u);
}

// Floyd's k-of-r subset algorithm, sequential, with the draws supplied:
// t[i] is the draw of iteration j = r-k+i and must lie in {0..j}.
// Writes the k chosen positions in ascending order.
void floyd_from_draws(int64_t r, int64_t k, const uint32_t* t, uint32_t* pos) {
  std::vector<uint8_t> in_set((size_t)r, 0);
  for (int64_t j = r - k; j < r; ++j) {
    const uint32_t tj = t[j - (r - k)];
    if (!in_set[tj]) in_set[tj] = 1;
    else             in_set[(size_t)j] = 1;
  }
  int64_t n = 0;
  for (int64_t p = 0; p < r; ++p)
    if (in_set[(size_t)p]) pos[n++] = (uint32_t)p;
}

void sample_positions(int64_t r, int64_t k, uint64_t seed, uint32_t step, uint32_t worker,
                      uint32_t segment, uint32_t* pos) {
  std::vector<uint32_t> t((size_t)k);
  for (int64_t j = r - k; j < r; ++j)
    t[(size_t)(j - (r - k))] = draw_t(seed, step, worker, segment, (uint32_t)j);
  floyd_from_draws(r, k, t.data(), pos);
}

inline uint32_t float_bits(float x) { uint32_t b; std::memcpy(&b, &x, 4); return b; }
inline float bits_float(uint32_t b) { float x; std::memcpy(&x, &b, 4); return x; }
inline uint32_t magnitude_key(float x) { return float_bits(x) & 0x7FFFFFFFu; }

struct KeyIdx { uint32_t key; uint32_t idx; };

// Definition 1: indices of the r largest-magnitude entries, ties to the lower
// index; returned in ascending index order.
void top_r_indices(const float* a, int64_t d, int64_t r, uint32_t* L) {
  std::vector<KeyIdx> order((size_t)d);
  for (int64_t i = 0; i < d; ++i) order[(size_t)i] = KeyIdx{magnitude_key(a[i]), (uint32_t)i};
  std::sort(order.begin(), order.end(), [](const KeyIdx& x, const KeyIdx& y) {
    if (x.key != y.key) return x.key > y.key;
    return x.idx < y.idx;
  });
  for (int64_t p = 0; p < r; ++p) L[p] = order[(size_t)p].idx;
  std::sort(L, L + r);
}

inline float widen_grad(const void* grad, int dtype, int64_t i) {
  if (dtype == GRAD_F32) return ((const float*)grad)[i];
  const uint16_t h = ((const uint16_t*)grad)[i];   // bfloat16 = top half of binary32
  return bits_float((uint32_t)h << 16);
}

// One worker, one slice [0, d) of its vector (Algorithm 1 node body).
// grad/residual point at the slice; idx_base is added to reported indices.
void sparsify_slice(const void* grad, int dtype, float* residual, int64_t d, int64_t r, int64_t k,
                    uint64_t seed, uint32_t step, uint32_t worker, uint32_t segment,
                    uint32_t idx_base, uint32_t* msg_idx, float* msg_val) {
  // the error-compensated vector (Algorithm 1), kept in the residual buffer from here on
  for (int64_t i = 0; i < d; ++i) {
    float s = widen_grad(grad, dtype, i) + residual[i];   // one binary32 add
    if (s != s) s = bits_float(0x7FC00000u);              // NaN payloads are not portable: store the default NaN
    residual[i] = s;
  }
  // Definition 1: full sort by (magnitude descending, index ascending), first r, listed by ascending index
  std::vector<uint32_t> L((size_t)r);
  top_r_indices(residual, d, r, L.data());
  // Definition 3: k positions of that list, by the sequential Floyd loop on Philox draws
  std::vector<uint32_t> pos((size_t)k);
  sample_positions(r, k, seed, step, worker, segment, pos.data());
  // the chosen coordinates are sent with their values; what is sent leaves the residual (+0.0f there)
  for (int64_t q = 0; q < k; ++q) {
    const uint32_t i = L[pos[(size_t)q]];
    msg_idx[q] = idx_base + i;
    msg_val[q] = residual[i];
    residual[i] = 0.0f;
  }
}

template <class F>
void for_each_row(int W, F&& body) {
  const int nt = std::max(1, std::min(g_threads, W));
  if (nt == 1) { for (int w = 0; w < W; ++w) body(w); return; }
  std::vector<std::thread> pool;
  for (int t = 0; t < nt; ++t)
    pool.emplace_back([&, t] { for (int w = t; w < W; w += nt) body(w); });
  for (auto& th : pool) th.join();
}

}  // namespace

extern "C" {

// Rows (workers) are independent; this only sets how many host threads walk them.
void oracle_set_threads(int n) { g_threads = n < 1 ? 1 : n; }
int  oracle_get_threads(void) { return g_threads; }

void oracle_philox4x32_10(const uint32_t* ctr, const uint32_t* key, uint32_t* out) {
  philox4x32_10(ctr, key, out);
}

uint32_t oracle_scale_draw(uint64_t u, uint32_t n) { return scale_draw(u, n); }

uint32_t oracle_draw(uint64_t seed, uint32_t step, uint32_t worker, uint32_t segment, uint32_t j) {
  return draw_t(seed, step, worker, segment, j);
}

int oracle_floyd_from_draws(int64_t r, int64_t k, const uint32_t* t, uint32_t* pos) {
  if (r < 1 || k < 1 || k > r || !t || !pos) return ORACLE_BAD_ARG;
  for (int64_t j = r - k; j < r; ++j)
    if ((int64_t)t[j - (r - k)] > j) return ORACLE_BAD_ARG;
  floyd_from_draws(r, k, t, pos);
  return ORACLE_OK;
}

int oracle_sample_positions(int64_t r, int64_t k, uint64_t seed, uint32_t step, uint32_t worker,
                            uint32_t segment, uint32_t* pos) {
  if (r < 1 || k < 1 || k > r || r > 0x7FFFFFFF || !pos) return ORACLE_BAD_ARG;
  sample_positions(r, k, seed, step, worker, segment, pos);
  return ORACLE_OK;
}

int oracle_top_r(const float* a, int64_t d, int64_t r, uint32_t* L) {
  if (!a || !L || d < 1 || r < 1 || r > d || d > 0x7FFFFFFF) return ORACLE_BAD_ARG;
  top_r_indices(a, d, r, L);
  return ORACLE_OK;
}

// Algorithm 1 node body for W workers held as rows of grad (W x ld_g) and
// residual (W x ld_m, updated in place).  Row w is worker worker_base + w.
// Messages: msg_idx / msg_val are W x k, ascending index within a row.
int oracle_sparsify(const void* grad, int grad_dtype, int64_t ld_g, float* residual, int64_t ld_m,
                    int64_t d, int32_t W, int32_t worker_base, int64_t r, int64_t k, uint64_t seed,
                    uint32_t step, uint32_t* msg_idx, float* msg_val) {
  if (!grad || !residual || !msg_idx || !msg_val) return ORACLE_BAD_ARG;
  if (d < 1 || d > 0x7FFFFFFF || W < 1 || k < 1 || k > r || r > d || ld_g < d || ld_m < d)
    return ORACLE_BAD_ARG;
  if (grad_dtype != GRAD_F32 && grad_dtype != GRAD_BF16) return ORACLE_BAD_ARG;
  const size_t gsz = grad_dtype == GRAD_F32 ? 4 : 2;
  for_each_row(W, [&](int w) {
    sparsify_slice((const char*)grad + (size_t)w * (size_t)ld_g * gsz, grad_dtype,
                   residual + (size_t)w * (size_t)ld_m, d, r, k, seed, step,
                   (uint32_t)(worker_base + w), 0u, 0u,
                   msg_idx + (size_t)w * (size_t)k, msg_val + (size_t)w * (size_t)k);
  });
  return ORACLE_OK;
}

// Per-tensor variant: the vector is cut at seg_off[0..S] (seg_off[0] = 0,
// seg_off[S] = d) and rTop-k with (seg_r[s], seg_k[s]) is applied to every
// slice independently; the Philox counter carries s.  A row's message holds
// K = sum_s seg_k[s] entries: slice 0's first, each with flat indices.
int oracle_sparsify_segmented(const void* grad, int grad_dtype, int64_t ld_g, float* residual,
                              int64_t ld_m, int64_t d, int32_t W, int32_t worker_base, int32_t S,
                              const int64_t* seg_off, const int64_t* seg_r, const int64_t* seg_k,
                              uint64_t seed, uint32_t step, uint32_t* msg_idx, float* msg_val) {
  if (!grad || !residual || !msg_idx || !msg_val || !seg_off || !seg_r || !seg_k) return ORACLE_BAD_ARG;
  if (d < 1 || d > 0x7FFFFFFF || W < 1 || S < 1 || ld_g < d || ld_m < d) return ORACLE_BAD_ARG;
  if (grad_dtype != GRAD_F32 && grad_dtype != GRAD_BF16) return ORACLE_BAD_ARG;
  if (seg_off[0] != 0 || seg_off[S] != d) return ORACLE_BAD_ARG;
  int64_t K = 0;
  for (int s = 0; s < S; ++s) {
    const int64_t len = seg_off[s + 1] - seg_off[s];
    if (len < 1 || seg_k[s] < 1 || seg_k[s] > seg_r[s] || seg_r[s] > len) return ORACLE_BAD_ARG;
    K += seg_k[s];
  }
  const size_t gsz = grad_dtype == GRAD_F32 ? 4 : 2;
  for_each_row(W, [&](int w) {
    int64_t at = 0;
    for (int s = 0; s < S; ++s) {
      const int64_t lo = seg_off[s], len = seg_off[s + 1] - lo;
      sparsify_slice((const char*)grad + ((size_t)w * (size_t)ld_g + (size_t)lo) * gsz, grad_dtype,
                     residual + (size_t)w * (size_t)ld_m + (size_t)lo, len, seg_r[s], seg_k[s],
                     seed, step, (uint32_t)(worker_base + w), (uint32_t)s, (uint32_t)lo,
                     msg_idx + (size_t)w * (size_t)K + (size_t)at,
                     msg_val + (size_t)w * (size_t)K + (size_t)at);
      at += seg_k[s];
    }
  });
  return ORACLE_OK;
}

// Algorithm 1, master: dense sum of the W sparse messages in double precision,
// workers in order, scaled by 1/W (mean) or 1 (sum).  out64 (optional) receives
// the double result; out32 (optional) the same rounded once to binary32.
// Algorithm 1, master step, with the scalings of the library's contract: S_i = sum of the values
// the workers sent for coordinate i (double, worker order), c_i = how many sent it;
//   MEAN S_i / W;  SUM S_i;  UNBIASED S_i * r / (W k) (the estimator in the proof of Theorem 1 with
//   subsampling fraction k / r);  COUNT S_i / c_i (0 where nobody sent i).
int oracle_aggregate_scaled(const uint32_t* msg_idx, const float* msg_val, int64_t d, int32_t W, int64_t k,
                            int scale_mode, int64_t r, double* out64, float* out32) {
  if (!msg_idx || !msg_val || d < 1 || W < 1 || k < 1) return ORACLE_BAD_ARG;
  if (scale_mode != SCALE_MEAN && scale_mode != SCALE_SUM && scale_mode != SCALE_UNBIASED && scale_mode != SCALE_COUNT)
    return ORACLE_BAD_ARG;
  if (scale_mode == SCALE_UNBIASED && (r < k || r > d)) return ORACLE_BAD_ARG;
  std::vector<double> acc((size_t)d, 0.0);
  std::vector<uint32_t> senders((size_t)d, 0u);
  for (int32_t w = 0; w < W; ++w)
    for (int64_t q = 0; q < k; ++q) {
      const uint32_t i = msg_idx[(size_t)w * (size_t)k + (size_t)q];
      if ((int64_t)i >= d) return ORACLE_BAD_ARG;
      acc[i] += (double)msg_val[(size_t)w * (size_t)k + (size_t)q];
      senders[i] += 1u;
    }
  for (int64_t i = 0; i < d; ++i) {
    const double s = acc[(size_t)i];
    double v = s;
    if (scale_mode == SCALE_MEAN) v = s / (double)W;
    else if (scale_mode == SCALE_UNBIASED) v = (s * (double)r) / ((double)W * (double)k);
    else if (scale_mode == SCALE_COUNT) v = senders[(size_t)i] ? s / (double)senders[(size_t)i] : 0.0;
    if (out64) out64[i] = v;
    if (out32) out32[i] = (float)v;
  }
  return ORACLE_OK;
}

int oracle_aggregate(const uint32_t* msg_idx, const float* msg_val, int64_t d, int32_t W, int64_t k,
                     int scale_mode, double* out64, float* out32) {
  if (scale_mode != SCALE_MEAN && scale_mode != SCALE_SUM && scale_mode != SCALE_COUNT) return ORACLE_BAD_ARG;
  return oracle_aggregate_scaled(msg_idx, msg_val, d, W, k, scale_mode, 0, out64, out32);
}

// Algorithm 1, master update: w <- w - eta * ghat with ghat the average (or sum) above, for every
// coordinate.  eta >= 0 (with a negative eta a zero weight at an unsent coordinate would change
// its sign, which the sparse restatements of this update never touch).
int oracle_apply_update(const uint32_t* msg_idx, const float* msg_val, int64_t d, int32_t W, int64_t k,
                        int scale_mode, int64_t r, float eta, float* weights) {
  if (!weights || !(eta >= 0.0f) || eta > 3.0e38f) return ORACLE_BAD_ARG;
  std::vector<float> ghat((size_t)d);
  const int rc = oracle_aggregate_scaled(msg_idx, msg_val, d, W, k, scale_mode, r, nullptr, ghat.data());
  if (rc != ORACLE_OK) return rc;
  for (int64_t i = 0; i < d; ++i)
    weights[i] = (float)((double)weights[i] - (double)eta * (double)ghat[(size_t)i]);
  return ORACLE_OK;
}

// Section IV trains with momentum SGD.  The paper prints no formula for it; the reading taken is the
// heavy-ball form on the master, applied to the average of Algorithm 1:
//     v <- mu * v + ghat ;   w <- w - eta * v        for every coordinate, sent or not
// (with mu = 0 it is the master update above).  Each of the two lines rounds once from binary64:
// v' = fp32(double(mu) * double(v) + double(ghat)) -- the product is exact in binary64, the sum is
// rounded to binary64 and then to binary32 -- and w' = fp32(double(w) - double(eta) * double(v')).
// 0 <= mu < 1, eta >= 0.
int oracle_apply_momentum(const uint32_t* msg_idx, const float* msg_val, int64_t d, int32_t W, int64_t k,
                          int scale_mode, int64_t r, float eta, float mu, float* velocity, float* weights) {
  if (!weights || !velocity || !(eta >= 0.0f) || eta > 3.0e38f || !(mu >= 0.0f) || !(mu < 1.0f)) return ORACLE_BAD_ARG;
  std::vector<float> ghat((size_t)d);
  const int rc = oracle_aggregate_scaled(msg_idx, msg_val, d, W, k, scale_mode, r, nullptr, ghat.data());
  if (rc != ORACLE_OK) return rc;
  for (int64_t i = 0; i < d; ++i) {
    const float v = (float)((double)mu * (double)velocity[i] + (double)ghat[(size_t)i]);
    velocity[i] = v;
    weights[i] = (float)((double)weights[i] - (double)eta * (double)v);
  }
  return ORACLE_OK;
}

// ----------------------------------------------------------------------------- warm-up schedule
// Section IV: sparsity is increased exponentially during the warm-up period, and k / r = 1 / n.
// density(t) = initial * (final / initial)^(t / T) for t < T, final afterwards;
// k = clamp(floor(density d), 1, d), r = min(d, n k).
int oracle_warmup_sizes(int64_t d, int32_t n, double initial, double final_, int64_t T, int64_t t, int64_t* r,
                        int64_t* k) {
  if (d < 1 || n < 1 || t < 0 || T < 0 || !r || !k || !(final_ > 0.0) || !(initial >= final_) || !(initial <= 1.0))
    return ORACLE_BAD_ARG;
  const double density = t < T ? initial * std::pow(final_ / initial, (double)t / (double)T) : final_;
  int64_t kk = (int64_t)(density * (double)d);
  kk = std::max<int64_t>(1, std::min<int64_t>(d, kk));
  *k = kk;
  *r = (int64_t)std::min<double>((double)d, (double)kk * (double)n);
  return ORACLE_OK;
}

// ----------------------------------------------------------------------------- message codec
// Section III notes that an index costs log d bits and a value a constant number of bits.  The
// library's packed message format states one such encoding:
//   * indices: b = ceil(log2 d) bits each (1 when d <= 2), entry j at bits [j b, (j + 1) b) of the
//     row's bit stream; bit p of the stream is bit (p mod 32) of 32-bit word p / 32;
//   * values: bfloat16 = the upper 16 bits of the binary32 value rounded to nearest, ties to even
//     (a NaN becomes 0x7FC0);
//   * error feedback of the rounding (Algorithm 1: m = a - ghat with ghat what is sent): the
//     residual slot of a sent coordinate receives a - widen(q(a)), one binary32 subtraction, or
//     +0.0f when widen(q(a)) is not finite.
int oracle_index_bits(int64_t d) {
  int b = 1;
  while (b < 63 && ((int64_t)1 << b) < d) ++b;
  return b;
}

uint16_t oracle_bf16_rne(float x) {
  uint32_t u;
  std::memcpy(&u, &x, 4);
  if ((u & 0x7FFFFFFFu) > 0x7F800000u) return 0x7FC0u;          // NaN
  const uint32_t lsb = (u >> 16) & 1u;
  u += 0x7FFFu + lsb;                                            // round to nearest, ties to even
  return (uint16_t)(u >> 16);
}

// One row: k ascending (index, value) pairs -> packed_idx (ceil(k b / 32) words, zero-filled first)
// and packed_val (k halves); residual (may be null) gets the rounding error at the sent coordinates.
int oracle_encode_row(const uint32_t* idx, const float* val, int64_t k, int64_t d, uint32_t* packed_idx,
                      uint16_t* packed_val, float* residual) {
  if (!idx || !val || !packed_idx || !packed_val || k < 1 || d < 1) return ORACLE_BAD_ARG;
  const int b = oracle_index_bits(d);
  if (b > 32) return ORACLE_BAD_ARG;
  const int64_t nwords = (k * b + 31) / 32;
  for (int64_t w = 0; w < nwords; ++w) packed_idx[w] = 0;
  for (int64_t j = 0; j < k; ++j) {
    if ((int64_t)idx[j] >= d) return ORACLE_BAD_ARG;
    for (int bit = 0; bit < b; ++bit)
      if ((idx[j] >> bit) & 1u) {
        const int64_t p = j * b + bit;
        packed_idx[p / 32] |= 1u << (p % 32);
      }
    const uint16_t q = oracle_bf16_rne(val[j]);
    packed_val[j] = q;
    if (residual) {
      const uint32_t wide = (uint32_t)q << 16;
      float back;
      std::memcpy(&back, &wide, 4);
      residual[idx[j]] = std::isfinite(back) ? val[j] - back : 0.0f;
    }
  }
  return ORACLE_OK;
}

int oracle_decode_row(const uint32_t* packed_idx, const uint16_t* packed_val, int64_t k, int64_t d, uint32_t* idx,
                      float* val) {
  if (!idx || !val || !packed_idx || !packed_val || k < 1 || d < 1) return ORACLE_BAD_ARG;
  const int b = oracle_index_bits(d);
  if (b > 32) return ORACLE_BAD_ARG;
  for (int64_t j = 0; j < k; ++j) {
    uint32_t v = 0;
    for (int bit = 0; bit < b; ++bit) {
      const int64_t p = j * b + bit;
      v |= ((packed_idx[p / 32] >> (p % 32)) & 1u) << bit;
    }
    idx[j] = v;
    const uint32_t wide = (uint32_t)packed_val[j] << 16;
    std::memcpy(&val[j], &wide, 4);
  }
  return ORACLE_OK;
}

// A second format, for rows in ascending index order (which every message here is): Section III's
// log d bits per index are what an index costs on its own, but a sorted row can say the high bits of
// its indices once per stretch.  The coordinates are cut into spans of 2^14 = 16384; a row states
//   * tab[t], t = 0 .. T with T = ceil(d / 16384): how many of its entries have an index below
//     t * 16384 (so tab[0] = 0, tab[T] = k, and the entries of span t are tab[t] .. tab[t + 1] - 1);
//   * low[j] = idx[j] mod 16384 for every entry (16 bits, the upper two zero);
//   * the values as bfloat16, with the same error feedback as above.
// 32 (T + 1) + 32 k bits per row instead of (ceil(log2 d) + 16) k.
constexpr int64_t TILED_SPAN = 16384;

int64_t oracle_tiled_spans(int64_t d) { return d < 1 ? 0 : (d + TILED_SPAN - 1) / TILED_SPAN; }

// One row: k (index, value) pairs in strictly ascending index order -> tab (T + 1 words), low (k halves),
// qval (k halves); residual (may be null) gets the rounding error at the sent coordinates.
int oracle_encode_tiled_row(const uint32_t* idx, const float* val, int64_t k, int64_t d, uint32_t* tab,
                            uint16_t* low, uint16_t* qval, float* residual) {
  if (!idx || !val || !tab || !low || !qval || k < 1 || d < 1 || d > 0xFFFFFFFFll) return ORACLE_BAD_ARG;
  for (int64_t j = 0; j < k; ++j) {
    if ((int64_t)idx[j] >= d) return ORACLE_BAD_ARG;
    if (j > 0 && idx[j] <= idx[j - 1]) return ORACLE_BAD_ARG;
  }
  const int64_t T = oracle_tiled_spans(d);
  for (int64_t t = 0; t <= T; ++t) {
    int64_t below = 0;
    for (int64_t j = 0; j < k; ++j)
      if ((int64_t)idx[j] < t * TILED_SPAN) ++below;
    tab[t] = (uint32_t)below;
  }
  for (int64_t j = 0; j < k; ++j) {
    low[j] = (uint16_t)(idx[j] % TILED_SPAN);
    const uint16_t q = oracle_bf16_rne(val[j]);
    qval[j] = q;
    if (residual) {
      const uint32_t wide = (uint32_t)q << 16;
      float back;
      std::memcpy(&back, &wide, 4);
      residual[idx[j]] = std::isfinite(back) ? val[j] - back : 0.0f;
    }
  }
  return ORACLE_OK;
}

int oracle_decode_tiled_row(const uint32_t* tab, const uint16_t* low, const uint16_t* qval, int64_t k, int64_t d,
                            uint32_t* idx, float* val) {
  if (!idx || !val || !tab || !low || !qval || k < 1 || d < 1) return ORACLE_BAD_ARG;
  const int64_t T = oracle_tiled_spans(d);
  if (tab[0] != 0 || (int64_t)tab[T] != k) return ORACLE_BAD_ARG;
  for (int64_t t = 0; t < T; ++t) {
    if (tab[t + 1] < tab[t]) return ORACLE_BAD_ARG;
    for (int64_t j = tab[t]; j < (int64_t)tab[t + 1]; ++j) {
      idx[j] = (uint32_t)(t * TILED_SPAN + low[j]);
      const uint32_t wide = (uint32_t)qval[j] << 16;
      std::memcpy(&val[j], &wide, 4);
    }
  }
  return ORACLE_OK;
}

// ----------------------------------------------------------------------------- threshold, then subsample
// The scheme in the proof of Theorem 1, applied to real-valued vectors as Section II describes for
// continuous observations (quantise by magnitude at a threshold first, then subsample):
//   * X_w marks the coordinates of a = g + m whose magnitude exceeds theta ("1"), the rest are "0";
//     ones_w = ||X_w||_1 travels with the message;
//   * if ones_w > k, k of those coordinates are kept uniformly at random (the same Floyd / Philox
//     subset as Definition 3, over the marked coordinates numbered by ascending index), otherwise
//     all of them; count_w = min(ones_w, k) entries are sent, the subsampling fraction is
//     S_w = count_w / ones_w;
//   * the estimator is (1/n) sum_w Xtilde_w / S_w.
// Readings: a kept coordinate carries its value a_i (as in Definition 3), "exceeds" is the strict
// comparison of the magnitude bit patterns (so a NaN counts as marked), the node keeps m' = a - ghat
// as in Algorithm 1, unused message slots hold index 0xFFFFFFFF and value +0, and one term of the
// estimator is double(value) * (double(ones_w) / double(count_w)), summed in worker order and
// divided by n once.
// `signs` != 0 is the scheme as Section II states it for signed, scaled observations: after the
// quantisation a coordinate is 0 or +-M with M = 2 theta, so a kept coordinate carries sign(a_i) * M
// (one bit on the wire) and the node keeps a_i - sign(a_i) * M there (one binary32 subtraction; a NaN
// difference is stored as the default quiet NaN, like a NaN sum).
int oracle_sparsify_threshold(const void* grad, int grad_dtype, int64_t ld_g, float* residual, int64_t ld_m,
                              int64_t d, int32_t W, int32_t worker_base, float theta, int64_t k, uint64_t seed,
                              uint32_t step, int signs, uint32_t* msg_idx, float* msg_val, uint32_t* msg_count,
                              uint32_t* msg_ones) {
  if (!grad || !residual || !msg_idx || !msg_val || !msg_count || !msg_ones) return ORACLE_BAD_ARG;
  if (d < 1 || d > 0x7FFFFFFF || W < 1 || k < 1 || k > d || ld_g < d || ld_m < d) return ORACLE_BAD_ARG;
  if (grad_dtype != GRAD_F32 && grad_dtype != GRAD_BF16) return ORACLE_BAD_ARG;
  if (!(theta >= 0.0f) || std::isinf(theta)) return ORACLE_BAD_ARG;
  const float M = theta + theta;
  if (signs && std::isinf(M)) return ORACLE_BAD_ARG;
  const size_t gsz = grad_dtype == GRAD_F32 ? 4 : 2;
  const uint32_t theta_key = magnitude_key(theta);
  for_each_row(W, [&](int w) {
    const char* g = (const char*)grad + (size_t)w * (size_t)ld_g * gsz;
    float* a = residual + (size_t)w * (size_t)ld_m;
    uint32_t* out_idx = msg_idx + (size_t)w * (size_t)k;
    float* out_val = msg_val + (size_t)w * (size_t)k;
    // a = g + m
    for (int64_t i = 0; i < d; ++i) {
      float s = widen_grad(g, grad_dtype, i) + a[i];
      if (s != s) s = bits_float(0x7FC00000u);
      a[i] = s;
    }
    // X: the marked coordinates, ascending
    std::vector<uint32_t> marked;
    for (int64_t i = 0; i < d; ++i)
      if (magnitude_key(a[i]) > theta_key) marked.push_back((uint32_t)i);
    const int64_t ones = (int64_t)marked.size();
    // Xtilde: all of them, or k drawn uniformly
    std::vector<uint32_t> kept;
    if (ones > k) {
      std::vector<uint32_t> pos((size_t)k);
      sample_positions(ones, k, seed, step, (uint32_t)(worker_base + w), 0u, pos.data());
      for (int64_t q = 0; q < k; ++q) kept.push_back(marked[pos[(size_t)q]]);
    } else {
      kept = marked;
    }
    msg_ones[w] = (uint32_t)ones;
    msg_count[w] = (uint32_t)kept.size();
    for (int64_t q = 0; q < k; ++q) {
      if (q < (int64_t)kept.size()) {
        const uint32_t i = kept[(size_t)q];
        out_idx[q] = i;
        if (!signs) {
          out_val[q] = a[i];
          a[i] = 0.0f;                                  // m' = a - ghat
        } else {
          const float sent = bits_float((float_bits(a[i]) & 0x80000000u) | float_bits(M));   // sign(a_i) * M
          float rest = a[i] - sent;
          if (rest != rest) rest = bits_float(0x7FC00000u);
          out_val[q] = sent;
          a[i] = rest;
        }
      } else {
        out_idx[q] = 0xFFFFFFFFu;
        out_val[q] = 0.0f;
      }
    }
  });
  return ORACLE_OK;
}

// The estimator of the same proof: out_i = (1/n) sum_w [i kept by w] value_{w,i} / S_w.
int oracle_aggregate_threshold(const uint32_t* msg_idx, const float* msg_val, const uint32_t* msg_count,
                               const uint32_t* msg_ones, int64_t d, int32_t W, int64_t k, double* out64,
                               float* out32) {
  if (!msg_idx || !msg_val || !msg_count || !msg_ones || d < 1 || W < 1 || k < 1) return ORACLE_BAD_ARG;
  std::vector<double> acc((size_t)d, 0.0);
  for (int32_t w = 0; w < W; ++w) {
    const int64_t count = msg_count[w], ones = msg_ones[w];
    if (count > k || count > ones || (ones > k && count != k)) return ORACLE_BAD_ARG;
    if (count == 0) continue;
    const double inv_S = (double)ones / (double)count;
    for (int64_t q = 0; q < count; ++q) {
      const uint32_t i = msg_idx[(size_t)w * (size_t)k + (size_t)q];
      if ((int64_t)i >= d) return ORACLE_BAD_ARG;
      acc[i] += (double)msg_val[(size_t)w * (size_t)k + (size_t)q] * inv_S;
    }
  }
  for (int64_t i = 0; i < d; ++i) {
    const double v = acc[(size_t)i] / (double)W;
    if (out64) out64[i] = v;
    if (out32) out32[i] = (float)v;
  }
  return ORACLE_OK;
}

}  // extern "C"
