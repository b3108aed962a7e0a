// Element access shared by every pass over the gradient and residual matrices: widening loads of
// the gradient type and the error-feedback add of Algorithm 1.
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
// stores it back when STORE, and returns the values with a 4-bit validity mask.
template <typename GradT, bool FUSE, bool STORE = FUSE>
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
      if (STORE) __stcs(reinterpret_cast<float4*>(residual + base_m + e), m4);
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
      if (FUSE) { v = ef_add(Grad<GradT>::ld1(grad, base_g + ee), v); if (STORE) residual[base_m + ee] = v; }
      a[j] = v;
      valid |= 1u << j;
    }
  }
  return valid;
}

}  // namespace rtopk
