// Device helpers shared by the direct-load kernels and the bulk-copy pipeline kernel (internal).
// Every fp32 operation is an explicit round-to-nearest intrinsic, so all kernels that use these
// helpers produce identical bits for identical inputs.
#pragma once
#include <cuda_runtime.h>

#include <cstdint>

#include "nb_kernels.h"

namespace nb {
namespace dev {

__device__ __forceinline__ float4 ld4(const float *p) { return *reinterpret_cast<const float4 *>(p); }
__device__ __forceinline__ void st4(float *p, float4 v) { *reinterpret_cast<float4 *>(p) = v; }

// Raw 4-column gradient fragment as loaded, before widening.
template <int SRC> struct Raw;
template <> struct Raw<kSrcF32> { float4 r; };
template <> struct Raw<kSrcBF16> { uint2 r; };

__device__ __forceinline__ float bf16_lo(uint32_t u) { return __uint_as_float(u << 16); }
__device__ __forceinline__ float bf16_hi(uint32_t u) { return __uint_as_float(u & 0xFFFF0000u); }

__device__ __forceinline__ float4 widen(const Raw<kSrcF32> &x) { return x.r; }
__device__ __forceinline__ float4 widen(const Raw<kSrcBF16> &x) {
  return make_float4(bf16_lo(x.r.x), bf16_hi(x.r.x), bf16_lo(x.r.y), bf16_hi(x.r.y));
}

// Loads columns [off, off+nvalid) of one gradient row; invalid lanes read as +0.  Streaming loads:
// the gradient stream is read exactly once per step.
template <bool ALIGNED>
__device__ __forceinline__ Raw<kSrcF32> load_raw(const float *p, int nvalid, Raw<kSrcF32> *) {
  Raw<kSrcF32> out;
  if (ALIGNED && nvalid == 4) {
    out.r = __ldcs(reinterpret_cast<const float4 *>(p));
  } else {
    out.r = make_float4(0.f, 0.f, 0.f, 0.f);
    if (nvalid > 0) out.r.x = __ldcs(p);
    if (nvalid > 1) out.r.y = __ldcs(p + 1);
    if (nvalid > 2) out.r.z = __ldcs(p + 2);
    if (nvalid > 3) out.r.w = __ldcs(p + 3);
  }
  return out;
}
template <bool ALIGNED>
__device__ __forceinline__ Raw<kSrcBF16> load_raw(const uint16_t *p, int nvalid, Raw<kSrcBF16> *) {
  Raw<kSrcBF16> out;
  if (ALIGNED && nvalid == 4) {
    out.r = __ldcs(reinterpret_cast<const uint2 *>(p));
  } else {
    uint32_t e0 = 0, e1 = 0, e2 = 0, e3 = 0;
    if (nvalid > 0) e0 = __ldcs(p);
    if (nvalid > 1) e1 = __ldcs(p + 1);
    if (nvalid > 2) e2 = __ldcs(p + 2);
    if (nvalid > 3) e3 = __ldcs(p + 3);
    out.r = make_uint2(e0 | (e1 << 16), e2 | (e3 << 16));
  }
  return out;
}

template <int SRC> struct ElemOf;
template <> struct ElemOf<kSrcF32> { using type = float; };
template <> struct ElemOf<kSrcBF16> { using type = uint16_t; };

// v' = mom * v + s * acc  (momentum; s is the per-learner normalisation / learning-rate adjustment)
__device__ __forceinline__ float4 momentum(float mom, float4 v, float s, float4 g) {
  return make_float4(__fmaf_rn(mom, v.x, __fmul_rn(s, g.x)), __fmaf_rn(mom, v.y, __fmul_rn(s, g.y)),
                     __fmaf_rn(mom, v.z, __fmul_rn(s, g.z)), __fmaf_rn(mom, v.w, __fmul_rn(s, g.w)));
}
// x - lr * v
__device__ __forceinline__ float4 descend(float4 x, float lr, float4 v) {
  return make_float4(__fmaf_rn(-lr, v.x, x.x), __fmaf_rn(-lr, v.y, x.y), __fmaf_rn(-lr, v.z, x.z),
                     __fmaf_rn(-lr, v.w, x.w));
}
__device__ __forceinline__ float4 add4(float4 a, float4 b) {
  return make_float4(__fadd_rn(a.x, b.x), __fadd_rn(a.y, b.y), __fadd_rn(a.z, b.z), __fadd_rn(a.w, b.w));
}
__device__ __forceinline__ float4 scale4(float4 a, float s) {
  return make_float4(__fmul_rn(a.x, s), __fmul_rn(a.y, s), __fmul_rn(a.z, s), __fmul_rn(a.w, s));
}

// sum_j W_ij x_j over the non-zeros of row i (Alg. 2 averaging step), from the staged tiles.
__device__ __forceinline__ float4 mix_row(const float4 *xs, int tpb, int tid, const int32_t *s_col,
                                          const float *s_val, int beg, int end) {
  float4 r = make_float4(0.f, 0.f, 0.f, 0.f);
  for (int e = beg; e < end; ++e) {
    const float w = s_val[e];
    const float4 x = xs[s_col[e] * tpb + tid];
    r.x = __fmaf_rn(w, x.x, r.x);
    r.y = __fmaf_rn(w, x.y, r.y);
    r.z = __fmaf_rn(w, x.z, r.z);
    r.w = __fmaf_rn(w, x.w, r.w);
  }
  return r;
}


}  // namespace dev
}  // namespace nb
