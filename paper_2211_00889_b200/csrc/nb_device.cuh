// Device helpers shared by the direct-load kernels and the bulk-copy pipeline kernel (internal).
// Every fp32 operation is an explicit round-to-nearest intrinsic, so all kernels that use these
// helpers produce identical bits for identical inputs.
#pragma once
#include <cuda_runtime.h>

#include <cstdint>

#include "nb_kernels.h"

namespace nb {
namespace dev {

// ---------------------------------------------------------------------------------------------
// Bounds-checked build (-DNB_DEBUG; see nb_bounds.h).  In the shipped build kDebug is false and
// every check below folds away.
// ---------------------------------------------------------------------------------------------
#ifdef NB_DEBUG
constexpr bool kDebug = true;
#else
constexpr bool kDebug = false;
#endif
// Records `code` when `ok` is false (first failure wins; err may be NULL) and returns `ok`: the
// caller skips the access it was about to make.
__device__ __forceinline__ bool dbg_check(bool ok, int *err, int code) {
  if (!ok && err) atomicCAS(err, 0, code);
  return ok;
}
// Columns [col0, col0 + cols) of `rows` rows `pitch` elements apart, `esize` bytes per element,
// starting at `base`: the first and the last row's span lie inside [lo, hi) (addresses are affine in
// the row index, so the rows in between do too).
__device__ __forceinline__ bool dbg_rows_inside(const void *base, int64_t pitch, int rows, int64_t col0, int cols,
                                                int esize, uintptr_t lo, uintptr_t hi) {
  if (rows <= 0 || cols <= 0) return true;
  const uintptr_t first = reinterpret_cast<uintptr_t>(base) + (uintptr_t)(col0 * esize);
  const uintptr_t last = first + (uintptr_t)((int64_t)(rows - 1) * pitch * esize);
  const uint64_t bytes = (uint64_t)cols * (uint64_t)esize;
  return bounds::span_inside(first, bytes, lo, hi) && bounds::span_inside(last, bytes, lo, hi);
}
// Footprint of one thread of the direct-load kernels: 4 columns at col0 of `model_rows` rows of X and
// V, of `acc_rows` rows of acc starting at row acc_row0, and (gradient stream) `nvalid` elements at
// col0 of every row (i, m).  False (and a recorded code) means: touch nothing.
__device__ __forceinline__ bool dbg_thread_footprint(const StepArgs &a, int64_t col0, int nvalid, int model_rows,
                                                     int acc_row0, int acc_rows, bool reads_g, int g_esize) {
  bool ok = dbg_check(dbg_rows_inside(a.X, a.ldx, model_rows, col0, 4, 4, a.ext.x_lo, a.ext.x_hi) &&
                          dbg_rows_inside(a.V, a.ldx, model_rows, col0, 4, 4, a.ext.v_lo, a.ext.v_hi) &&
                          dbg_rows_inside(a.acc + (int64_t)acc_row0 * a.ldx, a.ldx, acc_rows, col0, 4, 4, a.ext.acc_lo,
                                          a.ext.acc_hi),
                      a.err, bounds::kStateAddress);
  if (reads_g && !a.row_ptrs) {  // held rows are vectors of P elements of their own: col0 < P is the whole check
    const unsigned char *g = reinterpret_cast<const unsigned char *>(a.G);
    const unsigned char *last = g + ((int64_t)(a.K - 1) * a.ld_k + (int64_t)(a.M - 1) * a.ld_m) * g_esize;
    ok = dbg_check(dbg_rows_inside(g, 0, 1, col0, nvalid, g_esize, a.ext.g_lo, a.ext.g_hi) &&
                       dbg_rows_inside(last, 0, 1, col0, nvalid, g_esize, a.ext.g_lo, a.ext.g_hi),
                   a.err, bounds::kGradientAddress) && ok;
  }
  return ok;
}

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

// ---------------------------------------------------------------------------------------------
// fp32 arithmetic on pairs: sm_100 has packed add / mul / fma on two fp32 values held in one
// 64-bit register (add.rn.f32x2 and friends).  Each lane is the IEEE round-to-nearest operation,
// with subnormals kept, i.e. exactly what __fadd_rn / __fmul_rn / __fmaf_rn compute, at half the
// number of issued instructions.  A float4 loaded with one 128-bit access already sits in two
// aligned register pairs, so packing costs nothing.
// ---------------------------------------------------------------------------------------------
__device__ __forceinline__ uint64_t pack2(float x, float y) {
  uint64_t r;
  asm("mov.b64 %0, {%1, %2};" : "=l"(r) : "f"(x), "f"(y));
  return r;
}
__device__ __forceinline__ void unpack2(uint64_t v, float &x, float &y) {
  asm("mov.b64 {%0, %1}, %2;" : "=f"(x), "=f"(y) : "l"(v));
}
__device__ __forceinline__ uint64_t add2(uint64_t a, uint64_t b) {
  uint64_t r;
  asm("add.rn.f32x2 %0, %1, %2;" : "=l"(r) : "l"(a), "l"(b));
  return r;
}
__device__ __forceinline__ uint64_t mul2(uint64_t a, uint64_t b) {
  uint64_t r;
  asm("mul.rn.f32x2 %0, %1, %2;" : "=l"(r) : "l"(a), "l"(b));
  return r;
}
__device__ __forceinline__ uint64_t fma2(uint64_t a, uint64_t b, uint64_t c) {
  uint64_t r;
  asm("fma.rn.f32x2 %0, %1, %2, %3;" : "=l"(r) : "l"(a), "l"(b), "l"(c));
  return r;
}
__device__ __forceinline__ float4 from_pairs(uint64_t lo, uint64_t hi) {
  float4 r;
  unpack2(lo, r.x, r.y);
  unpack2(hi, r.z, r.w);
  return r;
}

// v' = mom * v + s * acc  (momentum; s is the per-learner normalisation / learning-rate adjustment)
__device__ __forceinline__ float4 momentum(float mom, float4 v, float s, float4 g) {
  const uint64_t m2 = pack2(mom, mom), s2 = pack2(s, s);
  return from_pairs(fma2(m2, pack2(v.x, v.y), mul2(s2, pack2(g.x, g.y))),
                    fma2(m2, pack2(v.z, v.w), mul2(s2, pack2(g.z, g.w))));
}
// x - lr * v
__device__ __forceinline__ float4 descend(float4 x, float lr, float4 v) {
  const uint64_t n2 = pack2(-lr, -lr);
  return from_pairs(fma2(n2, pack2(v.x, v.y), pack2(x.x, x.y)), fma2(n2, pack2(v.z, v.w), pack2(x.z, x.w)));
}
__device__ __forceinline__ float4 add4(float4 a, float4 b) {
  return from_pairs(add2(pack2(a.x, a.y), pack2(b.x, b.y)), add2(pack2(a.z, a.w), pack2(b.z, b.w)));
}
__device__ __forceinline__ float4 scale4(float4 a, float s) {
  const uint64_t s2 = pack2(s, s);
  return from_pairs(mul2(pack2(a.x, a.y), s2), mul2(pack2(a.z, a.w), s2));
}
// r + w * x
__device__ __forceinline__ float4 fma4(float w, float4 x, float4 r) {
  const uint64_t w2 = pack2(w, w);
  return from_pairs(fma2(w2, pack2(x.x, x.y), pack2(r.x, r.y)), fma2(w2, pack2(x.z, x.w), pack2(r.z, r.w)));
}

// sum_j W_ij x_j over the non-zeros of row i (Alg. 2 averaging step), from the staged tiles.
__device__ __forceinline__ float4 mix_row(const float4 *xs, int tpb, int tid, const int32_t *s_col,
                                          const float *s_val, int beg, int end) {
  float4 r = make_float4(0.f, 0.f, 0.f, 0.f);
  for (int e = beg; e < end; ++e) r = fma4(s_val[e], xs[s_col[e] * tpb + tid], r);
  return r;
}

}  // namespace dev
}  // namespace nb
