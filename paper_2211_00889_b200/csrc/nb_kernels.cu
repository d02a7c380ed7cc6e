// CUDA kernels (sm_100a) of the Non-blocking SGD aggregate-and-update step.
//
// Work decomposition: every thread owns 4 consecutive parameter columns for ALL K learners, every
// CTA owns a contiguous column tile.  Nothing couples columns (the method only couples learners
// and mini-batches), so CTAs never communicate, nothing waits on another CTA, and every output
// element has exactly one writer.  All traffic is 128-bit (fp32) or 64-bit (bf16) per thread and
// contiguous across a warp.  Gradient rows m >= n_i are never touched: skipping the mini-batches a
// learner had not finished when the terminal signal came is the method (Alg. 1, inner loop).
//
// fp32 arithmetic is written with explicit round-to-nearest intrinsics so that the fused kernel
// and the accumulate -> step pair perform the identical operation sequence and agree bit for bit.
#include <cuda_runtime.h>

#include <cstdint>

#include "nb_internal.h"
#include "nb_device.cuh"
#include "nb_kernels.h"

namespace nb {
namespace {

using namespace dev;

constexpr int kColsPerThread = 4;
constexpr int kChunk = 8;  // gradient rows loaded back to back before they are summed

// acc_i = sum_{m < n_i} G[i, m, cols], fp32, m ascending, starting from +0
// (Alg. 1 accumulate step; Eq. 19).  SRC = kSrcAcc reads what nb_accumulate stored instead.
template <int SRC, bool ALIGNED>
__device__ __forceinline__ float4 gather(const StepArgs &a, int i, int64_t col0, int nvalid) {
  if constexpr (SRC == kSrcAcc) {
    return __ldcs(reinterpret_cast<const float4 *>(a.acc + (int64_t)i * a.ldx + col0));
  } else {
    using E = typename ElemOf<SRC>::type;
    const E *base = reinterpret_cast<const E *>(a.G) + (int64_t)i * a.ld_k + col0;
    const void *const *rows = a.row_ptrs ? a.row_ptrs + (int64_t)i * a.M : nullptr;  // held rows: one vector per row
    const int n = a.n[i];
    float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
    for (int m0 = 0; m0 < n; m0 += kChunk) {
      Raw<SRC> r[kChunk];
#pragma unroll
      for (int u = 0; u < kChunk; ++u)
        if (m0 + u < n) {
          const E *row = rows ? reinterpret_cast<const E *>(rows[m0 + u]) + a.row_col0 + col0 : base + (int64_t)(m0 + u) * a.ld_m;
          r[u] = load_raw<ALIGNED>(row, nvalid, (Raw<SRC> *)nullptr);
        }
#pragma unroll
      for (int u = 0; u < kChunk; ++u)
        if (m0 + u < n) {
          acc = add4(acc, widen(r[u]));
        }
    }
    return acc;
  }
}

// -------------------------------------------------------------------------------------------------
// K1: masked accumulate.  grid = (column tiles, K)
// -------------------------------------------------------------------------------------------------
template <int SRC, bool ALIGNED>
__global__ void __launch_bounds__(256) nb_accumulate_kernel(const __grid_constant__ StepArgs a) {
  const int64_t col0 = ((int64_t)blockIdx.x * blockDim.x + threadIdx.x) * kColsPerThread;
  if (col0 >= a.P) return;
  const int nvalid = (a.P - col0 < 4) ? (int)(a.P - col0) : 4;
  const int i = blockIdx.y;
  if constexpr (kDebug) {
    if (!dbg_check(bounds::index_inside(i, a.K), a.err, bounds::kLearnerIndex)) return;
    if (!dbg_thread_footprint(a, col0, nvalid, 0, i, 1, true, SRC == kSrcBF16 ? 2 : 4)) return;
  }
  const float4 g = gather<SRC, ALIGNED>(a, i, col0, nvalid);
  st4(a.acc + (int64_t)i * a.ldx + col0, g);
}

// Streaming accumulate: acc_row = (first ? +0 : acc_row) + g, one mini-batch gradient at a time
// (the same sum, in the same order, as nb_accumulate_kernel builds in one go).
template <int SRC, bool ALIGNED>
__global__ void __launch_bounds__(256) nb_add_minibatch_kernel(float *acc_row, const void *g, int64_t P, int first,
                                                               uintptr_t acc_lo, uintptr_t acc_hi, int *err) {
  const int64_t col0 = ((int64_t)blockIdx.x * blockDim.x + threadIdx.x) * kColsPerThread;
  if (col0 >= P) return;
  const int nvalid = (P - col0 < 4) ? (int)(P - col0) : 4;
  using E = typename ElemOf<SRC>::type;
  if constexpr (kDebug) {  // the gradient vector is the caller's: only its length P is known, and col0 < P holds
    if (!dbg_check(dbg_rows_inside(acc_row, 0, 1, col0, 4, 4, acc_lo, acc_hi), err, bounds::kStateAddress)) return;
  }
  const float4 r = widen(load_raw<ALIGNED>(reinterpret_cast<const E *>(g) + col0, nvalid, (Raw<SRC> *)nullptr));
  float4 a = first ? make_float4(0.f, 0.f, 0.f, 0.f) : ld4(acc_row + col0);
  st4(acc_row + col0, add4(a, r));
}

// -------------------------------------------------------------------------------------------------
// K2 / K2f: normalise + momentum + mix + update (SRC = kSrcAcc), or the same fused with the masked
// accumulate (SRC = kSrcF32 / kSrcBF16).
//   MEAN = true : W = (1/K) 1 1^T; one column mean, no staging (Eq. 4-5).
//   MEAN = false: sparse W; the thread's K old models are staged in shared memory so that row i can
//                 pick its neighbours by index while X is updated in place (Alg. 2; Eq. 6).
// -------------------------------------------------------------------------------------------------
template <int SRC, bool ALIGNED, bool MEAN>
__global__ void __launch_bounds__(256) nb_step_kernel(const __grid_constant__ StepArgs a) {
  extern __shared__ float4 smem[];
  const int tid = threadIdx.x;
  const int tpb = blockDim.x;
  const int K = a.K;
  float4 *xs = smem;
  int32_t *s_col = nullptr, *s_beg = nullptr, *s_end = nullptr;
  float *s_val = nullptr;
  if constexpr (!MEAN) {
    s_col = reinterpret_cast<int32_t *>(smem + (size_t)K * tpb);
    s_val = reinterpret_cast<float *>(s_col + a.mix_slots);
    s_beg = reinterpret_cast<int32_t *>(s_val + a.mix_slots);
    s_end = s_beg + K;
    for (int e = tid; e < a.mix_slots; e += tpb) {
      s_col[e] = a.mix->col[e];
      s_val[e] = a.mix->val[e];
    }
    for (int e = tid; e < K; e += tpb) {
      s_beg[e] = a.mix->row_beg[e];
      s_end[e] = a.mix->row_end[e];
    }
    __syncthreads();
  }
  const int64_t col0 = ((int64_t)blockIdx.x * tpb + tid) * kColsPerThread;
  if (col0 >= a.P) return;
  const int nvalid = (a.P - col0 < 4) ? (int)(a.P - col0) : 4;
  if constexpr (kDebug) {
    if (!dbg_thread_footprint(a, col0, nvalid, K, 0, SRC == kSrcAcc ? K : 0, SRC != kSrcAcc, SRC == kSrcBF16 ? 2 : 4))
      return;
    if constexpr (!MEAN) {  // every column index of the staged table names a learner
      bool tab_ok = true;
      for (int i = 0; i < K; ++i) tab_ok = tab_ok && s_beg[i] >= 0 && s_beg[i] <= s_end[i] && s_end[i] <= a.mix_slots;
      for (int e = 0; e < a.mix_slots; ++e) tab_ok = tab_ok && bounds::index_inside(s_col[e], K);
      if (!dbg_check(tab_ok, a.err, bounds::kLearnerIndex)) return;
    }
  }
  float *Xc = a.X + col0;
  float *Vc = a.V + col0;
  const int64_t ldx = a.ldx;
  const float lr = a.lr, mom = a.mom;

  if (a.order == NB_ORDER_MIX_THEN_UPDATE) {
    float4 mean = make_float4(0.f, 0.f, 0.f, 0.f);
    if constexpr (MEAN) {
      for (int j = 0; j < K; ++j) mean = add4(mean, ld4(Xc + (int64_t)j * ldx));
      mean = scale4(mean, a.inv_K);
    } else {
      for (int j = 0; j < K; ++j) xs[j * tpb + tid] = ld4(Xc + (int64_t)j * ldx);
    }
    for (int i = 0; i < K; ++i) {
      const float4 v = ld4(Vc + (int64_t)i * ldx);
      const float4 g = gather<SRC, ALIGNED>(a, i, col0, nvalid);
      const float4 vn = momentum(mom, v, a.s[i], g);
      float4 xh;
      if constexpr (MEAN) xh = mean;
      else xh = mix_row(xs, tpb, tid, s_col, s_val, s_beg[i], s_end[i]);
      st4(Vc + (int64_t)i * ldx, vn);
      st4(Xc + (int64_t)i * ldx, descend(xh, lr, vn));
    }
  } else {  // NB_ORDER_UPDATE_THEN_MIX: local step first, then average (Eq. 4-6)
    float4 ysum = make_float4(0.f, 0.f, 0.f, 0.f);
    for (int j = 0; j < K; ++j) {
      const float4 x = ld4(Xc + (int64_t)j * ldx);
      const float4 v = ld4(Vc + (int64_t)j * ldx);
      const float4 g = gather<SRC, ALIGNED>(a, j, col0, nvalid);
      const float4 vn = momentum(mom, v, a.s[j], g);
      st4(Vc + (int64_t)j * ldx, vn);
      const float4 y = descend(x, lr, vn);
      if constexpr (MEAN) ysum = add4(ysum, y);
      else xs[j * tpb + tid] = y;
    }
    if constexpr (MEAN) {
      const float4 m = scale4(ysum, a.inv_K);
      for (int i = 0; i < K; ++i) st4(Xc + (int64_t)i * ldx, m);
    } else {
      for (int i = 0; i < K; ++i)
        st4(Xc + (int64_t)i * ldx, mix_row(xs, tpb, tid, s_col, s_val, s_beg[i], s_end[i]));
    }
  }
}

// -------------------------------------------------------------------------------------------------
// Non-blocking synchronous centralized step (Alg. 3): one shared model.
//   g = (1/K) sum_i s_i acc_i ; v <- mom v + g ; x <- x - lr v
// -------------------------------------------------------------------------------------------------
template <int SRC, bool ALIGNED>
__global__ void __launch_bounds__(256) nb_centralized_kernel(const __grid_constant__ StepArgs a) {
  const int64_t col0 = ((int64_t)blockIdx.x * blockDim.x + threadIdx.x) * kColsPerThread;
  if (col0 >= a.P) return;
  const int nvalid = (a.P - col0 < 4) ? (int)(a.P - col0) : 4;
  if constexpr (kDebug) {
    if (!dbg_thread_footprint(a, col0, nvalid, 1, 0, SRC == kSrcAcc ? a.K : 0, SRC != kSrcAcc, SRC == kSrcBF16 ? 2 : 4))
      return;
  }
  float4 gs = make_float4(0.f, 0.f, 0.f, 0.f);
  for (int i = 0; i < a.K; ++i) {
    const float4 g = gather<SRC, ALIGNED>(a, i, col0, nvalid);
    const float s = a.s[i];
    gs = fma4(s, g, gs);
  }
  const float4 v = ld4(a.V + col0);
  const float4 x = ld4(a.X + col0);
  const float4 vn = momentum(a.mom, v, a.inv_K, gs);
  st4(a.V + col0, vn);
  st4(a.X + col0, descend(x, a.lr, vn));
}

// -------------------------------------------------------------------------------------------------
// Short column ranges (the ragged tail after the bulk-copy kernel's tiles, the first tile of a stream
// that starts off a 16-byte boundary, problems narrower than one tile).  The kernels above give a
// thread 4 columns of ALL learners, one learner after the other: on a few hundred columns that is a
// single CTA walking K dependent rounds of memory latency (50-100 us at K = 16-64).  Here a thread
// owns 4 columns of ONE learner (blockDim = (column quads, K)): every learner's loads are in flight
// at once, the learners meet in shared memory for the mix, and the range takes a few microseconds.
// Same operations in the same order per output element: identical bits.
//   MODE 0: sparse W   1: W = (1/K) 1 1^T   2: centralized (Alg. 3; learners folded in ascending order)
// -------------------------------------------------------------------------------------------------
constexpr int kTailSparse = 0, kTailMean = 1, kTailCentralized = 2;
constexpr int kTailQuads = 16;         // column quads per CTA
constexpr int64_t kTailMaxColumns = 4096;  // ranges up to this many columns take this kernel

template <int SRC, bool ALIGNED, int MODE>
__global__ void __launch_bounds__(kTailQuads * NB_MAX_K) nb_step_tail_kernel(const __grid_constant__ StepArgs a) {
  extern __shared__ float4 smem[];
  const int QC = blockDim.x, q = threadIdx.x, i = threadIdx.y, K = a.K;
  const int tid = i * QC + q, nthreads = QC * K;
  float4 *xs = smem;  // [K][QC]: every learner's old model (or local step, or accumulated gradient) of the CTA's columns
  int32_t *s_col = nullptr, *s_beg = nullptr, *s_end = nullptr;
  float *s_val = nullptr;
  if constexpr (MODE == kTailSparse) {
    s_col = reinterpret_cast<int32_t *>(smem + (size_t)K * QC);
    s_val = reinterpret_cast<float *>(s_col + a.mix_slots);
    s_beg = reinterpret_cast<int32_t *>(s_val + a.mix_slots);
    s_end = s_beg + K;
    for (int e = tid; e < a.mix_slots; e += nthreads) {
      s_col[e] = a.mix->col[e];
      s_val[e] = a.mix->val[e];
    }
    for (int e = tid; e < K; e += nthreads) {
      s_beg[e] = a.mix->row_beg[e];
      s_end[e] = a.mix->row_end[e];
    }
  }
  const int64_t col0 = ((int64_t)blockIdx.x * QC + q) * kColsPerThread;
  bool active = col0 < a.P;
  const int nvalid = !active ? 0 : (a.P - col0 < 4) ? (int)(a.P - col0) : 4;
  if constexpr (kDebug) {
    if (active)
      active = dbg_thread_footprint(a, col0, nvalid, MODE == kTailCentralized ? 1 : K, 0, SRC == kSrcAcc ? K : 0,
                                    SRC != kSrcAcc, SRC == kSrcBF16 ? 2 : 4);
  }
  const int64_t row = (int64_t)i * a.ldx + col0;
  const float4 zero = make_float4(0.f, 0.f, 0.f, 0.f);

  if constexpr (MODE == kTailCentralized) {
    xs[tid] = active ? gather<SRC, ALIGNED>(a, i, col0, nvalid) : zero;
    __syncthreads();
    if (active && i == 0) {
      float4 gs = zero;
      for (int j = 0; j < K; ++j) gs = fma4(a.s[j], xs[j * QC + q], gs);
      const float4 v = ld4(a.V + col0);
      const float4 x = ld4(a.X + col0);
      const float4 vn = momentum(a.mom, v, a.inv_K, gs);
      st4(a.V + col0, vn);
      st4(a.X + col0, descend(x, a.lr, vn));
    }
  } else {
    const bool mix_first = a.order == NB_ORDER_MIX_THEN_UPDATE;
    float4 vn = zero;
    if (active) {
      const float4 x = ld4(a.X + row);
      const float4 v = ld4(a.V + row);
      const float4 g = gather<SRC, ALIGNED>(a, i, col0, nvalid);
      vn = momentum(a.mom, v, a.s[i], g);
      st4(a.V + row, vn);
      xs[tid] = mix_first ? x : descend(x, a.lr, vn);  // Alg. 2 mixes the old models, Eq. 4-6 the local steps
    } else {
      xs[tid] = zero;
    }
    __syncthreads();
    if (active) {
      float4 xh;
      if constexpr (MODE == kTailMean) {
        xh = zero;
        for (int j = 0; j < K; ++j) xh = add4(xh, xs[j * QC + q]);
        xh = scale4(xh, a.inv_K);
      } else {
        if constexpr (kDebug) {
          bool tab_ok = s_beg[i] >= 0 && s_beg[i] <= s_end[i] && s_end[i] <= a.mix_slots;
          for (int e = s_beg[i]; tab_ok && e < s_end[i]; ++e) tab_ok = bounds::index_inside(s_col[e], K);
          if (!dbg_check(tab_ok, a.err, bounds::kLearnerIndex)) return;
        }
        xh = mix_row(xs, QC, q, s_col, s_val, s_beg[i], s_end[i]);
      }
      st4(a.X + row, mix_first ? descend(xh, a.lr, vn) : xh);
    }
  }
}

// -------------------------------------------------------------------------------------------------
// K3: MATCHA activation + W builder.  One Bernoulli draw per matching per step from the counter
// generator; row i of W = I - alpha * sum_active L_j is written as (diagonal, active partners).
// -------------------------------------------------------------------------------------------------
__global__ void nb_matcha_build_kernel(const __grid_constant__ MatchaArgs a) {
  const int i = threadIdx.x;
  const uint32_t bits = matcha_bits(a.seed, a.step, a.n_matchings, a.thr);
  const int stride = 1 + a.n_matchings;
  if (i < a.K) {
    const int e = i * stride;
    int cnt = 0;
    for (int c = 0; c < a.n_matchings; ++c) {
      const int v = a.partner[c * a.K + i];
      if (((bits >> c) & 1u) && v >= 0) {
        ++cnt;
        if constexpr (kDebug) {
          if (!dbg_check(bounds::index_inside(e + cnt, NB_MAX_NNZ) && bounds::index_inside(v, a.K), a.err,
                         bounds::kLearnerIndex)) {
            --cnt;
            continue;
          }
        }
        a.mix->col[e + cnt] = v;
        a.mix->val[e + cnt] = a.alpha;
      }
    }
    a.mix->col[e] = i;
    a.mix->val[e] = __fsub_rn(1.0f, __fmul_rn(a.alpha, (float)cnt));
    a.mix->row_beg[i] = e;
    a.mix->row_end[i] = e + cnt + 1;
  }
  if (i == 0) {
    a.mix->bits = bits;
    a.mix->n_slots = a.K * stride;
  }
}

// Average of the learners' models (Alg. 1 / Alg. 2 "Output"), ascending learner order.
__global__ void __launch_bounds__(256) nb_mean_kernel(const float *X, int64_t ldx, int K, int64_t P, float *out,
                                                      uintptr_t x_lo, uintptr_t x_hi, int *err) {
  const int64_t p = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (p >= P) return;
  if constexpr (kDebug) {
    if (!dbg_check(dbg_rows_inside(X, ldx, K, p, 1, 4, x_lo, x_hi), err, bounds::kStateAddress)) return;
  }
  float s = 0.f;
  for (int i = 0; i < K; ++i) s = __fadd_rn(s, X[(int64_t)i * ldx + p]);
  out[p] = __fdiv_rn(s, (float)K);
}

size_t step_smem_bytes(const StepArgs &a, int tpb) {
  if (a.mean_mode) return 0;
  return (size_t)a.K * tpb * sizeof(float4) + (size_t)a.mix_slots * 8 + (size_t)a.K * 8;
}

template <typename F> cudaError_t allow_big_smem(F *f) {
  return cudaFuncSetAttribute(f, cudaFuncAttributeMaxDynamicSharedMemorySize, 227 * 1024);
}

template <int SRC, bool ALIGNED>
cudaError_t launch_step_t(const StepArgs &a, cudaStream_t st) {
  const int tpb = step_threads_per_block(a);
  const int64_t per_block = (int64_t)tpb * kColsPerThread;
  const unsigned grid = (unsigned)((a.P + per_block - 1) / per_block);
  if (a.mean_mode)
    nb_step_kernel<SRC, ALIGNED, true><<<grid, tpb, 0, st>>>(a);
  else
    nb_step_kernel<SRC, ALIGNED, false><<<grid, tpb, step_smem_bytes(a, tpb), st>>>(a);
  return cudaGetLastError();
}

}  // namespace

int step_threads_per_block(const StepArgs &a) {
  if (a.mean_mode) return 256;
  // staged tile = K * threads * 16 B; keep several CTAs resident per SM
  if (a.K <= 17) return 256;
  if (a.K <= 35) return 128;
  return 64;
}

cudaError_t configure_kernels() {
  cudaError_t e;
#define NB_CFG(SRC, AL) \
  if ((e = allow_big_smem(nb_step_kernel<SRC, AL, false>)) != cudaSuccess) return e;
  NB_CFG(kSrcF32, true) NB_CFG(kSrcF32, false) NB_CFG(kSrcBF16, true) NB_CFG(kSrcBF16, false)
  NB_CFG(kSrcAcc, true)
#undef NB_CFG
  return configure_pipeline();
}

namespace {
// The accumulator presented as a one-row fp32 gradient stream (0 + acc == acc bit for bit: acc is never -0).
StepArgs acc_as_stream(const StepArgs &a) {
  StepArgs p = a;
  p.G = a.acc;
  p.ld_m = a.ldx;
  p.ld_k = a.ldx;
  p.M = 1;
  for (int i = 0; i < a.K; ++i) p.n[i] = 1;
  p.ext.g_lo = a.ext.acc_lo;
  p.ext.g_hi = a.ext.acc_hi;
  return p;
}
}  // namespace

StepArgs column_range(const StepArgs &a, int64_t c0, int64_t cols, int es) {
  StepArgs r = a;
  r.row_col0 += c0;  // held rows: the table stays as it is, the kernels add the range's first column
  r.X += c0;
  r.V += c0;
  r.acc += c0;
  if (a.G) r.G = reinterpret_cast<const unsigned char *>(a.G) + c0 * es;
  r.P = cols;
  return r;
}

namespace {

cudaError_t launch_accumulate_direct(const StepArgs &a, int src, cudaStream_t st) {
  const int tpb = 256;
  const int64_t per_block = (int64_t)tpb * kColsPerThread;
  dim3 grid((unsigned)((a.P + per_block - 1) / per_block), (unsigned)a.K);
  if (src == kSrcF32) {
    if (a.g_aligned) nb_accumulate_kernel<kSrcF32, true><<<grid, tpb, 0, st>>>(a);
    else nb_accumulate_kernel<kSrcF32, false><<<grid, tpb, 0, st>>>(a);
  } else {
    if (a.g_aligned) nb_accumulate_kernel<kSrcBF16, true><<<grid, tpb, 0, st>>>(a);
    else nb_accumulate_kernel<kSrcBF16, false><<<grid, tpb, 0, st>>>(a);
  }
  return cudaGetLastError();
}

template <int SRC, bool ALIGNED>
cudaError_t launch_tail_t(const StepArgs &a, int mode, cudaStream_t st) {
  const dim3 block(kTailQuads, a.K);
  const unsigned grid = (unsigned)((a.P + kTailQuads * kColsPerThread - 1) / (kTailQuads * kColsPerThread));
  size_t smem = (size_t)a.K * kTailQuads * sizeof(float4);
  if (mode == kTailSparse) {
    smem += (size_t)a.mix_slots * 8 + (size_t)a.K * 8;
    nb_step_tail_kernel<SRC, ALIGNED, kTailSparse><<<grid, block, smem, st>>>(a);
  } else if (mode == kTailMean) {
    nb_step_tail_kernel<SRC, ALIGNED, kTailMean><<<grid, block, smem, st>>>(a);
  } else {
    nb_step_tail_kernel<SRC, ALIGNED, kTailCentralized><<<grid, block, smem, st>>>(a);
  }
  return cudaGetLastError();
}
cudaError_t launch_tail(const StepArgs &a, int src, int mode, cudaStream_t st) {
  if (src == kSrcAcc) return launch_tail_t<kSrcAcc, true>(a, mode, st);
  if (src == kSrcF32) return a.g_aligned ? launch_tail_t<kSrcF32, true>(a, mode, st) : launch_tail_t<kSrcF32, false>(a, mode, st);
  return a.g_aligned ? launch_tail_t<kSrcBF16, true>(a, mode, st) : launch_tail_t<kSrcBF16, false>(a, mode, st);
}

cudaError_t launch_step_direct(const StepArgs &a, int src, cudaStream_t st) {
  if (src == kSrcAcc) return launch_step_t<kSrcAcc, true>(a, st);
  if (src == kSrcF32) return a.g_aligned ? launch_step_t<kSrcF32, true>(a, st) : launch_step_t<kSrcF32, false>(a, st);
  return a.g_aligned ? launch_step_t<kSrcBF16, true>(a, st) : launch_step_t<kSrcBF16, false>(a, st);
}

cudaError_t launch_centralized_direct(const StepArgs &a, int src, cudaStream_t st) {
  const int tpb = 256;
  const int64_t per_block = (int64_t)tpb * kColsPerThread;
  const unsigned grid = (unsigned)((a.P + per_block - 1) / per_block);
  if (src == kSrcAcc) nb_centralized_kernel<kSrcAcc, true><<<grid, tpb, 0, st>>>(a);
  else if (src == kSrcF32) {
    if (a.g_aligned) nb_centralized_kernel<kSrcF32, true><<<grid, tpb, 0, st>>>(a);
    else nb_centralized_kernel<kSrcF32, false><<<grid, tpb, 0, st>>>(a);
  } else {
    if (a.g_aligned) nb_centralized_kernel<kSrcBF16, true><<<grid, tpb, 0, st>>>(a);
    else nb_centralized_kernel<kSrcBF16, false><<<grid, tpb, 0, st>>>(a);
  }
  return cudaGetLastError();
}

// Covers all P columns of `a`: the bulk-copy kernel on the tiles `plan` names (when there is a plan),
// the direct-load kernel on the columns before and after them.  `p` is `a` as the bulk-copy kernel
// sees it (the unfused step presents the accumulator as a one-row gradient stream).
// pipe(range, plan) returns cudaErrorNotSupported when the driver refused a tensor map for this
// memory: nothing was launched then, and the direct-load kernel takes the whole range.
template <typename Pipe, typename Direct>
cudaError_t cover_columns(const StepArgs &a, const StepArgs &p, int es, const PipePlan *plan, int *launches,
                          PipePlan *used, Pipe pipe, Direct direct) {
  *launches = 0;
  if (used) *used = PipePlan{};
  int64_t lo = 0, hi = 0;  // columns [lo, hi) are done by the bulk-copy kernel
  if (plan) {
    const int64_t c0 = plan->head, cols = (int64_t)plan->n_tiles * plan->T;
    cudaError_t e = pipe(column_range(p, c0, cols, es), *plan);
    if (e == cudaSuccess) {
      ++*launches;
      if (used) *used = *plan;
      lo = c0;
      hi = c0 + cols;
    } else if (e != cudaErrorNotSupported) {
      return e;
    }
  }
  if (lo > 0) {  // the first tile of a stream that does not start on a 16-byte boundary
    cudaError_t e = direct(column_range(a, 0, lo, es));
    if (e != cudaSuccess) return e;
    ++*launches;
  }
  if (hi < a.P) {  // ragged tail (or everything, when the bulk-copy kernel does not apply)
    cudaError_t e = direct(column_range(a, hi, a.P - hi, es));
    if (e != cudaSuccess) return e;
    ++*launches;
  }
  return cudaSuccess;
}

}  // namespace

cudaError_t launch_accumulate_direct_only(const StepArgs &a, int src, cudaStream_t st) {
  return launch_accumulate_direct(a, src, st);
}
cudaError_t launch_step_direct_only(const StepArgs &a, int src, cudaStream_t st) { return launch_step_direct(a, src, st); }

cudaError_t launch_accumulate(const StepArgs &a, int src, bool pipeline, int *err_flag, int *launches, cudaStream_t st) {
  const int es = src == kSrcBF16 ? 2 : 4;
  PipePlan plan;
  const bool planned = pipeline && plan_stream(a, es, false, &plan);
  return cover_columns(
      a, a, es, planned ? &plan : nullptr, launches, nullptr,
      [&](const StepArgs &r, const PipePlan &pl) { return launch_stream_pipeline(r, es, false, pl, err_flag, st); },
      [&](const StepArgs &r) { return launch_accumulate_direct(r, src, st); });
}

cudaError_t launch_step(const StepArgs &a, int src, bool pipeline, int *err_flag, int *launches, PipePlan *used,
                        cudaStream_t st) {
  const int es = src == kSrcBF16 ? 2 : 4;
  const StepArgs p = src == kSrcAcc ? acc_as_stream(a) : a;
  PipePlan plan;
  const bool planned = pipeline && plan_pipeline(p, es, &plan);
  return cover_columns(
      a, p, es, planned ? &plan : nullptr, launches, used,
      [&](const StepArgs &r, const PipePlan &pl) { return launch_step_pipeline(r, es, pl, err_flag, st); },
      [&](const StepArgs &r) {
        if (pipeline && r.P <= kTailMaxColumns) return launch_tail(r, src, r.mean_mode ? kTailMean : kTailSparse, st);
        return launch_step_direct(r, src, st);
      });
}

cudaError_t launch_centralized(const StepArgs &a, int src, bool pipeline, int *err_flag, int *launches, PipePlan *used,
                               cudaStream_t st) {
  const int es = src == kSrcBF16 ? 2 : 4;
  const StepArgs p = src == kSrcAcc ? acc_as_stream(a) : a;
  PipePlan plan;
  const bool planned = pipeline && plan_stream(p, es, true, &plan);
  return cover_columns(
      a, p, es, planned ? &plan : nullptr, launches, used,
      [&](const StepArgs &r, const PipePlan &pl) { return launch_stream_pipeline(r, es, true, pl, err_flag, st); },
      [&](const StepArgs &r) {
        if (pipeline && r.P <= kTailMaxColumns) return launch_tail(r, src, kTailCentralized, st);
        return launch_centralized_direct(r, src, st);
      });
}

cudaError_t launch_add_minibatch(float *acc_row, const void *g, int src, bool aligned, int64_t P, bool first,
                                 const bounds::Extents &ext, int *err, cudaStream_t st) {
  const unsigned grid = (unsigned)((P + 1023) / 1024);
#define NB_ADD(SRC, AL) \
  nb_add_minibatch_kernel<SRC, AL><<<grid, 256, 0, st>>>(acc_row, g, P, first, ext.acc_lo, ext.acc_hi, err)
  if (src == kSrcF32) {
    if (aligned) NB_ADD(kSrcF32, true);
    else NB_ADD(kSrcF32, false);
  } else {
    if (aligned) NB_ADD(kSrcBF16, true);
    else NB_ADD(kSrcBF16, false);
  }
#undef NB_ADD
  return cudaGetLastError();
}

cudaError_t launch_matcha_build(const MatchaArgs &a, cudaStream_t st) {
  nb_matcha_build_kernel<<<1, NB_MAX_K, 0, st>>>(a);
  return cudaGetLastError();
}

cudaError_t launch_mean(const float *X, int64_t ldx, int K, int64_t P, float *out, const bounds::Extents &ext, int *err,
                        cudaStream_t st) {
  const unsigned grid = (unsigned)((P + 255) / 256);
  nb_mean_kernel<<<grid, 256, 0, st>>>(X, ldx, K, P, out, ext.x_lo, ext.x_hi, err);
  return cudaGetLastError();
}

}  // namespace nb
