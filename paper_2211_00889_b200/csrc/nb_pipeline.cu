// Persistent bulk-copy pipeline kernel for the fused step (sm_100a).
//
// The step is bound by HBM bandwidth, and what limits a plain load/store kernel is the number of
// bytes it can keep in flight: every outstanding load pins registers of a resident thread.  Here
// the loads are issued by ONE producer thread per CTA as 1-D bulk asynchronous copies
// (cp.async.bulk, global -> shared, completion counted on an mbarrier), so the bytes in flight are
// bounded by shared memory, not by occupancy:
//
//   * the CTA owns column tiles of T columns (persistent, tile = blockIdx.x + k * gridDim.x);
//   * per tile the producer first brings the K old model rows X[j, tile] into the X stage (the mix
//     needs every neighbour's OLD value while X is updated in place), then streams, learner by
//     learner, "items" into a ring of slots: item = momentum row V[i, tile] + up to R finished
//     gradient rows G[i, m, tile]; rows m >= n_i are never requested (the abandoned mini-batches
//     of Alg. 1 cost no bandwidth);
//   * T/4 consumer threads wait on a slot's "full" barrier, sum the rows in fp32 (m ascending),
//     apply normalisation + momentum + mix + update with the same operation sequence as the
//     direct-load kernels (bit-identical results), store x_i and v_i with 128-bit stores and hand
//     the slot back through its "empty" barrier.
//
// No CTA ever waits on another CTA.  Every mbarrier wait is bounded: after ~1 s of cycles a
// waiting thread records an error code in global memory, all roles drain and the kernel returns
// (the host reports it as an error status); nothing traps.
#include <cuda_runtime.h>

#include <cstdint>
#include <cstdlib>

#include "nb_device.cuh"
#include "nb_internal.h"
#include "nb_kernels.h"

namespace nb {
namespace {

using namespace dev;

constexpr long long kWaitLimitCycles = 2000000000ll;  // ~1 s at 1.9 GHz
constexpr long long kDrainCycles = 4000000ll;         // ~2 ms: lets copies in flight land before exit

__device__ __forceinline__ uint32_t smem_u32(const void *p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint64_t *bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(bar)), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint64_t *bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_u32(bar)), "r"(bytes) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint64_t *bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_u32(bar)) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint64_t *bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n"
      ".reg .pred p;\n"
      "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n"
      "selp.u32 %0, 1, 0, p;\n"
      "}\n"
      : "=r"(ok)
      : "r"(smem_u32(bar)), "r"(parity)
      : "memory");
  return ok != 0;
}
// Bounded wait.  Returns false when the limit passes or another thread has already reported an
// error; the caller then leaves its loop.
__device__ __forceinline__ bool mbar_wait(uint64_t *bar, uint32_t parity, int *err, int code) {
  if (mbar_try_wait(bar, parity)) return true;
  const long long t0 = clock64();
  int spins = 0;
  while (!mbar_try_wait(bar, parity)) {
    if ((++spins & 1023) == 0) {
      if (*reinterpret_cast<volatile int *>(err) != 0) return false;
      if (clock64() - t0 > kWaitLimitCycles) {
        atomicCAS(err, 0, code);
        return false;
      }
    }
  }
  return true;
}
// 1-D bulk copy global -> shared; completion is counted in bytes on `bar`.  dst, src and bytes are
// multiples of 16.
__device__ __forceinline__ void bulk_load(void *dst, const void *src, uint32_t bytes, uint64_t *bar) {
  asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(
                   smem_u32(dst)),
               "l"(src), "r"(bytes), "r"(smem_u32(bar))
               : "memory");
}
__device__ __forceinline__ void drain_and_exit_delay() {
  const long long t0 = clock64();
  while (clock64() - t0 < kDrainCycles) {
  }
}

struct PipeLayout {
  int32_t off_tab, off_xs, off_slots, slot_bytes, total;
};

__host__ __device__ inline PipeLayout pipe_layout(int K, int T, int es, int R, int n_slots, int mix_slots) {
  PipeLayout L;
  int off = (2 * n_slots + 2) * 8;
  off = (off + 127) / 128 * 128;
  L.off_tab = off;
  off += mix_slots * 8 + K * 8;
  off = (off + 127) / 128 * 128;
  L.off_xs = off;
  off += K * T * 4;
  L.off_slots = off;
  L.slot_bytes = T * 4 + R * T * es;
  L.total = off + n_slots * L.slot_bytes;
  return L;
}

// ES = bytes per gradient element (2: bf16, 4: fp32).
template <int ES, bool MEAN>
__global__ void __launch_bounds__(32 + 256, 2) nb_step_pipeline_kernel(const __grid_constant__ PipeArgs a) {
  extern __shared__ __align__(128) unsigned char smem_raw[];
  constexpr int SRC = ES == 2 ? kSrcBF16 : kSrcF32;
  const StepArgs &s = a.s;
  const int K = s.K, T = a.T, R = a.rows_per_item, NS = a.n_slots;
  const PipeLayout L = pipe_layout(K, T, ES, R, NS, s.mix_slots);
  uint64_t *full = reinterpret_cast<uint64_t *>(smem_raw);
  uint64_t *empty = full + NS;
  uint64_t *xfull = empty + NS;
  uint64_t *xempty = xfull + 1;
  int32_t *s_col = reinterpret_cast<int32_t *>(smem_raw + L.off_tab);
  float *s_val = reinterpret_cast<float *>(s_col + s.mix_slots);
  int32_t *s_beg = reinterpret_cast<int32_t *>(s_val + s.mix_slots);
  int32_t *s_end = s_beg + K;
  float *xs = reinterpret_cast<float *>(smem_raw + L.off_xs);
  unsigned char *slots = smem_raw + L.off_slots;

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int n_cons_warps = T / 128;
  if (threadIdx.x == 0) {
    for (int q = 0; q < NS; ++q) {
      mbar_init(&full[q], 1);
      mbar_init(&empty[q], n_cons_warps);
    }
    mbar_init(xfull, 1);
    mbar_init(xempty, n_cons_warps);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if constexpr (!MEAN) {
    for (int e = threadIdx.x; e < s.mix_slots; e += blockDim.x) {
      s_col[e] = s.mix->col[e];
      s_val[e] = s.mix->val[e];
    }
    for (int e = threadIdx.x; e < K; e += blockDim.x) {
      s_beg[e] = s.mix->row_beg[e];
      s_end[e] = s.mix->row_end[e];
    }
  }
  __syncthreads();

  const int64_t ldx = s.ldx;
  bool ok = true;

  if (warp == 0) {
    // ------------------------------------------------------------------ producer (one thread)
    if (lane == 0) {
      const unsigned char *G = reinterpret_cast<const unsigned char *>(s.G);
      uint32_t slot = 0, phase = 0;
      int titer = 0;
      for (int tile = blockIdx.x; ok && tile < a.n_tiles; tile += gridDim.x, ++titer) {
        const int64_t col0 = (int64_t)tile * T;
        if (!(ok = mbar_wait(xempty, (titer & 1) ^ 1, a.err, 1))) break;
        mbar_expect_tx(xfull, (uint32_t)(K * T * 4));
        for (int j = 0; j < K; ++j) bulk_load(xs + (size_t)j * T, s.X + (int64_t)j * ldx + col0, T * 4, xfull);
        for (int i = 0; ok && i < K; ++i) {
          const int n = s.n[i];
          int m0 = 0;
          do {
            const int rows = (n - m0 < R) ? (n - m0) : R;
            if (!(ok = mbar_wait(&empty[slot], phase ^ 1, a.err, 2))) break;
            unsigned char *dst = slots + (size_t)slot * L.slot_bytes;
            const uint32_t bytes = (uint32_t)(rows * T * ES + (m0 == 0 ? T * 4 : 0));
            mbar_expect_tx(&full[slot], bytes);
            if (m0 == 0) bulk_load(dst, s.V + (int64_t)i * ldx + col0, T * 4, &full[slot]);
            const unsigned char *src = G + ((int64_t)i * s.ld_k + (int64_t)m0 * s.ld_m + col0) * ES;
            for (int r = 0; r < rows; ++r)
              bulk_load(dst + T * 4 + (size_t)r * T * ES, src + (int64_t)r * s.ld_m * ES, T * ES, &full[slot]);
            if (++slot == (uint32_t)NS) { slot = 0; phase ^= 1; }
            m0 += R;
          } while (m0 < n);
        }
      }
    }
  } else {
    // ------------------------------------------------------------------ consumers (T/4 threads)
    const int ct = threadIdx.x - 32;
    const int nq = T / 4;  // float4 per staged row
    if (ct < nq) {
      const float4 *xs4 = reinterpret_cast<const float4 *>(xs);
      float4 *xs4w = reinterpret_cast<float4 *>(xs);
      const float lr = s.lr, mom = s.mom;
      uint32_t slot = 0, phase = 0;
      int titer = 0;
      for (int tile = blockIdx.x; ok && tile < a.n_tiles; tile += gridDim.x, ++titer) {
        const int64_t col0 = (int64_t)tile * T + (int64_t)ct * 4;
        float *Xc = s.X + col0;
        float *Vc = s.V + col0;
        ok = __all_sync(0xffffffffu, mbar_wait(xfull, titer & 1, a.err, 3));  // warp-uniform outcome
        if (!ok) break;
        const bool mix_first = s.order == NB_ORDER_MIX_THEN_UPDATE;
        float4 mean = make_float4(0.f, 0.f, 0.f, 0.f);
        if (MEAN && mix_first) {
          for (int j = 0; j < K; ++j) mean = add4(mean, xs4[j * nq + ct]);
          mean = scale4(mean, s.inv_K);
        }
        for (int i = 0; ok && i < K; ++i) {
          const int n = s.n[i];
          float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
          float4 v = make_float4(0.f, 0.f, 0.f, 0.f);
          int m0 = 0;
          do {
            const int rows = (n - m0 < R) ? (n - m0) : R;
            ok = __all_sync(0xffffffffu, mbar_wait(&full[slot], phase, a.err, 4));
            if (!ok) break;
            const unsigned char *src = slots + (size_t)slot * L.slot_bytes;
            if (m0 == 0) v = reinterpret_cast<const float4 *>(src)[ct];
            const unsigned char *rowp = src + T * 4 + (size_t)ct * 4 * ES;
            for (int r = 0; r < rows; ++r) {
              Raw<SRC> raw;
              if constexpr (ES == 2) raw.r = *reinterpret_cast<const uint2 *>(rowp + (size_t)r * T * ES);
              else raw.r = *reinterpret_cast<const float4 *>(rowp + (size_t)r * T * ES);
              acc = add4(acc, widen(raw));
            }
            __syncwarp();
            if (lane == 0) mbar_arrive(&empty[slot]);
            if (++slot == (uint32_t)NS) { slot = 0; phase ^= 1; }
            m0 += R;
          } while (m0 < n);
          if (!ok) break;
          const float4 vn = momentum(mom, v, s.s[i], acc);
          st4(Vc + (int64_t)i * ldx, vn);
          if (mix_first) {
            float4 xh;
            if constexpr (MEAN) xh = mean;
            else xh = mix_row(xs4, nq, ct, s_col, s_val, s_beg[i], s_end[i]);
            st4(Xc + (int64_t)i * ldx, descend(xh, lr, vn));
          } else {
            const float4 y = descend(xs4[i * nq + ct], lr, vn);
            if constexpr (MEAN) mean = add4(mean, y);
            else xs4w[i * nq + ct] = y;
          }
        }
        if (!ok) break;
        if (!mix_first) {
          if constexpr (MEAN) {
            const float4 m = scale4(mean, s.inv_K);
            for (int i = 0; i < K; ++i) st4(Xc + (int64_t)i * ldx, m);
          } else {
            for (int i = 0; i < K; ++i)
              st4(Xc + (int64_t)i * ldx, mix_row(xs4, nq, ct, s_col, s_val, s_beg[i], s_end[i]));
            // the stage was written by this thread; order those writes before the next bulk copy
            asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
          }
        }
        __syncwarp();
        if (lane == 0) mbar_arrive(xempty);
      }
    }
  }
  if (!ok) drain_and_exit_delay();
}

struct PipeTuning {
  int enabled = 1, T = 0, slots = 0, ctas_per_sm = 0, rows = 0;
  int sm_count = 0;
};

PipeTuning &tuning() {
  static PipeTuning t = [] {
    PipeTuning q;
    auto geti = [](const char *name, int dflt) {
      const char *v = std::getenv(name);
      return v ? std::atoi(v) : dflt;
    };
    q.enabled = geti("NB_PIPELINE", 1);
    q.T = geti("NB_PIPELINE_TILE", 0);
    q.slots = geti("NB_PIPELINE_SLOTS", 0);
    q.ctas_per_sm = geti("NB_PIPELINE_CTAS_PER_SM", 0);
    q.rows = geti("NB_PIPELINE_ROWS", 0);
    return q;
  }();
  return t;
}

constexpr int kSmemBudget = 227 * 1024;

}  // namespace

// Chooses tile width, slot count and CTAs per SM; returns false when the pipeline kernel does not
// apply (then the direct-load kernel runs the whole range).
bool plan_pipeline(const StepArgs &a, int es, PipePlan *plan) {
  PipeTuning &t = tuning();
  if (!t.enabled) return false;
  if (t.sm_count == 0) {
    int dev = 0;
    cudaGetDevice(&dev);
    cudaDeviceGetAttribute(&t.sm_count, cudaDevAttrMultiProcessorCount, dev);
    if (t.sm_count <= 0) t.sm_count = 148;
  }
  // bulk copies need 16-byte aligned sources and sizes
  if ((uintptr_t)a.G % 16 != 0 || (a.ld_m * es) % 16 != 0 || (a.ld_k * es) % 16 != 0) return false;
  int T = t.T ? t.T : (a.K <= 16 ? 512 : (a.K <= 32 ? 256 : 128));
  if (T % 128 != 0 || T < 128 || T > 1024) return false;
  if (a.P < T) return false;
  const int R = t.rows ? t.rows : (es == 2 ? 8 : 4);
  const int ctas = t.ctas_per_sm ? t.ctas_per_sm : 2;
  const int budget = kSmemBudget / ctas - 1024;
  int slots = t.slots;
  if (!slots) {
    const PipeLayout L0 = pipe_layout(a.K, T, es, R, 0, a.mix_slots);
    slots = (budget - L0.total - 64) / (T * 4 + R * T * es);
    if (slots > 24) slots = 24;
  }
  if (slots < 2) return false;
  const PipeLayout L = pipe_layout(a.K, T, es, R, slots, a.mix_slots);
  if (L.total > kSmemBudget) return false;
  plan->T = T;
  plan->rows_per_item = R;
  plan->n_slots = slots;
  plan->smem_bytes = L.total;
  plan->n_tiles = (int)(a.P / T);
  const int64_t max_ctas = (int64_t)ctas * t.sm_count;
  plan->grid = (int)(plan->n_tiles < max_ctas ? plan->n_tiles : max_ctas);
  return plan->n_tiles > 0;
}

cudaError_t configure_pipeline() {
  cudaError_t e;
#define NB_CFG(ES, MEAN)                                                                              \
  if ((e = cudaFuncSetAttribute(nb_step_pipeline_kernel<ES, MEAN>, cudaFuncAttributeMaxDynamicSharedMemorySize, \
                                kSmemBudget)) != cudaSuccess)                                         \
    return e;
  NB_CFG(2, true) NB_CFG(2, false) NB_CFG(4, true) NB_CFG(4, false)
#undef NB_CFG
  return cudaSuccess;
}

cudaError_t launch_step_pipeline(const StepArgs &a, int es, const PipePlan &plan, int *err_flag, cudaStream_t st) {
  PipeArgs p;
  p.s = a;
  p.T = plan.T;
  p.n_slots = plan.n_slots;
  p.rows_per_item = plan.rows_per_item;
  p.n_tiles = plan.n_tiles;
  p.err = err_flag;
  const int threads = 32 + plan.T / 4;
  if (es == 2) {
    if (a.mean_mode) nb_step_pipeline_kernel<2, true><<<plan.grid, threads, plan.smem_bytes, st>>>(p);
    else nb_step_pipeline_kernel<2, false><<<plan.grid, threads, plan.smem_bytes, st>>>(p);
  } else {
    if (a.mean_mode) nb_step_pipeline_kernel<4, true><<<plan.grid, threads, plan.smem_bytes, st>>>(p);
    else nb_step_pipeline_kernel<4, false><<<plan.grid, threads, plan.smem_bytes, st>>>(p);
  }
  return cudaGetLastError();
}

}  // namespace nb
