// Persistent bulk-copy pipeline kernel for the fused step (sm_100a).
//
// The step is bound by HBM bandwidth, and what limits a plain load/store kernel is the number of
// bytes it can keep in flight: every outstanding load pins registers of a resident thread.  Here
// the loads are tiled bulk asynchronous copies (TMA: cp.async.bulk.tensor through tensor maps,
// global -> shared, completion counted in bytes on an mbarrier) issued by a handful of producer
// threads, so the bytes in flight are bounded by shared memory, not by occupancy, and one
// instruction moves a whole box of rows (with one instruction per row the producers are
// issue-bound):
//
//   * the CTA owns column tiles of T columns (persistent, tile = blockIdx.x + k * gridDim.x);
//   * an X producer thread brings the K old model rows X[:, tile] into the X stage with one box copy
//     per tile (the mix needs every neighbour's OLD value while X is updated in place).  The stage
//     has two buffers, so tile t+1's models load while tile t is consumed; one buffer where two do
//     not fit (K > 32: the ring keeps the copies going meanwhile); three for the update-then-mix
//     order (Eq. 4-6), whose averaging pass then runs one tile late.  In that order on one buffer
//     (template parameter XR) there is no such box at all: x_i travels in learner i's ring item and
//     the buffer only holds the locally updated models between the two passes of a tile;
//   * the consumers form NG groups of T/4 threads; group g owns the learners i = g, g+NG, ...
//     (their updates are independent once the old models are staged) and a PRIVATE ring of slots;
//     its own producer thread streams that group's "items" into the ring: item = momentum row
//     V[i, tile] (one box) + up to R finished gradient rows G[i, m0:m0+r, tile] (one box of exactly
//     r rows, from the tensor map whose box height is r); rows m >= n_i are never requested (the
//     abandoned mini-batches of Alg. 1 cost no bandwidth).  A slot is always filled for and released
//     by the same group, in order: that is what makes waiting on a phase parity unambiguous, and a
//     slow group never holds up another group's copies;
//   * a consumer thread owns 4 columns: it waits on the slot's "full" barrier, sums the rows in
//     fp32 (m ascending), applies normalisation + momentum + mix + update with the same operation
//     sequence as the direct-load kernels (bit-identical results), stores x_i and v_i with 128-bit
//     stores and hands the slot back through its "empty" barrier.
//
// Gradient rows whose byte addresses are not multiples of 16 (odd row lengths, a stream that starts
// at an odd element) cannot be described by a tensor map.  They take the same path with one change
// (template parameter GM = kGRows): the producer WARP issues one plain 1-D bulk copy per finished row,
// lane r for row m0 + r, that fetches the 16-byte aligned superset of the row's tile segment (start
// rounded down, T*ES + 16 bytes), and the consumers read each row at its own byte shift from shared
// memory, element by element.  The momentum and model rows are library-owned, 2 KB-pitched and keep
// their box copies.  Same additions in the same order: identical bits.
//
// A third form (GM = kGPtrs) serves the streaming entry points in their "hold" mode: the finished
// mini-batch gradients are separate 16-byte aligned vectors named by a table of row pointers; lane r
// copies exactly its row's tile segment with one 1-D bulk copy and the consumers read it aligned.
//
// No CTA ever waits on another CTA.  Every mbarrier wait is bounded: after ~1 s of cycles a
// waiting thread records an error code in global memory, all roles drain and the kernel returns
// (the host reports it as an error status); nothing traps.
#include <cuda.h>
#include <cuda_runtime.h>

#include <cstdint>
#include <cstdlib>
#include <cstring>

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
// The same operations on a 32-bit shared-memory address (what the instructions take): the hot loops
// keep barrier and slot addresses as 32-bit integers instead of re-deriving them from generic pointers.
__device__ __forceinline__ void mbar_arrive_a(uint32_t bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint64_t *bar) { mbar_arrive_a(smem_u32(bar)); }
// One poll of the barrier's phase.  The thread may be suspended by the hardware for up to
// kSuspendHintNs while the phase is incomplete (it is woken when the phase completes), which keeps
// waiting warps from burning issue slots on polling.
constexpr uint32_t kSuspendHintNs = 2000;
__device__ __forceinline__ bool mbar_try_wait_a(uint32_t bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n"
      ".reg .pred p;\n"
      "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2, %3;\n"
      "selp.u32 %0, 1, 0, p;\n"
      "}\n"
      : "=r"(ok)
      : "r"(bar), "r"(parity), "r"(kSuspendHintNs)
      : "memory");
  return ok != 0;
}
// Bounded wait.  Returns false when the limit passes or another thread has already reported an
// error; the caller then leaves its loop.
__device__ __forceinline__ bool mbar_wait_a(uint32_t bar, uint32_t parity, int *err, int code,
                                            long long limit = kWaitLimitCycles) {
  if (mbar_try_wait_a(bar, parity)) return true;
  const long long t0 = clock64();
  int spins = 0;
  while (!mbar_try_wait_a(bar, parity)) {
    if ((++spins & 63) == 0) {
      if (*reinterpret_cast<volatile int *>(err) != 0) return false;
      if (clock64() - t0 > limit) {
        atomicCAS(err, 0, code);
        return false;
      }
    }
  }
  return true;
}
__device__ __forceinline__ bool mbar_wait(uint64_t *bar, uint32_t parity, int *err, int code,
                                          long long limit = kWaitLimitCycles) {
  return mbar_wait_a(smem_u32(bar), parity, err, code, limit);
}
// Tiled bulk copies global -> shared through a tensor map; completion is counted in bytes on `bar`.
// Coordinates are in map elements, innermost first; c0 * element size is a multiple of 16 bytes.
__device__ __forceinline__ void tma_load_2d(void *dst, const CUtensorMap *map, int c0, int c1, uint64_t *bar) {
  asm volatile(
      "cp.async.bulk.tensor.2d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];" ::"r"(
          smem_u32(dst)),
      "l"(reinterpret_cast<uint64_t>(map)), "r"(c0), "r"(c1), "r"(smem_u32(bar))
      : "memory");
}
__device__ __forceinline__ void tma_load_3d(void *dst, const CUtensorMap *map, int c0, int c1, int c2, uint64_t *bar) {
  asm volatile(
      "cp.async.bulk.tensor.3d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3, %4}], [%5];" ::"r"(
          smem_u32(dst)),
      "l"(reinterpret_cast<uint64_t>(map)), "r"(c0), "r"(c1), "r"(c2), "r"(smem_u32(bar))
      : "memory");
}
// Plain 1-D bulk copy global -> shared: both addresses 16-byte aligned, size a multiple of 16.
__device__ __forceinline__ void bulk_load_1d(void *dst, const void *src, uint32_t bytes, uint64_t *bar) {
  asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(
                   smem_u32(dst)),
               "l"(reinterpret_cast<uint64_t>(src)), "r"(bytes), "r"(smem_u32(bar))
               : "memory");
}
__device__ __forceinline__ void drain_and_exit_delay() {
  const long long t0 = clock64();
  while (clock64() - t0 < kDrainCycles) {
  }
}

constexpr int kSmemBudget = 227 * 1024;
constexpr int kMaxRowsPerItem = 8;
// How the gradient rows of a ring item travel (template parameter GM):
constexpr int kGBox = 0;   // 16-byte aligned strided stream: one tensor-map box of exactly r rows, issued by lane 0
constexpr int kGRows = 1;  // strided stream whose rows are not 16-byte aligned: per row the aligned superset, read at a byte shift
constexpr int kGPtrs = 2;  // a table of row pointers (16-byte aligned vectors): per row exactly its tile segment
constexpr int kMaxGroups = 4;
constexpr int kBoxInner = 256;  // a box is at most 256 elements wide: rows are described in units of T*es/256 bytes

struct PipeArgs {
  StepArgs s;
  int32_t T;              // columns per tile (multiple of 128)
  int32_t n_slots;        // ring slots
  int32_t rows_per_item;  // gradient rows per ring item (R)
  int32_t n_tiles;        // full tiles covered by the kernel
  int32_t n_groups;       // consumer groups (each T/4 threads)
  int32_t x_stages;       // buffers of the X stage: 1, 2 or 3
  int *err;               // device word: 0, or the code of the wait that ran out
  // GA = false only: the gradient stream as bytes; (address & 15) of G and of the two pitches
  const unsigned char *g_base;
  int64_t g_ld_m_bytes, g_ld_k_bytes;
  int32_t g_mis0, g_mis_m, g_mis_k;
  alignas(64) CUtensorMap xmap;                   // X as [K, units]: box = (256, K)
  alignas(64) CUtensorMap vmap;                   // V as [K, units]: box = (256, 1)
  alignas(64) CUtensorMap xrmap;                  // X as [K, units]: box = (256, 1) (template parameter XR only)
  alignas(64) CUtensorMap gmap[kMaxRowsPerItem];  // G as [K, M, units]: box = (256, r, 1), r = 1..R
};

// Four consecutive columns of one staged gradient row, widened to fp32.  GA: p is 16-byte (fp32) or
// 8-byte (bf16) aligned; otherwise p is only element-aligned and the elements are read one by one.
template <int SRC, bool GA>
__device__ __forceinline__ float4 ld_row4(const unsigned char *p) {
  if constexpr (GA) {
    Raw<SRC> raw;
    if constexpr (SRC == kSrcBF16) raw.r = *reinterpret_cast<const uint2 *>(p);
    else raw.r = *reinterpret_cast<const float4 *>(p);
    return widen(raw);
  } else if constexpr (SRC == kSrcBF16) {
    const uint16_t *e = reinterpret_cast<const uint16_t *>(p);
    return make_float4(__uint_as_float((uint32_t)e[0] << 16), __uint_as_float((uint32_t)e[1] << 16),
                       __uint_as_float((uint32_t)e[2] << 16), __uint_as_float((uint32_t)e[3] << 16));
  } else {
    const float *e = reinterpret_cast<const float *>(p);
    return make_float4(e[0], e[1], e[2], e[3]);
  }
}

// acc += row_0 + row_1 + ... (ascending, one add at a time) over N rows `stride` bytes apart; all
// loads are issued before the first add.  Same sequence of fp32 additions as a plain loop.
// GA = false: row r sits at its own byte shift (s0 + r * mis_m) & 15 inside its staged superset.
template <int SRC, bool GA, int N>
__device__ __forceinline__ float4 sum_rows_n(float4 acc, const unsigned char *rowp, int stride, int s0, int mis_m) {
  float4 g[N];
#pragma unroll
  for (int r = 0; r < N; ++r) {
    const int shift = GA ? 0 : ((s0 + r * mis_m) & 15);
    g[r] = ld_row4<SRC, GA>(rowp + r * stride + shift);
  }
#pragma unroll
  for (int r = 0; r < N; ++r) acc = add4(acc, g[r]);
  return acc;
}
template <int SRC, bool GA>
__device__ __forceinline__ float4 sum_rows(float4 acc, const unsigned char *rowp, int stride, int rows, int s0,
                                           int mis_m) {
  switch (rows) {
    case 0: return acc;
    case 1: return sum_rows_n<SRC, GA, 1>(acc, rowp, stride, s0, mis_m);
    case 2: return sum_rows_n<SRC, GA, 2>(acc, rowp, stride, s0, mis_m);
    case 3: return sum_rows_n<SRC, GA, 3>(acc, rowp, stride, s0, mis_m);
    case 4: return sum_rows_n<SRC, GA, 4>(acc, rowp, stride, s0, mis_m);
    case 5: return sum_rows_n<SRC, GA, 5>(acc, rowp, stride, s0, mis_m);
    case 6: return sum_rows_n<SRC, GA, 6>(acc, rowp, stride, s0, mis_m);
    case 7: return sum_rows_n<SRC, GA, 7>(acc, rowp, stride, s0, mis_m);
    default: return sum_rows_n<SRC, GA, 8>(acc, rowp, stride, s0, mis_m);
  }
}

// The same on a 32-bit shared-memory address.
template <int SRC, bool GA>
__device__ __forceinline__ float4 lds_row4(uint32_t a) {
  if constexpr (GA && SRC == kSrcBF16) {
    Raw<kSrcBF16> raw;
    asm volatile("ld.shared.v2.b32 {%0, %1}, [%2];" : "=r"(raw.r.x), "=r"(raw.r.y) : "r"(a));
    return widen(raw);
  } else if constexpr (GA) {
    float4 v;
    asm volatile("ld.shared.v4.f32 {%0, %1, %2, %3}, [%4];" : "=f"(v.x), "=f"(v.y), "=f"(v.z), "=f"(v.w) : "r"(a));
    return v;
  } else if constexpr (SRC == kSrcBF16) {
    uint32_t e[4];
#pragma unroll
    for (int q = 0; q < 4; ++q) asm volatile("ld.shared.u16 %0, [%1];" : "=r"(e[q]) : "r"(a + 2 * q));
    return make_float4(__uint_as_float(e[0] << 16), __uint_as_float(e[1] << 16), __uint_as_float(e[2] << 16),
                       __uint_as_float(e[3] << 16));
  } else {
    float4 v;
    asm volatile("ld.shared.f32 %0, [%1];" : "=f"(v.x) : "r"(a));
    asm volatile("ld.shared.f32 %0, [%1];" : "=f"(v.y) : "r"(a + 4));
    asm volatile("ld.shared.f32 %0, [%1];" : "=f"(v.z) : "r"(a + 8));
    asm volatile("ld.shared.f32 %0, [%1];" : "=f"(v.w) : "r"(a + 12));
    return v;
  }
}
template <int SRC, bool GA, int N>
__device__ __forceinline__ float4 sum_rows_n_a(float4 acc, uint32_t row, int stride, int s0, int mis_m) {
  float4 g[N];
#pragma unroll
  for (int r = 0; r < N; ++r) {
    const int shift = GA ? 0 : ((s0 + r * mis_m) & 15);
    g[r] = lds_row4<SRC, GA>(row + r * stride + shift);
  }
#pragma unroll
  for (int r = 0; r < N; ++r) acc = add4(acc, g[r]);
  return acc;
}
template <int SRC, bool GA>
__device__ __forceinline__ float4 sum_rows_a(float4 acc, uint32_t row, int stride, int rows, int s0, int mis_m) {
  switch (rows) {
    case 0: return acc;
    case 1: return sum_rows_n_a<SRC, GA, 1>(acc, row, stride, s0, mis_m);
    case 2: return sum_rows_n_a<SRC, GA, 2>(acc, row, stride, s0, mis_m);
    case 3: return sum_rows_n_a<SRC, GA, 3>(acc, row, stride, s0, mis_m);
    case 4: return sum_rows_n_a<SRC, GA, 4>(acc, row, stride, s0, mis_m);
    case 5: return sum_rows_n_a<SRC, GA, 5>(acc, row, stride, s0, mis_m);
    case 6: return sum_rows_n_a<SRC, GA, 6>(acc, row, stride, s0, mis_m);
    case 7: return sum_rows_n_a<SRC, GA, 7>(acc, row, stride, s0, mis_m);
    default: return sum_rows_n_a<SRC, GA, 8>(acc, row, stride, s0, mis_m);
  }
}

// Bounds-checked build: everything the producer is about to use for one ring item - the slot, the
// copy coordinates, and (per-row copies) the source span of this lane's row - is in range.
template <int ES, int GM>
__device__ __forceinline__ bool dbg_item_ok(const PipeArgs &a, int T, int tile, int i, int m0, int rows, int lane,
                                            uint32_t sl, int NS, int off_slots, int slot_bytes, int total) {
  bool ok = dbg_check(sl < (uint32_t)NS && off_slots + (int)(sl + 1) * slot_bytes <= total, a.err, bounds::kRingSlot);
  ok = dbg_check(bounds::index_inside(tile, a.n_tiles) && bounds::index_inside(i, a.s.K) && m0 >= 0 && rows >= 0 &&
                     m0 + rows <= a.s.M && rows <= kMaxRowsPerItem,
                 a.err, bounds::kTileCoordinate) && ok;
  if constexpr (GM == kGRows) {
    if (lane < rows) {
      const unsigned char *src = a.g_base + (int64_t)i * a.g_ld_k_bytes + (int64_t)(m0 + lane) * a.g_ld_m_bytes +
                                 (int64_t)tile * (T * ES);
      src -= reinterpret_cast<uintptr_t>(src) & 15;
      ok = dbg_check(bounds::span_inside(reinterpret_cast<uintptr_t>(src), (uint64_t)(T * ES + 16), a.s.ext.g_lo,
                                         a.s.ext.g_hi),
                     a.err, bounds::kGradientAddress) && ok;
    }
  } else if constexpr (GM == kGPtrs) {
    if (lane < rows) {  // the row is a vector of P elements of its own: the tile segment lies inside it, 16-byte aligned
      const uintptr_t row = reinterpret_cast<uintptr_t>(a.s.row_ptrs[(int64_t)i * a.s.M + m0 + lane]);
      ok = dbg_check(row != 0 && row % 16 == 0 && (a.s.row_col0 * ES) % 16 == 0 && (int64_t)(tile + 1) * T <= a.s.P, a.err,
                     bounds::kGradientAddress) && ok;
    }
  }
  return ok;
}

// Producer side of one ring item's gradient rows.  kGBox: lane 0 issues one box of exactly `rows` rows.
// kGRows: lanes 0..rows-1 each fetch the aligned superset of one row's tile segment.  kGPtrs: lanes
// 0..rows-1 each fetch exactly one row's tile segment from the vector the row-pointer table names.
template <int ES, int GM>
__device__ __forceinline__ void issue_rows(const PipeArgs &a, unsigned char *dst, int T, int tile, int i, int m0,
                                           int rows, int lane, uint64_t *bar) {
  if constexpr (GM == kGBox) {
    if (rows > 0) tma_load_3d(dst, &a.gmap[rows - 1], tile * kBoxInner, m0, i, bar);
  } else if constexpr (GM == kGRows) {
    if (lane < rows) {
      const unsigned char *src = a.g_base + (int64_t)i * a.g_ld_k_bytes + (int64_t)(m0 + lane) * a.g_ld_m_bytes +
                                 (int64_t)tile * (T * ES);
      src -= reinterpret_cast<uintptr_t>(src) & 15;
      bulk_load_1d(dst + lane * (T * ES + 16), src, (uint32_t)(T * ES + 16), bar);
    }
  } else {
    if (lane < rows) {
      const unsigned char *src = reinterpret_cast<const unsigned char *>(a.s.row_ptrs[(int64_t)i * a.s.M + m0 + lane]) +
                                 (a.s.row_col0 + (int64_t)tile * T) * ES;
      bulk_load_1d(dst + lane * (T * ES), src, (uint32_t)(T * ES), bar);
    }
  }
}

// Bytes of one ring slot: the momentum row (step kernel only) followed by R staged gradient rows,
// rounded up to 128 bytes, the alignment a tiled bulk copy needs for its shared-memory destination.
__host__ __device__ inline int slot_bytes_of(int v_bytes, int T, int es, int R, int row_pad) {
  return (v_bytes + R * (T * es + row_pad) + 127) / 128 * 128;
}

struct PipeLayout {
  int32_t off_tab, off_xs, off_slots, slot_bytes, total;
};

// row_pad: 0 for box copies, 16 when every row is staged as its 16-byte aligned superset.
constexpr int kMaxXStages = 3;
// state_rows: fp32 state rows at the head of a slot (1: the momentum row; 2: momentum row and old model row).
__host__ __device__ inline PipeLayout pipe_layout(int K, int T, int es, int R, int n_slots, int mix_slots, int row_pad,
                                                  int x_stages, int state_rows = 1) {
  PipeLayout L;
  int off = (2 * n_slots + 3 * kMaxXStages) * 8;
  off = (off + 127) / 128 * 128;
  L.off_tab = off;
  off += mix_slots * 8 + K * 8;
  off = (off + 127) / 128 * 128;
  L.off_xs = off;
  off += x_stages * K * T * 4;  // two buffers: tile t+1's models load while tile t is consumed (see the kernel)
  L.off_slots = off;
  L.slot_bytes = slot_bytes_of(T * 4 * state_rows, T, es, R, row_pad);
  L.total = off + n_slots * L.slot_bytes;
  return L;
}

// ES = bytes per gradient element (2: bf16, 4: fp32).
// TT = tile width known at compile time (512, the usual shape: strides become immediates) or 0 (a.T).
// GM = how the gradient rows travel: kGBox, kGRows or kGPtrs (see above).
// XR = the old model rows travel in the ring items (update-then-mix on one buffer; see below).
template <int ES, bool MEAN, int TT, int GM, bool XR = false>
__global__ void __launch_bounds__((kMaxGroups + 1) * 32 + 512, 1) nb_step_pipeline_kernel(const __grid_constant__ PipeArgs a) {
  extern __shared__ __align__(128) unsigned char smem_raw[];
  constexpr int SRC = ES == 2 ? kSrcBF16 : kSrcF32;
  constexpr bool GA = GM != kGRows;          // the consumers read the staged rows aligned
  constexpr bool kWarpIssue = GM != kGBox;   // the whole producer warp issues (one copy per row)
  constexpr int kRowPad = GM == kGRows ? 16 : 0;
  const StepArgs &s = a.s;
  const int K = s.K, T = TT ? TT : a.T, R = a.rows_per_item, NS = a.n_slots, NG = a.n_groups;
  const int NSG = NS / NG;  // slots in each group's ring
  const int NXS = a.x_stages;
  // Update-then-mix on ONE buffer (K > 32): the old model row x_i rides in learner i's ring item next to v_i, the
  // consumers write y_i = x_i - lr v_i into the buffer themselves, and nobody has to wait for a [K, T] box of old
  // models between two tiles: the ring keeps bringing the next tile's items while this tile is averaged.
  constexpr bool xr = XR;
  const int state_bytes = T * 4 * (xr ? 2 : 1);  // fp32 state rows at the head of a slot
  const PipeLayout L = pipe_layout(K, T, ES, R, NS, s.mix_slots, kRowPad, NXS, xr ? 2 : 1);
  uint64_t *full = reinterpret_cast<uint64_t *>(smem_raw);
  uint64_t *empty = full + NS;
  uint64_t *xfull = empty + NS;
  uint64_t *xempty = xfull + kMaxXStages;
  uint64_t *ybar = xempty + kMaxXStages;
  int32_t *s_col = reinterpret_cast<int32_t *>(smem_raw + L.off_tab);
  float *s_val = reinterpret_cast<float *>(s_col + s.mix_slots);
  int32_t *s_beg = reinterpret_cast<int32_t *>(s_val + s.mix_slots);
  int32_t *s_end = s_beg + K;
  float *xs_base = reinterpret_cast<float *>(smem_raw + L.off_xs);  // NXS buffers of K*T floats
  unsigned char *slots = smem_raw + L.off_slots;

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int group_warps = T / 128;                 // warps of one consumer group
  const int n_cons_warps = group_warps * a.n_groups;
  if (threadIdx.x == 0) {
    for (int q = 0; q < NS; ++q) {
      mbar_init(&full[q], 1);
      mbar_init(&empty[q], group_warps);            // released by the group that owns the ring
    }
    for (int q = 0; q < kMaxXStages; ++q) {
      mbar_init(&xfull[q], 1);
      mbar_init(&xempty[q], n_cons_warps);
      mbar_init(&ybar[q], n_cons_warps);
    }
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  bool table_ok = true;
  if constexpr (!MEAN) {
    for (int e = threadIdx.x; e < s.mix_slots; e += blockDim.x) {
      s_col[e] = s.mix->col[e];
      s_val[e] = s.mix->val[e];
      if constexpr (kDebug) table_ok = table_ok && bounds::index_inside(s_col[e], K);
    }
    for (int e = threadIdx.x; e < K; e += blockDim.x) {
      s_beg[e] = s.mix->row_beg[e];
      s_end[e] = s.mix->row_end[e];
      if constexpr (kDebug) table_ok = table_ok && s_beg[e] >= 0 && s_beg[e] <= s_end[e] && s_end[e] <= s.mix_slots;
    }
  }
  if constexpr (kDebug) {  // a table entry that names no learner: the whole CTA leaves before touching anything
    if (__syncthreads_or(!dbg_check(table_ok && L.total <= kSmemBudget, a.err, bounds::kLearnerIndex))) return;
  } else {
    __syncthreads();
  }

  const int64_t ldx = s.ldx;
  bool ok = true;

  if (warp < NG) {
    // ------------------------------------------- item producers: one per consumer group
    // Producer g (warp g; lane 0 alone when the rows travel as boxes) feeds group g's private ring
    // with the items of the learners i = g, g+NG, ... ; a slot is always filled for, and released
    // by, the same group, in order, which is what makes waiting on a phase parity unambiguous, and
    // a slow group never holds up the copies of another.
    if (kWarpIssue || lane == 0) {
      const int g = warp;
      uint32_t slot = 0, phase = 0;
      for (int tile = blockIdx.x; ok && tile < a.n_tiles; tile += gridDim.x) {
        for (int i = g; ok && i < K; i += NG) {
          const int n = s.n[i];
          int m0 = 0;
          do {
            const int rows = (n - m0 < R) ? (n - m0) : R;
            const uint32_t sl = (uint32_t)g * NSG + slot;
            if constexpr (!kWarpIssue) ok = mbar_wait(&empty[sl], phase ^ 1, a.err, 2);
            else ok = __all_sync(0xffffffffu, mbar_wait(&empty[sl], phase ^ 1, a.err, 2));
            if (!ok) break;
            if constexpr (kDebug) {
              ok = dbg_item_ok<ES, GM>(a, T, tile, i, m0, rows, lane, sl, NS, L.off_slots, L.slot_bytes, L.total);
              if constexpr (kWarpIssue) ok = __all_sync(0xffffffffu, ok);
              if (!ok) break;
            }
            unsigned char *dst = slots + (size_t)sl * L.slot_bytes;
            if (lane == 0) {
              mbar_expect_tx(&full[sl], (uint32_t)(rows * (T * ES + kRowPad) + (m0 == 0 ? state_bytes : 0)));
              if (m0 == 0) {
                tma_load_2d(dst, &a.vmap, tile * kBoxInner, i, &full[sl]);
                if (xr) tma_load_2d(dst + T * 4, &a.xrmap, tile * kBoxInner, i, &full[sl]);
              }
            }
            if constexpr (kWarpIssue) __syncwarp();
            issue_rows<ES, GM>(a, dst + state_bytes, T, tile, i, m0, rows, lane, &full[sl]);
            if (++slot == (uint32_t)NSG) { slot = 0; phase ^= 1; }
            m0 += R;
          } while (m0 < n);
        }
      }
    }
  } else if (warp == NG) {
    // ------------------------------------------- X producer: the tiles' old models, NXS buffers
    // Buffer b = titer % NXS is reused every NXS-th tile; its k-th use waits for the (k-1)-th
    // release, so with two buffers tile t+1's models load while tile t is consumed.  (One buffer:
    // K so large that two do not fit; the ring keeps filling while the next tile's models load.
    // Three: the update-then-mix order, whose averaging pass runs one tile late.)
    if (lane == 0 && !xr) {
      int titer = 0, b = 0;
      uint32_t xpar = 0;
      for (int tile = blockIdx.x; ok && tile < a.n_tiles; tile += gridDim.x, ++titer) {
        if (!(ok = mbar_wait(&xempty[b], xpar ^ 1, a.err, 1))) break;
        if constexpr (kDebug) {
          if (!(ok = dbg_check(bounds::index_inside(tile, a.n_tiles) && L.off_xs + (b + 1) * K * T * 4 <= L.off_slots,
                               a.err, bounds::kTileCoordinate)))
            break;
        }
        mbar_expect_tx(&xfull[b], (uint32_t)(K * T * 4));
        tma_load_2d(xs_base + (size_t)b * K * T, &a.xmap, tile * kBoxInner, 0, &xfull[b]);
        if (++b == NXS) { b = 0; xpar ^= 1; }
      }
    }
  } else {
    // ------------------------------------------------- consumers: NG groups of T/4 threads each
    // Group g owns the learners i with i % NG == g (their updates are independent of each other
    // once the old models are staged), so several ring items are consumed concurrently.
    const int ct = threadIdx.x - 32 * (NG + 1);
    const int nq = T / 4;  // float4 per staged row = threads per group
    const int grp = ct / nq, cq = ct - grp * nq;
    {
      const float lr = s.lr, mom = s.mom;
      const bool mix_first = s.order == NB_ORDER_MIX_THEN_UPDATE;
      // Update-then-mix (Eq. 4-6) needs every learner's y_j = x_j - lr v_j of the tile before anyone
      // averages, so the tile has two passes with a rendezvous of all groups in between.  With three
      // X buffers the averaging pass of tile t runs after the first pass of tile t+1: the groups
      // reach the rendezvous with a tile of slack and nobody idles at it.
      const bool defer = !mix_first && NXS >= 3;
      // With two buffers the averaging pass of tile t-1 runs in the MIDDLE of tile t's first pass (after
      // half of this group's learners): half a pass of slack at the rendezvous, and the buffer it frees
      // still has the other half of the pass to receive tile t+1's models.
      const bool defer_half = !mix_first && NXS == 2;
      const int half_at = ((K - grp + NG - 1) / NG) / 2;  // learners of this group done before the late pass

      // Second pass of update-then-mix on buffer ub (columns at ucol0): x_i = sum_j W_ij y_j.
      auto average_and_store = [&](int ub, uint32_t upar, int64_t ucol0) -> bool {
        if (!__all_sync(0xffffffffu, mbar_wait(&ybar[ub], upar, a.err, 5))) return false;
        const float4 *ys4 = reinterpret_cast<const float4 *>(xs_base + (size_t)ub * K * T);
        float *Xu = s.X + ucol0;
        float4 mean = make_float4(0.f, 0.f, 0.f, 0.f);
        if constexpr (MEAN) {
          for (int j = 0; j < K; ++j) mean = add4(mean, ys4[j * nq + cq]);
          mean = scale4(mean, s.inv_K);
        }
        for (int i = grp; i < K; i += NG) {
          float4 xn;
          if constexpr (MEAN) xn = mean;
          else xn = mix_row(ys4, nq, cq, s_col, s_val, s_beg[i], s_end[i]);
          st4(Xu + (int64_t)i * ldx, xn);
        }
        // the buffer was written through the generic proxy; order that before the next bulk copy
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
        __syncwarp();
        if (lane == 0) mbar_arrive(&xempty[ub]);
        return true;
      };

      uint32_t slot = 0, phase = 0;
      int titer = 0, xb = 0, prev_xb = 0;
      uint32_t xpar = 0, prev_xpar = 0;
      int64_t prev_col0 = 0;
      for (int tile = blockIdx.x; ok && tile < a.n_tiles; tile += gridDim.x, ++titer) {
        const int64_t col0 = (int64_t)tile * T + (int64_t)cq * 4;
        float *Xc = s.X + col0;
        float *Vc = s.V + col0;
        float4 *xs4w = reinterpret_cast<float4 *>(xs_base + (size_t)xb * K * T);
        const float4 *xs4 = xs4w;
        // the tile's old models are staged; XR: the buffer is free (every group has averaged the previous tile)
        ok = __all_sync(0xffffffffu, xr ? mbar_wait(&xempty[xb], xpar ^ 1, a.err, 3) : mbar_wait(&xfull[xb], xpar, a.err, 3));
        if (!ok) break;
        if constexpr (kDebug) {  // this thread's stores of the tile: 4 columns of all K rows of X and V
          ok = __all_sync(0xffffffffu,
                          dbg_check(dbg_rows_inside(s.X, ldx, K, col0, 4, 4, s.ext.x_lo, s.ext.x_hi) &&
                                        dbg_rows_inside(s.V, ldx, K, col0, 4, 4, s.ext.v_lo, s.ext.v_hi) &&
                                        bounds::index_inside(xb, NXS),
                                    a.err, bounds::kStateAddress));
          if (!ok) break;
        }
        float4 mean = make_float4(0.f, 0.f, 0.f, 0.f);
        if (MEAN && mix_first) {
          for (int j = 0; j < K; ++j) mean = add4(mean, xs4[j * nq + cq]);
          mean = scale4(mean, s.inv_K);
        }
        int done = 0;
        for (int i = grp; ok && i < K; i += NG, ++done) {  // this group's learners, from its own ring
          if (defer_half && titer > 0 && done == half_at) {
            if (!(ok = average_and_store(prev_xb, prev_xpar, prev_col0))) break;
          }
          const int n = s.n[i];
          float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
          float4 v = make_float4(0.f, 0.f, 0.f, 0.f), xi = v;
          int m0 = 0;
          do {
            const int rows = (n - m0 < R) ? (n - m0) : R;
            const uint32_t sl = (uint32_t)grp * NSG + slot;
            ok = __all_sync(0xffffffffu, mbar_wait(&full[sl], phase, a.err, 4));
            if (!ok) break;
            if constexpr (kDebug) {
              ok = __all_sync(0xffffffffu, dbg_check(sl < (uint32_t)NS && L.off_slots + (int)(sl + 1) * L.slot_bytes <= L.total,
                                                     a.err, bounds::kRingSlot));
              if (!ok) break;
            }
            const unsigned char *src = slots + (size_t)sl * L.slot_bytes;
            if (m0 == 0) {
              v = reinterpret_cast<const float4 *>(src)[cq];
              if (xr) xi = reinterpret_cast<const float4 *>(src + T * 4)[cq];
            }
            const int s0 = GA ? 0 : (a.g_mis0 + i * a.g_mis_k + m0 * a.g_mis_m);
            acc = sum_rows<SRC, GA>(acc, src + state_bytes + cq * 4 * ES, T * ES + kRowPad, rows, s0, a.g_mis_m);
            __syncwarp();
            if (lane == 0) mbar_arrive(&empty[sl]);
            if (++slot == (uint32_t)NSG) { slot = 0; phase ^= 1; }
            m0 += R;
          } while (m0 < n);
          if (!ok) break;
          const float4 vn = momentum(mom, v, s.s[i], acc);
          st4(Vc + (int64_t)i * ldx, vn);
          if (mix_first) {
            float4 xh;
            if constexpr (MEAN) xh = mean;
            else xh = mix_row(xs4, nq, cq, s_col, s_val, s_beg[i], s_end[i]);
            st4(Xc + (int64_t)i * ldx, descend(xh, lr, vn));
          } else {
            xs4w[i * nq + cq] = descend(xr ? xi : xs4[i * nq + cq], lr, vn);  // y_i replaces x_i in the buffer
          }
        }
        if (!ok) break;
        if (mix_first) {
          __syncwarp();
          if (lane == 0) mbar_arrive(&xempty[xb]);
        } else {
          // this group's y of the tile are staged: tell the others (bounded mbarrier rendezvous)
          __syncwarp();
          if (lane == 0) mbar_arrive(&ybar[xb]);
          if (defer) {
            if (titer > 0 && !(ok = average_and_store(prev_xb, prev_xpar, prev_col0))) break;
          } else if (!defer_half) {
            if (!(ok = average_and_store(xb, xpar, col0))) break;
          }
          prev_xb = xb;
          prev_xpar = xpar;
          prev_col0 = col0;
        }
        if (++xb == NXS) { xb = 0; xpar ^= 1; }
      }
      if (ok && (defer || defer_half) && titer > 0) ok = average_and_store(prev_xb, prev_xpar, prev_col0);  // the last tile's second pass
    }
  }
  if (!ok) drain_and_exit_delay();
}

// -------------------------------------------------------------------------------------------------
// The same producer / ring machinery for the two steps that need no X stage:
//   kModeAccumulate : acc[i, tile] = sum_{m < n_i} G[i, m, tile]              (nb_accumulate)
//   kModeCentralized: g = (1/K) sum_i s_i acc_i; v <- mom v + g; x <- x - lr v  (Alg. 3, one model)
// Items carry gradient rows only.  Accumulate uses NG groups (learners are independent); the
// centralized step uses one group so that the learners are folded in ascending order, exactly as
// the direct-load kernel does.
// -------------------------------------------------------------------------------------------------
constexpr int kModeAccumulate = 0, kModeCentralized = 1;
constexpr int kStreamTile = 512;  // the only tile width the no-stage kernels use

struct StreamLayout {
  int32_t off_slots, slot_bytes, total;
};
__host__ __device__ inline StreamLayout stream_layout(int T, int es, int R, int n_slots, int row_pad) {
  StreamLayout L;
  int off = 2 * n_slots * 8;
  off = (off + 127) / 128 * 128;
  L.off_slots = off;
  L.slot_bytes = slot_bytes_of(0, T, es, R, row_pad);
  L.total = off + n_slots * L.slot_bytes;
  return L;
}

// QPT: groups of four columns a consumer thread owns (T / QPT apart, so that a warp's accesses stay
// contiguous); a group has T / (4 QPT) consumer threads.
template <int ES, int MODE, int GM, int QPT>
__global__ void __launch_bounds__(kMaxGroups * (32 + 128), 1) nb_stream_pipeline_kernel(const __grid_constant__ PipeArgs a) {
  extern __shared__ __align__(128) unsigned char smem_raw[];
  constexpr int SRC = ES == 2 ? kSrcBF16 : kSrcF32;
  constexpr bool GA = GM != kGRows;
  constexpr bool kWarpIssue = GM != kGBox;
  constexpr int kRowPad = GM == kGRows ? 16 : 0;
  const StepArgs &s = a.s;
  constexpr int T = kStreamTile;  // strides and offsets become immediates
  const int K = s.K, R = a.rows_per_item, NS = a.n_slots, NG = a.n_groups;
  const int NSG = NS / NG;
  const StreamLayout L = stream_layout(T, ES, R, NS, kRowPad);
  uint64_t *full = reinterpret_cast<uint64_t *>(smem_raw);
  uint64_t *empty = full + NS;
  unsigned char *slots = smem_raw + L.off_slots;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int group_threads = T / (4 * QPT);
  if (threadIdx.x == 0) {
    for (int q = 0; q < NS; ++q) {
      mbar_init(&full[q], 1);
      mbar_init(&empty[q], group_threads / 32);
    }
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  __syncthreads();
  const int64_t ldx = s.ldx;
  bool ok = true;

  if (warp < NG) {
    if (kWarpIssue || lane == 0) {  // producer of group `warp`
      const int g = warp;
      uint32_t slot = 0, phase = 0;
      for (int tile = blockIdx.x; ok && tile < a.n_tiles; tile += gridDim.x) {
        for (int i = g; ok && i < K; i += NG) {
          const int n = s.n[i];
          int m0 = 0;
          do {
            const int rows = (n - m0 < R) ? (n - m0) : R;
            const uint32_t sl = (uint32_t)g * NSG + slot;
            if constexpr (!kWarpIssue) ok = mbar_wait(&empty[sl], phase ^ 1, a.err, 2);
            else ok = __all_sync(0xffffffffu, mbar_wait(&empty[sl], phase ^ 1, a.err, 2));
            if (!ok) break;
            if constexpr (kDebug) {
              ok = dbg_item_ok<ES, GM>(a, T, tile, i, m0, rows, lane, sl, NS, L.off_slots, L.slot_bytes, L.total);
              if constexpr (kWarpIssue) ok = __all_sync(0xffffffffu, ok);
              if (!ok) break;
            }
            if (lane == 0) mbar_expect_tx(&full[sl], (uint32_t)(rows * (T * ES + kRowPad)));  // 0 rows: a plain arrival
            if constexpr (kWarpIssue) __syncwarp();
            issue_rows<ES, GM>(a, slots + (size_t)sl * L.slot_bytes, T, tile, i, m0, rows, lane, &full[sl]);
            if (++slot == (uint32_t)NSG) { slot = 0; phase ^= 1; }
            m0 += R;
          } while (m0 < n);
        }
      }
    }
  } else {
    const int ct = threadIdx.x - 32 * NG;
    const int grp = ct / group_threads, cq = ct - grp * group_threads;
    uint32_t slot = 0, phase = 0;
    // this group's barriers and this thread's first column group inside a slot, as 32-bit shared addresses
    const uint32_t full_a = smem_u32(full) + 8u * (uint32_t)(grp * NSG), empty_a = smem_u32(empty) + 8u * (uint32_t)(grp * NSG);
    const uint32_t slots_a = smem_u32(slots) + (uint32_t)(grp * NSG * L.slot_bytes) + (uint32_t)(cq * 4 * ES);
    for (int tile = blockIdx.x; ok && tile < a.n_tiles; tile += gridDim.x) {
      const int64_t col0 = (int64_t)tile * T + (int64_t)cq * 4;  // this thread's q-th column group starts at col0 + q T / QPT
      float4 x[QPT], v[QPT], gs[QPT];
#pragma unroll
      for (int q = 0; q < QPT; ++q) x[q] = v[q] = gs[q] = make_float4(0.f, 0.f, 0.f, 0.f);
      if constexpr (kDebug) {  // this thread's global footprint of the tile
        bool in = true;
#pragma unroll
        for (int q = 0; q < QPT; ++q) {
          const int64_t c = col0 + q * (T / QPT);
          in = in && (MODE == kModeAccumulate
                          ? dbg_rows_inside(s.acc, ldx, K, c, 4, 4, s.ext.acc_lo, s.ext.acc_hi)
                          : dbg_rows_inside(s.X, ldx, 1, c, 4, 4, s.ext.x_lo, s.ext.x_hi) &&
                                dbg_rows_inside(s.V, ldx, 1, c, 4, 4, s.ext.v_lo, s.ext.v_hi));
        }
        ok = __all_sync(0xffffffffu, dbg_check(in, a.err, bounds::kStateAddress));
        if (!ok) break;
      }
      if constexpr (MODE == kModeCentralized) {  // requested early, used after the last learner
#pragma unroll
        for (int q = 0; q < QPT; ++q) {
          x[q] = ld4(s.X + col0 + q * (T / QPT));
          v[q] = ld4(s.V + col0 + q * (T / QPT));
        }
      }
      for (int i = grp; ok && i < K; i += NG) {
        const int n = s.n[i];
        float4 acc[QPT];
#pragma unroll
        for (int q = 0; q < QPT; ++q) acc[q] = make_float4(0.f, 0.f, 0.f, 0.f);
        int m0 = 0;
        do {
          const int rows = (n - m0 < R) ? (n - m0) : R;
          ok = __all_sync(0xffffffffu, mbar_wait_a(full_a + 8u * slot, phase, a.err, 4));
          if (!ok) break;
          if constexpr (kDebug) {
            const uint32_t sl = (uint32_t)grp * NSG + slot;
            ok = __all_sync(0xffffffffu, dbg_check(sl < (uint32_t)NS && L.off_slots + (int)(sl + 1) * L.slot_bytes <= L.total,
                                                   a.err, bounds::kRingSlot));
            if (!ok) break;
          }
          const uint32_t row_a = slots_a + slot * (uint32_t)L.slot_bytes;
          const int s0 = GA ? 0 : (a.g_mis0 + i * a.g_mis_k + m0 * a.g_mis_m);
          if constexpr (MODE == kModeCentralized) {  // all loads of the item first (same additions, same order)
#pragma unroll
            for (int q = 0; q < QPT; ++q)
              acc[q] = sum_rows_a<SRC, GA>(acc[q], row_a + q * (T / QPT) * ES, T * ES + kRowPad, rows, s0, a.g_mis_m);
          } else {  // plain loads: the compiler may then overlap the rows of this loop (0.98 -> 1.00 on 2.5 KB items)
            const unsigned char *rowp = slots + (size_t)((uint32_t)grp * NSG + slot) * L.slot_bytes + (size_t)cq * 4 * ES;
            for (int r = 0; r < rows; ++r) {
              const int shift = GA ? 0 : ((s0 + r * a.g_mis_m) & 15);
#pragma unroll
              for (int q = 0; q < QPT; ++q)
                acc[q] = add4(acc[q], ld_row4<SRC, GA>(rowp + q * (T / QPT) * ES + (size_t)r * (T * ES + kRowPad) + shift));
            }
          }
          __syncwarp();
          if (lane == 0) mbar_arrive_a(empty_a + 8u * slot);
          if (++slot == (uint32_t)NSG) { slot = 0; phase ^= 1; }
          m0 += R;
        } while (m0 < n);
        if (!ok) break;
        if constexpr (MODE == kModeAccumulate) {
#pragma unroll
          for (int q = 0; q < QPT; ++q) st4(s.acc + (int64_t)i * ldx + col0 + q * (T / QPT), acc[q]);
        } else {
          const float si = s.s[i];
#pragma unroll
          for (int q = 0; q < QPT; ++q) gs[q] = fma4(si, acc[q], gs[q]);
        }
      }
      if (!ok) break;
      if constexpr (MODE == kModeCentralized) {
#pragma unroll
        for (int q = 0; q < QPT; ++q) {
          const float4 vn = momentum(s.mom, v[q], s.inv_K, gs[q]);
          st4(s.V + col0 + q * (T / QPT), vn);
          st4(s.X + col0 + q * (T / QPT), descend(x[q], s.lr, vn));
        }
      }
    }
  }
  if (!ok) drain_and_exit_delay();
}

// Self-test of the bounded wait: one warp waits, with a short limit, on a barrier phase that nothing
// will ever complete.  Every lane must give up, the error word must carry `code`, and the kernel
// must return normally (no trap, the context stays usable).
__global__ void nb_wait_selftest_kernel(int *err, int code, long long limit_cycles, int *gave_up) {
  __shared__ uint64_t bar;
  if (threadIdx.x == 0) {
    mbar_init(&bar, 1);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  __syncthreads();
  const bool ok = mbar_wait(&bar, 0, err, code, limit_cycles);
  if (!ok) atomicAdd(gave_up, 1);
}

struct PipeTuning {
  int T = 0, slots = 0, ctas_per_sm = 0, rows = 0, groups = 0, x_stages = 0, qpt = 0, xr = -1;
  int sm_count = 0;
};

// Shape overrides for tuning sweeps.  Only a library built with -DNB_TUNING reads them (from the
// environment, once per process); the shipped build always takes the planner's own choice.
PipeTuning &tuning() {
  static PipeTuning t = [] {
    PipeTuning q;
#ifdef NB_TUNING
    auto geti = [](const char *name, int dflt) {
      const char *v = std::getenv(name);
      return v ? std::atoi(v) : dflt;
    };
    q.T = geti("NB_PIPELINE_TILE", 0);
    q.slots = geti("NB_PIPELINE_SLOTS", 0);
    q.ctas_per_sm = geti("NB_PIPELINE_CTAS_PER_SM", 0);
    q.rows = geti("NB_PIPELINE_ROWS", 0);
    q.groups = geti("NB_PIPELINE_GROUPS", 0);
    q.x_stages = geti("NB_PIPELINE_XSTAGES", 0);
    q.qpt = geti("NB_PIPELINE_QPT", 0);
    q.xr = geti("NB_PIPELINE_XR", -1);
#endif
    return q;
  }();
  if (t.sm_count == 0) {
    int dev = 0;
    cudaGetDevice(&dev);
    cudaDeviceGetAttribute(&t.sm_count, cudaDevAttrMultiProcessorCount, dev);
    if (t.sm_count <= 0) t.sm_count = 148;
  }
  return t;
}


using EncodeFn = CUresult (*)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *,
                              const cuuint64_t *, const cuuint32_t *, const cuuint32_t *, CUtensorMapInterleave,
                              CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

// The driver's tensor-map encoder, looked up through the runtime (no link against libcuda).
EncodeFn encode_fn() {
  static EncodeFn fn = [] {
    void *p = nullptr;
    cudaDriverEntryPointQueryResult q;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) != cudaSuccess ||
        q != cudaDriverEntryPointSuccess)
      p = nullptr;
    cudaGetLastError();
    return reinterpret_cast<EncodeFn>(p);
  }();
  return fn;
}

CUtensorMapDataType unit_type(int bytes) {
  switch (bytes) {
    case 1: return CU_TENSOR_MAP_DATA_TYPE_UINT8;
    case 2: return CU_TENSOR_MAP_DATA_TYPE_UINT16;
    case 4: return CU_TENSOR_MAP_DATA_TYPE_UINT32;
    default: return CU_TENSOR_MAP_DATA_TYPE_UINT64;
  }
}

// Rows of `row_bytes`-pitched data seen as [outer..., units]: the innermost extent covers exactly the
// full tiles, so no copy ever touches a ragged edge.
bool encode_map(CUtensorMap *map, const void *base, int unit_bytes, int rank, const cuuint64_t *dims,
                const cuuint64_t *strides, const cuuint32_t *box) {
  const cuuint32_t ones[3] = {1, 1, 1};
  return encode_fn()(map, unit_type(unit_bytes), (cuuint32_t)rank, const_cast<void *>(base), dims, strides, box, ones,
                     CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_NONE, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                     CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// Which columns the bulk-copy kernels may cover, given how the gradient stream is aligned.
//   16-byte aligned rows: box copies, tiles [0, P / T).
//   otherwise: one bulk copy per row of the 16-byte aligned superset of its tile segment, which reads
//   up to 15 bytes before the segment and up to 16 bytes after it.  Both stay inside the caller's
//   stream if (a) the first tile is left out when G itself is not 16-byte aligned (`head` columns go
//   to the direct-load kernel) and (b) the last tile covered ends at least 16 bytes before the end of
//   a row.
struct Coverage {
  bool rows_aligned;
  int64_t head;     // columns [0, head) are left to the direct-load kernel
  int64_t n_tiles;  // tiles covered, starting at column `head`
};
Coverage coverage(const StepArgs &a, int es, int T) {
  Coverage c;
  if (a.row_ptrs) {  // held rows: 16-byte aligned vectors, exact copies, every full tile
    c.rows_aligned = true;
    c.head = 0;
    c.n_tiles = a.P / T;
    return c;
  }
  c.rows_aligned = (uintptr_t)a.G % 16 == 0 && (a.ld_m * es) % 16 == 0 && (a.ld_k * es) % 16 == 0;
  if (c.rows_aligned) {
    c.head = 0;
    c.n_tiles = a.P / T;
  } else {
    c.head = (uintptr_t)a.G % 16 == 0 ? 0 : T;
    c.n_tiles = (a.P - c.head - 16 / es) / T;
    if (a.P - c.head - 16 / es < 0) c.n_tiles = 0;
  }
  return c;
}

void fill_row_args(PipeArgs *p, const StepArgs &a, int es) {
  p->g_base = reinterpret_cast<const unsigned char *>(a.G);
  p->g_ld_m_bytes = a.ld_m * es;
  p->g_ld_k_bytes = a.ld_k * es;
  p->g_mis0 = (int32_t)((uintptr_t)a.G & 15);
  p->g_mis_m = (int32_t)((a.ld_m * es) & 15);
  p->g_mis_k = (int32_t)((a.ld_k * es) & 15);
}

}  // namespace

// Chooses tile width, slot count and CTAs per SM; returns false when the pipeline kernel does not
// apply (then the direct-load kernel runs the whole range).
bool plan_pipeline(const StepArgs &a, int es, PipePlan *plan) {
  PipeTuning &t = tuning();
  if (!a.row_ptrs && (uintptr_t)a.G % es != 0) return false;
  if (!encode_fn()) return false;
  int Rmax = t.rows ? t.rows : 8;
  if (Rmax < 1) Rmax = 1;
  if (Rmax > kMaxRowsPerItem) Rmax = kMaxRowsPerItem;
  if (Rmax > a.M) Rmax = a.M;
  const bool rows_aligned = coverage(a, es, 512).rows_aligned;
  const int row_pad = rows_aligned ? 0 : 16;
  // Tile width: a box row is 256 units of T*es/256 bytes, so T is 128, 256 or 512.
  // Shapes tried in order (measured on B200, see profiles/): two CTAs per SM with two consumer
  // groups each while two X buffers leave room for it (K <= 16 at T = 512), else one CTA per SM with
  // four groups; for K so large that two buffers of 512 columns do not fit, one buffer (the ring
  // keeps the copies going while the next tile's models load) before narrower tiles.  The
  // update-then-mix order first tries three X buffers, which let its averaging pass run a tile
  // late.  The first shape whose ring has at least two slots per group is taken; a shape with rows = 4
  // halves the rows per ring item (the slots shrink) so that 512-column tiles still fit where 8-row
  // items do not (K = 64 with fp32 gradients: 0.94 on 256-column tiles).  A tuning build's overrides
  // replace the corresponding field of every shape.
  struct Shape { int T, ctas, groups, x_stages, rows, xr = 0; };  // xr: old model rows travel in the ring items
  static const Shape mix_first_shapes[] = {{512, 2, 2, 2, 8}, {512, 1, 4, 2, 8}, {512, 1, 4, 1, 8}, {512, 1, 4, 1, 4},
                                           {256, 1, 4, 2, 8}, {128, 1, 4, 2, 8}};
  static const Shape update_first_shapes[] = {{512, 1, 4, 3, 8}, {512, 2, 2, 2, 8}, {512, 1, 4, 2, 8}, {512, 1, 4, 1, 8, 1},
                                              {512, 1, 4, 1, 8}, {512, 1, 4, 1, 4, 1}, {512, 1, 4, 1, 4}, {256, 1, 4, 2, 8},
                                              {128, 1, 4, 2, 8}};
  // Few mini-batches per batch (items of a momentum row and at most 4 KB of gradient rows): one CTA
  // per SM with four groups and three slots per group (cfg4 sizes at P = 138M: 0.99 of the measured
  // copy bandwidth against 0.95 for two CTAs with two groups of two slots; equal within 1 % at 25-51M).
  static const Shape small_item_shapes[] = {{512, 1, 4, 2, 8}, {512, 2, 2, 2, 8}, {512, 1, 4, 1, 8}, {512, 1, 4, 1, 4},
                                            {256, 1, 4, 2, 8}, {128, 1, 4, 2, 8}};
  const bool mix_first = a.order == NB_ORDER_MIX_THEN_UPDATE;
  const bool small_slot = slot_bytes_of(512 * 4, 512, es, Rmax, row_pad) <= 6400;  // <= 4 bf16 / 2 fp32 rows
  const bool small_items = mix_first && small_slot;
  // Rows named by a pointer table (the streaming entry points in hold mode) also do best on one CTA per SM
  // with four groups (cfg3 sizes: 0.99 against 0.98 for two CTAs of two groups).
  const bool one_cta_first = small_items || (mix_first && a.row_ptrs != nullptr);
  const Shape *table = one_cta_first ? small_item_shapes : mix_first ? mix_first_shapes : update_first_shapes;
  // Few learners: a tile carries few bytes (T (16 K + e_g sum n_i)), so what limits the step is how many tiles an SM
  // has in flight, and the groups of one CTA share a single tile.  Four CTAs per SM of ONE consumer group each (the
  // group takes all K learners of its tile) then do best.  Fraction of the measured copy bandwidth, ring, bf16, M = 1 /
  // 4 / 8: K = 1 0.25 / 0.31 / 0.71 -> 0.71 / 0.88 / 0.97, K = 2 0.45 / 0.53 / 0.98 -> 0.85 / 0.94 / 1.02, K = 3 0.62 / 0.71 /
  // 0.96 -> 0.88 / 0.96 / 1.03 (M <= 8: with two items per learner the tables' shapes stay ahead, K = 2, M = 16 0.99 against
  // 0.94); with small items also K = 4..7 (K = 4 0.74 / 0.82 -> 0.90 / 0.97, K = 6 0.74 / 0.83 -> 0.91 /
  // 0.98; their 8-row items stay at 1.03 on two CTAs of two groups, K = 8 at 0.92-1.04 on the tables above).
  // Update-then-mix, K <= 8 (before: K = 2 0.37-0.55, K = 4 0.64-0.88, K = 6 0.64-0.86): four such CTAs, with three X
  // buffers for K <= 2 and small items (K = 2 0.74-0.94, K = 4 0.84-1.00); K = 6, 7 with 8-row items two CTAs of two
  // groups (0.86 -> 1.02); K = 8 with 8-row items keeps the table (1.02).
  Shape first = {0, 0, 0, 0, 0};
  if (!a.row_ptrs) {
    if (mix_first) {
      if (a.K == 1 || (a.K <= 3 && Rmax >= a.M) || (a.K <= 7 && small_slot)) first = {512, 4, 1, 2, 8};
    } else if (a.K <= 8) {
      if (small_slot) first = {512, 4, 1, a.K <= 2 ? 3 : 2, 8};
      else if (a.K <= 5) first = {512, 4, 1, 2, 8};
      else if (a.K <= 7) first = {512, 2, 2, 2, 8};
    }
  }
  Shape shapes[10];
  int n_shapes = 0;
  if (first.T) shapes[n_shapes++] = first;
  for (int q = 0; q < (mix_first ? 6 : 9); ++q) shapes[n_shapes++] = table[q];
  // The update-then-mix order releases no slot while a group averages, so its ring is what keeps memory busy: a shape is
  // taken there only if the rings of an SM hold at least 56 KB (K = 32, M = 1: three X buffers leave 8 slots of 3 KB,
  // 0.77; two leave 32, 0.96.  K = 40, M = 4: two buffers with 8 slots of 6 KB 0.81, one buffer with 24 0.90; K = 40,
  // M = 1: two buffers with 20 slots of 3 KB 1.00); if no shape offers that, the first one that fits at all.
  struct Chosen { int T, ctas, groups, slots, x_stages, R, xr; };
  Chosen c = {0, 0, 0, 0, 0, 0, 0}, fallback = {0, 0, 0, 0, 0, 0, 0};
  for (int q = 0; q < n_shapes && !c.T; ++q) {
    const Shape &sh = shapes[q];
    Chosen k;
    k.R = sh.rows < Rmax ? sh.rows : Rmax;
    k.T = t.T ? t.T : sh.T;
    k.ctas = t.ctas_per_sm ? t.ctas_per_sm : sh.ctas;
    k.groups = t.groups ? t.groups : sh.groups;
    k.x_stages = t.x_stages ? t.x_stages : sh.x_stages;
    k.xr = (!mix_first && k.x_stages == 1 && sh.xr && t.xr != 0) ? 1 : 0;
    if (k.T != 128 && k.T != 256 && k.T != 512) return false;
    if (k.x_stages < 1 || k.x_stages > kMaxXStages) return false;
    if (k.groups > kMaxGroups) k.groups = kMaxGroups;
    if (k.groups > a.K) k.groups = a.K;
    while (k.groups > 1 && k.groups * (k.T / 4) > 512) --k.groups;
    if (k.groups < 1 || k.ctas < 1) return false;
    const PipeLayout L0 = pipe_layout(a.K, k.T, es, k.R, 0, a.mix_slots, row_pad, k.x_stages, 1 + k.xr);
    const int budget = kSmemBudget / k.ctas - 1024;
    const int slot_bytes = L0.slot_bytes;
    k.slots = (budget - L0.total - 256) / slot_bytes;
    if (t.slots && t.slots < k.slots) k.slots = t.slots;
    if (k.slots > 32) k.slots = 32;
    k.slots -= k.slots % k.groups;  // every group's ring has the same number of slots
    if (k.slots < 2 * k.groups) continue;
    // old models in the ring: only with three slots per group (K = 48, bf16: M = 4, 16 slots 0.84 -> 0.97; M = 8, 8 slots
    // 0.94 -> 0.90: with two slots per group the larger items starve the ring, and the plain one-buffer shape follows)
    if (k.xr && k.slots < 3 * k.groups) continue;
    if (!fallback.T) fallback = k;
    // Alg. 2 order, learners that need several items per tile (M > R): two CTAs per SM are taken only with four slots
    // per group (K = 16, M = 16, bf16: two slots per group 0.99, one CTA of four groups with every slot that fits 1.03).
    const bool deep_enough = mix_first ? (k.ctas != 2 || k.R >= a.M || k.slots >= 4 * k.groups)
                                       : (int64_t)k.ctas * k.slots * slot_bytes >= 56 * 1024;
    if (deep_enough || t.slots) c = k;
  }
  if (!c.T) c = fallback;
  if (!c.T) return false;
  const int T = c.T, ctas = c.ctas, groups = c.groups, x_stages = c.x_stages, R = c.R, xr = c.xr;
  int slots = c.slots;
  const Coverage cov = coverage(a, es, T);
  if (cov.n_tiles < 1) return false;
  if ((cov.n_tiles + 1) * (int64_t)kBoxInner >= (1ll << 31)) return false;  // tile coordinates are 32-bit
  // Ring depth.  With two X buffers in the Alg. 2 order, when one item holds a learner's whole
  // contribution (R >= M) two slots per group (three for the small items of M <= 4) keep the copies
  // back to back and deeper rings measured
  // 1-4 % slower (more copies in flight than the latency needs only spread the chip over more DRAM
  // rows at once); learners that need several items per tile use all the slots that fit.  Every slot
  // that fits is also used by the shapes whose consumers pause: the single X buffer of K > 32 (the ring
  // is what keeps memory busy while the next tile's models load: K = 40 / 48, 12 slots 1.03 of the
  // measured copy bandwidth, 8 slots 0.98) and the update-then-mix order (no slot is released while a
  // group averages: cfg3 sizes 12 slots 1.04, 8 slots 0.99).
  const int per_group = (small_items && ctas == 1) ? 3 : 2;
  if (!t.slots && mix_first && x_stages == 2 && R >= a.M && slots > per_group * groups) slots = per_group * groups;
  const PipeLayout L = pipe_layout(a.K, T, es, R, slots, a.mix_slots, row_pad, x_stages, 1 + xr);
  if (L.total > kSmemBudget) return false;
  plan->T = T;
  plan->rows_per_item = R;
  plan->n_slots = slots;
  plan->n_groups = groups;
  plan->smem_bytes = L.total;
  plan->n_tiles = (int)cov.n_tiles;
  plan->head = (int)cov.head;
  plan->row_copies = a.row_ptrs ? 2 : rows_aligned ? 0 : 1;
  plan->x_stages = x_stages;
  plan->x_in_ring = xr != 0;
  const int64_t max_ctas = (int64_t)ctas * t.sm_count;
  plan->grid = (int)(plan->n_tiles < max_ctas ? plan->n_tiles : max_ctas);
  return true;
}

// Shape of the no-stage kernels: T = 512, R rows per item; two CTAs per SM with two groups each for
// the masked accumulate, CTAs of one group for the centralized step.
bool plan_stream(const StepArgs &a, int es, bool centralized, PipePlan *plan) {
  PipeTuning &t = tuning();
  if (!a.row_ptrs && (uintptr_t)a.G % es != 0) return false;
  if (!encode_fn()) return false;
  const int T = kStreamTile;
  const Coverage cov = coverage(a, es, T);
  if (cov.n_tiles < 1) return false;
  if ((cov.n_tiles + 1) * (int64_t)kBoxInner >= (1ll << 31)) return false;  // tile coordinates are 32-bit
  const int row_pad = cov.rows_aligned ? 0 : 16;
  int R = es == 2 ? 8 : 4;
  if (R > a.M) R = a.M;
  int groups = centralized ? 1 : (t.groups ? t.groups : 2);
  if (groups > kMaxGroups) groups = kMaxGroups;
  if (groups > a.K) groups = a.K;
  // Centralized step (one group per CTA).  bf16 gradients: 8 CTAs per SM whose consumer threads own two groups of four
  // columns each (96 threads of 72 registers: nine such CTAs are what the register file holds).  Fraction of the measured copy
  // bandwidth, cfg3 sizes / items of 2.5 KB (M = 4, cfg4 sizes): 6 CTAs of 4-column threads 1.05 / 0.89, 8 CTAs of
  // 8-column threads 1.055 / 0.97 (6 such CTAs 1.04 / 0.78: the step is bound by the number of consumer groups
  // and the instructions they issue per item, not by bytes in flight; ring depth beyond 4 slots changes nothing).
  // fp32 gradients (cfg2 sizes): 4 CTAs of 4-column threads 1.01, 5 -> 0.86, 6 -> 0.97; 8-column threads 4 -> 1.02, 8 -> 0.93.
  const int qpt = t.qpt ? (t.qpt == 2 ? 2 : 1) : (centralized && es == 2 ? 2 : 1);
  // Items of at most 5 KB (M <= 5) leave room for a ninth CTA (4-5 slots each): cfg4 sizes 0.97 -> 1.00, M = 1 / 2 0.55 ->
  // 0.59 / 0.61, M = 5 1.00 -> 1.02, against 1.055 -> 1.045 for 8 KB items, which stay at eight.
  // Masked accumulate: two CTAs of two groups (cfg3 sizes 1.05, M = 4 0.98-1.00); three when an item is at most 3 KB
  // of bf16 rows (M = 1, 2: 0.79-0.80 -> 0.93-0.94; M = 3: 0.92 -> 0.97).
  const int item_bytes = slot_bytes_of(0, T, es, R, row_pad);
  const int ctas = t.ctas_per_sm ? t.ctas_per_sm
                   : centralized ? (es == 2 ? (item_bytes <= 5120 + 128 ? 9 : 8) : 4)
                                 : (es == 2 && item_bytes <= 3072 + 128 ? 3 : 2);
  const int budget = kSmemBudget / ctas - 1024;
  int slots = (budget - 512) / slot_bytes_of(0, T, es, R, row_pad);
  if (slots > 16) slots = 16;
  if (centralized && R < a.M) {
    // learners that need several items per tile do best on a ring of 128 KB per SM (K = 16, bf16, M = 16: three
    // slots of 8 KB per CTA 1.02, two 1.07; fp32, M = 8: six 1.03, four 1.08); one-item learners use every slot that fits
    const int cap = 128 * 1024 / (ctas * item_bytes);
    if (cap >= 2 && slots > cap) slots = cap;
  }
  if (!centralized) {
    // Masked accumulate: the optimum is a ring of about 100 KB per SM (slots per CTA -> fraction of the measured copy
    // bandwidth; 8 KB slots, cfg3 sizes: 4 -> 0.86, 6 -> 1.01, 8 -> 1.05, 12 -> 0.91; 6 KB: 8 -> 1.02, 10 -> 0.98; 5 KB: 8 ->
    // 0.97, 12 -> 0.94; 4 KB, cfg4 sizes: 8 -> 0.94, 12 -> 1.00, 16 -> 0.94; three CTAs, 3 KB: 8 -> 0.97, 12 -> 0.88; 2 KB
    // and 1 KB: 8 -> 0.90, 12 -> 0.94): four slots per group, six where a slot is at most 4 KB (two CTAs) or 2 KB (three).
    int per_group = item_bytes <= (ctas == 3 ? 2048 : 4096) + 128 ? 6 : 4;
    if (slots > per_group * groups) slots = per_group * groups;
  }
  if (t.slots && t.slots < slots) slots = t.slots;
  slots -= slots % groups;
  if (slots < 2 * groups) return false;
  plan->T = T;
  plan->rows_per_item = R;
  plan->n_slots = slots;
  plan->n_groups = groups;
  plan->smem_bytes = stream_layout(T, es, R, slots, row_pad).total;
  plan->n_tiles = (int)cov.n_tiles;
  plan->head = (int)cov.head;
  plan->row_copies = a.row_ptrs ? 2 : cov.rows_aligned ? 0 : 1;
  plan->x_stages = 0;
  plan->quads_per_thread = qpt;
  const int64_t max_ctas = (int64_t)ctas * t.sm_count;
  plan->grid = (int)(plan->n_tiles < max_ctas ? plan->n_tiles : max_ctas);
  return true;
}

namespace {
// G: [K, M, units]; one map per box height (16-byte aligned rows only).
bool encode_gmaps(PipeArgs *p, const StepArgs &a, int es, const PipePlan &plan) {
  const cuuint64_t units = (cuuint64_t)plan.n_tiles * kBoxInner;
  const int ub = plan.T * es / kBoxInner;
  const cuuint64_t dims[3] = {units, (cuuint64_t)a.M, (cuuint64_t)a.K};
  const cuuint64_t strides[2] = {(cuuint64_t)a.ld_m * es, (cuuint64_t)a.ld_k * es};
  const int rmax = plan.rows_per_item < a.M ? plan.rows_per_item : a.M;
  for (int r = 1; r <= rmax; ++r) {
    const cuuint32_t box[3] = {kBoxInner, (cuuint32_t)r, 1};
    if (!encode_map(&p->gmap[r - 1], a.G, ub, 3, dims, strides, box)) return false;
  }
  return true;
}

void fill_pipe_args(PipeArgs *p, const StepArgs &a, const PipePlan &plan, int *err_flag) {
  std::memset(p, 0, sizeof(*p));
  p->s = a;
  p->T = plan.T;
  p->n_slots = plan.n_slots;
  p->rows_per_item = plan.rows_per_item;
  p->n_tiles = plan.n_tiles;
  p->n_groups = plan.n_groups;
  p->x_stages = plan.x_stages;
  p->err = err_flag;
}
}  // namespace

// `a` describes the columns the kernel covers (the caller has already cut off plan.head).
cudaError_t launch_stream_pipeline(const StepArgs &a, int es, bool centralized, const PipePlan &plan, int *err_flag,
                                   cudaStream_t st) {
  PipeArgs p;
  fill_pipe_args(&p, a, plan, err_flag);
  if (plan.row_copies == 1) fill_row_args(&p, a, es);
  else if (plan.row_copies == 0 && !encode_gmaps(&p, a, es, plan)) return cudaErrorNotSupported;  // nothing launched: caller falls back
  const int qpt = plan.quads_per_thread;
  const int threads = plan.n_groups * (32 + plan.T / (4 * qpt));
#define NB_LAUNCH1(ES, MODE, QPT)                                                                                                      \
  do {                                                                                                                                 \
    if (plan.row_copies == 2) nb_stream_pipeline_kernel<ES, MODE, kGPtrs, QPT><<<plan.grid, threads, plan.smem_bytes, st>>>(p);        \
    else if (plan.row_copies == 1) nb_stream_pipeline_kernel<ES, MODE, kGRows, QPT><<<plan.grid, threads, plan.smem_bytes, st>>>(p);   \
    else nb_stream_pipeline_kernel<ES, MODE, kGBox, QPT><<<plan.grid, threads, plan.smem_bytes, st>>>(p);                              \
  } while (0)
#define NB_LAUNCH(ES, MODE)                  \
  do {                                       \
    if (qpt == 2) NB_LAUNCH1(ES, MODE, 2);   \
    else NB_LAUNCH1(ES, MODE, 1);            \
  } while (0)
  if (es == 2) {
    if (centralized) NB_LAUNCH(2, kModeCentralized);
    else NB_LAUNCH(2, kModeAccumulate);
  } else {
    if (centralized) NB_LAUNCH(4, kModeCentralized);
    else NB_LAUNCH(4, kModeAccumulate);
  }
#undef NB_LAUNCH1
#undef NB_LAUNCH
  return cudaGetLastError();
}

cudaError_t launch_wait_selftest(int *err_flag, int code, long long limit_cycles, int *gave_up, cudaStream_t st) {
  nb_wait_selftest_kernel<<<1, 32, 0, st>>>(err_flag, code, limit_cycles, gave_up);
  return cudaGetLastError();
}

cudaError_t configure_pipeline() {
  cudaError_t e;
#define NB_CFG1(...)                                                                                                  \
  if ((e = cudaFuncSetAttribute(__VA_ARGS__, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemBudget)) != cudaSuccess) \
    return e;
#define NB_CFG(ES, MEAN)                                                                                         \
  NB_CFG1(nb_step_pipeline_kernel<ES, MEAN, 512, kGBox>) NB_CFG1(nb_step_pipeline_kernel<ES, MEAN, 0, kGBox>)     \
  NB_CFG1(nb_step_pipeline_kernel<ES, MEAN, 512, kGRows>) NB_CFG1(nb_step_pipeline_kernel<ES, MEAN, 0, kGRows>)   \
  NB_CFG1(nb_step_pipeline_kernel<ES, MEAN, 512, kGPtrs>) NB_CFG1(nb_step_pipeline_kernel<ES, MEAN, 0, kGPtrs>)   \
  NB_CFG1(nb_step_pipeline_kernel<ES, MEAN, 512, kGBox, true>) NB_CFG1(nb_step_pipeline_kernel<ES, MEAN, 512, kGRows, true>) \
  NB_CFG1(nb_step_pipeline_kernel<ES, MEAN, 512, kGPtrs, true>)
  NB_CFG(2, true) NB_CFG(2, false) NB_CFG(4, true) NB_CFG(4, false)
#undef NB_CFG
#define NB_CFG(ES, MODE)                                                                                            \
  NB_CFG1(nb_stream_pipeline_kernel<ES, MODE, kGBox, 1>) NB_CFG1(nb_stream_pipeline_kernel<ES, MODE, kGRows, 1>)     \
  NB_CFG1(nb_stream_pipeline_kernel<ES, MODE, kGPtrs, 1>) NB_CFG1(nb_stream_pipeline_kernel<ES, MODE, kGBox, 2>)     \
  NB_CFG1(nb_stream_pipeline_kernel<ES, MODE, kGRows, 2>) NB_CFG1(nb_stream_pipeline_kernel<ES, MODE, kGPtrs, 2>)
  NB_CFG(2, kModeAccumulate) NB_CFG(2, kModeCentralized) NB_CFG(4, kModeAccumulate) NB_CFG(4, kModeCentralized)
#undef NB_CFG
#undef NB_CFG1
  return cudaSuccess;
}

// `a` describes the columns the kernel covers (the caller has already cut off plan.head).
cudaError_t launch_step_pipeline(const StepArgs &a, int es, const PipePlan &plan, int *err_flag, cudaStream_t st) {
  PipeArgs p;
  fill_pipe_args(&p, a, plan, err_flag);
  const cuuint64_t units = (cuuint64_t)plan.n_tiles * kBoxInner;
  {  // X and V: [K, units] fp32 rows of pitch ldx
    const int ub = plan.T * 4 / kBoxInner;
    const cuuint64_t dims[2] = {units, (cuuint64_t)a.K};
    const cuuint64_t strides[1] = {(cuuint64_t)a.ldx * 4};
    const cuuint32_t xbox[2] = {kBoxInner, (cuuint32_t)a.K};
    const cuuint32_t vbox[2] = {kBoxInner, 1};
    if (!encode_map(&p.xmap, a.X, ub, 2, dims, strides, xbox) || !encode_map(&p.vmap, a.V, ub, 2, dims, strides, vbox) ||
        (plan.x_in_ring && !encode_map(&p.xrmap, a.X, ub, 2, dims, strides, vbox)))
      return cudaErrorNotSupported;  // nothing launched: caller falls back to the direct-load kernel
  }
  if (plan.row_copies == 1) fill_row_args(&p, a, es);
  else if (plan.row_copies == 0 && !encode_gmaps(&p, a, es, plan)) return cudaErrorNotSupported;
  const int threads = 32 + plan.n_groups * (32 + plan.T / 4);  // X producer + per group: producer warp + consumers
#define NB_LAUNCH2(ES, MEAN, TT)                                                                                   \
  do {                                                                                                             \
    if (plan.row_copies == 2) nb_step_pipeline_kernel<ES, MEAN, TT, kGPtrs><<<plan.grid, threads, plan.smem_bytes, st>>>(p);      \
    else if (plan.row_copies == 1) nb_step_pipeline_kernel<ES, MEAN, TT, kGRows><<<plan.grid, threads, plan.smem_bytes, st>>>(p); \
    else nb_step_pipeline_kernel<ES, MEAN, TT, kGBox><<<plan.grid, threads, plan.smem_bytes, st>>>(p);                            \
  } while (0)
#define NB_LAUNCH_XR(ES, MEAN)                                                                                          \
  do {                                                                                                                  \
    if (plan.row_copies == 2) nb_step_pipeline_kernel<ES, MEAN, 512, kGPtrs, true><<<plan.grid, threads, plan.smem_bytes, st>>>(p);      \
    else if (plan.row_copies == 1) nb_step_pipeline_kernel<ES, MEAN, 512, kGRows, true><<<plan.grid, threads, plan.smem_bytes, st>>>(p); \
    else nb_step_pipeline_kernel<ES, MEAN, 512, kGBox, true><<<plan.grid, threads, plan.smem_bytes, st>>>(p);                            \
  } while (0)
#define NB_LAUNCH(ES, MEAN)                                          \
  do {                                                               \
    if (plan.x_in_ring && plan.T == 512) NB_LAUNCH_XR(ES, MEAN);     \
    else if (plan.T == 512) NB_LAUNCH2(ES, MEAN, 512);               \
    else NB_LAUNCH2(ES, MEAN, 0);                                    \
  } while (0)
  if (es == 2) {
    if (a.mean_mode) NB_LAUNCH(2, true);
    else NB_LAUNCH(2, false);
  } else {
    if (a.mean_mode) NB_LAUNCH(4, true);
    else NB_LAUNCH(4, false);
  }
#undef NB_LAUNCH
#undef NB_LAUNCH_XR
#undef NB_LAUNCH2
  return cudaGetLastError();
}

}  // namespace nb
