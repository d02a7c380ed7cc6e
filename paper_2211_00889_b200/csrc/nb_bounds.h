// Range predicates of the bounds-checked build (-DNB_DEBUG) and the codes a failed check records.
//
// In a debug build every kernel checks, before it touches memory, that the whole footprint it is
// about to form - tile coordinates, ring slots, shared-memory offsets, global addresses of the
// models, the momentum, the accumulator and the caller's gradient stream - lies inside the arrays
// it belongs to.  A failed check SKIPS the access, records its code in the context's device error
// word (first failure wins) and lets the kernel finish; nothing traps or asserts.  The host then
// reports NB_ERR_CUDA at its next look at that word (nb_check_guards, copies to host memory).
// The predicates are plain host/device functions so that a host test can feed them bad indices.
#pragma once
#include <cstdint>

#if defined(__CUDACC__)
#define NB_BOUNDS_HD __host__ __device__ __forceinline__
#else
#define NB_BOUNDS_HD inline
#endif

namespace nb {
namespace bounds {

enum Code : int {
  kOk = 0,
  kStateAddress = 101,     // X, V or acc address outside its array
  kGradientAddress = 102,  // gradient read outside the caller's stream
  kRingSlot = 103,         // ring slot index outside the ring
  kSharedOffset = 104,     // shared-memory offset outside the CTA's allocation
  kTileCoordinate = 105,   // tile index or copy coordinate outside the planned range
  kLearnerIndex = 106      // learner or mixing-table index outside [0, K) / the table
};

// [addr, addr + bytes) inside [lo, hi)
NB_BOUNDS_HD bool span_inside(uintptr_t addr, uint64_t bytes, uintptr_t lo, uintptr_t hi) {
  return addr >= lo && addr <= hi && bytes <= (uint64_t)(hi - addr);
}
// 0 <= index < count
NB_BOUNDS_HD bool index_inside(int64_t index, int64_t count) { return index >= 0 && index < count; }
// the code a kernel records for a footprint check, kOk when it passes
NB_BOUNDS_HD int span_code(uintptr_t addr, uint64_t bytes, uintptr_t lo, uintptr_t hi, int code) {
  return span_inside(addr, bytes, lo, hi) ? kOk : code;
}

// Address ranges of the arrays one launch may touch (filled by the host for every launch).
struct Extents {
  uintptr_t x_lo, x_hi, v_lo, v_hi, acc_lo, acc_hi, g_lo, g_hi;
};

}  // namespace bounds
}  // namespace nb
