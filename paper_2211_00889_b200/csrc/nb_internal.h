// Internal declarations shared by the library's translation units (not part of the C ABI).
#pragma once
#include <cstdint>
#include <string>
#include <vector>

#include "nb.h"

#if defined(__CUDACC__)
#define NB_HD __host__ __device__ __forceinline__
#else
#define NB_HD inline
#endif

namespace nb {

// ---------------------------------------------------------------------------------------------
// Counter-based generator: 64 bits addressed by (seed, stream, a, b); four chained rounds of a
// 64-bit finaliser.  The same few lines serve host and device code of the library.
// ---------------------------------------------------------------------------------------------
constexpr uint64_t kGolden = 0x9E3779B97F4A7C15ull;
enum Stream : uint64_t { kInit = 0, kGrad = 1, kStraggler = 2, kMatcha = 3, kGraph = 4, kSlowSet = 5 };

NB_HD uint64_t mix64(uint64_t z) {
  z = (z ^ (z >> 30)) * 0xBF58476D1CE4E5B9ull;
  z = (z ^ (z >> 27)) * 0x94D049BB133111EBull;
  return z ^ (z >> 31);
}
NB_HD uint64_t rng(uint64_t seed, uint64_t stream, uint64_t a, uint64_t b) {
  uint64_t h = mix64(seed + kGolden);
  h = mix64(h + stream + kGolden);
  h = mix64(h + a + kGolden);
  return mix64(h + b + kGolden);
}
// Activation threshold of a Bernoulli(prob) draw on the top 32 bits: active iff (r >> 32) < thr.
NB_HD uint64_t activation_threshold(float prob) {
  double t = (double)prob * 4294967296.0;
  if (t <= 0.0) return 0;
  if (t >= 4294967296.0) return 4294967296ull;
  return (uint64_t)t;
}
// One independent Bernoulli draw per matching per step; thr[j] = activation_threshold(p_j).
NB_HD uint32_t matcha_bits(uint64_t seed, int64_t step, int n_matchings, const uint64_t *thr) {
  uint32_t bits = 0;
  for (int j = 0; j < n_matchings; ++j)
    if ((rng(seed, kMatcha, (uint64_t)step, (uint64_t)j) >> 32) < thr[j]) bits |= (1u << j);
  return bits;
}

// ---------------------------------------------------------------------------------------------
// Host-side description of how learners are combined
// ---------------------------------------------------------------------------------------------
struct Mixing {
  int variant = NB_ALLREDUCE;
  int K = 0;
  // fixed sparse W (NB_DPSGD): CSR
  std::vector<int32_t> row_ptr, col;
  std::vector<float> val;
  // NB_MATCHA
  int n_matchings = 0;
  std::vector<int32_t> partner;  // [n_matchings*K]
  float alpha = 0.f;
  std::vector<float> probs;      // [n_matchings] activation probabilities
  std::vector<uint64_t> thr;     // [n_matchings] activation thresholds
  uint64_t seed = 0;
  int attempts = 0;
};

// Validates (variant, topo, K) and fills `out`.  Returns an nb_status; `err` receives the reason.
int build_mixing(const nb_topology *topo, int variant, int K, Mixing *out, std::string *err);
// Dense W used at `step` (row-major [K*K]) and the activation word (0 unless MATCHA).
void dense_W(const Mixing &mx, int64_t step, float *W, uint32_t *bits);

}  // namespace nb
