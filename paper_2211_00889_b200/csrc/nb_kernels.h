// Device-side data structures and kernel launchers (internal).
#pragma once
#include <cuda_runtime.h>

#include <cstdint>

#include "nb.h"
#include "nb_bounds.h"

namespace nb {

// Sparse mixing matrix in device memory.  Row i owns slots [row_beg[i], row_end[i]).  A fixed W is
// uploaded once; the MATCHA builder kernel rewrites the table every step.
struct MixTable {
  int32_t row_beg[NB_MAX_K];
  int32_t row_end[NB_MAX_K];
  int32_t col[NB_MAX_NNZ];
  float val[NB_MAX_NNZ];
  uint32_t bits;      // MATCHA: activation word of the step the table was built for
  int32_t n_slots;    // slots in use (upper bound of every row_end)
  int32_t pad[2];
};

enum GradSource : int { kSrcF32 = 0, kSrcBF16 = 1, kSrcAcc = 2 };

// Everything one step needs, passed by value as a kernel parameter (no per-step uploads).
struct StepArgs {
  float *X;            // [K, ldx] models (NB_CENTRALIZED: [1, ldx])
  float *V;            // [K, ldx] momentum
  float *acc;          // [K, ldx] accumulator (written by accumulate, read by the unfused step)
  const void *G;       // gradient stream, element (i,m,p) at G[i*ld_k + m*ld_m + p]
  const void *const *row_ptrs;  // or (G == NULL): device table [K*M], row (i,m) is the vector row_ptrs[i*M+m][0..P)
  const MixTable *mix; // sparse W (ignored in mean mode)
  int64_t ldx, ld_m, ld_k, P;
  int64_t row_col0;    // row_ptrs only: the first column of this launch's range inside the held vectors
  int32_t K, M;
  int32_t mix_slots;   // number of table slots to stage in shared memory
  int32_t mean_mode;   // 1: W = (1/K) 1 1^T, computed as one column mean
  int32_t order;       // nb_order
  int32_t g_aligned;   // 1: G base, ld_m, ld_k allow 4-element vector loads
  float lr, mom, inv_K;
  int32_t n[NB_MAX_K]; // finished counts
  float s[NB_MAX_K];   // per-learner scale (1/n_i or n_i/M)
  // bounds-checked build only: where the arrays begin and end, and the word a failed check reports to
  bounds::Extents ext;
  int *err;
};

struct MatchaArgs {
  MixTable *mix;
  const int32_t *partner;  // device [n_matchings*K]
  uint64_t seed;
  uint64_t thr[NB_MAX_MATCHINGS];  // per-matching activation thresholds
  int64_t step;
  int32_t K, n_matchings;
  float alpha;
  int *err;  // bounds-checked build only: where a failed check reports to
};

// Bulk-copy pipeline kernel (nb_pipeline.cu)
struct PipePlan {
  int T, rows_per_item, n_slots, n_groups, smem_bytes, n_tiles, grid;  // all 0: the pipeline kernel did not run
  int head;        // columns [0, head) left to the direct-load kernel (a stream whose start is not 16-byte aligned)
  int row_copies;  // 0: gradient rows travel as tensor-map boxes; 1: one bulk copy per row (rows not 16-byte aligned);
                   // 2: one bulk copy per row from a table of row pointers
  int x_stages;    // buffers of the step kernel's X stage (0 for the kernels that have none)
  bool x_in_ring = false;  // step kernel, update-then-mix on one buffer: old model rows travel in the ring items
  int quads_per_thread = 1;  // groups of four columns per consumer thread (no-stage kernels: 1 or 2)
};
bool plan_pipeline(const StepArgs &a, int es, PipePlan *plan);
bool plan_stream(const StepArgs &a, int es, bool centralized, PipePlan *plan);
cudaError_t launch_stream_pipeline(const StepArgs &a, int es, bool centralized, const PipePlan &plan, int *err_flag,
                                   cudaStream_t st);
cudaError_t configure_pipeline();
cudaError_t launch_wait_selftest(int *err_flag, int code, long long limit_cycles, int *gave_up, cudaStream_t st);
cudaError_t launch_step_pipeline(const StepArgs &a, int es, const PipePlan &plan, int *err_flag, cudaStream_t st);

// The same problem restricted to columns [c0, c0 + cols): every step of the path is independent per
// column, so a column range is a complete problem of its own (es = bytes per gradient element).
StepArgs column_range(const StepArgs &a, int64_t c0, int64_t cols, int es);

int step_threads_per_block(const StepArgs &a);
// Masked accumulate on all P columns (pipeline kernel on the full tiles when it applies).
cudaError_t launch_accumulate(const StepArgs &a, int src, bool pipeline, int *err_flag, int *launches, cudaStream_t st);
cudaError_t launch_accumulate_direct_only(const StepArgs &a, int src, cudaStream_t st);
// Runs the step on all P columns: pipeline kernel on the full tiles when it applies (and `pipeline`
// allows it), direct-load kernel on the rest.  *launches receives the number of kernels launched.
cudaError_t launch_step(const StepArgs &a, int src, bool pipeline, int *err_flag, int *launches, PipePlan *used,
                        cudaStream_t st);
// The direct-load step kernel on all P columns (no pipeline kernel, no device error word).
cudaError_t launch_step_direct_only(const StepArgs &a, int src, cudaStream_t st);
cudaError_t launch_add_minibatch(float *acc_row, const void *g, int src, bool aligned, int64_t P, bool first,
                                 const bounds::Extents &ext, int *err, cudaStream_t st);
cudaError_t launch_centralized(const StepArgs &a, int src, bool pipeline, int *err_flag, int *launches, PipePlan *used,
                               cudaStream_t st);
cudaError_t launch_matcha_build(const MatchaArgs &a, cudaStream_t st);
cudaError_t launch_mean(const float *X, int64_t ldx, int K, int64_t P, float *out, const bounds::Extents &ext, int *err,
                        cudaStream_t st);
cudaError_t configure_kernels();

}  // namespace nb
