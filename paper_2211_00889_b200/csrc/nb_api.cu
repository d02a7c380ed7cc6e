// C ABI of the library: context management, argument validation, launches.  See include/nb.h for
// the contract of every entry point.
#include <cuda_runtime.h>

#include <cstdio>
#include <cstdlib>
#include <cstring>
#include <new>
#include <utility>
#include <string>
#include <vector>

#include "nb_internal.h"
#include "nb_kernels.h"

struct nb_ctx {
  int device = 0;
  int K = 0, M = 0, rows = 0;  // rows = model rows held (K, or 1 for NB_CENTRALIZED)
  int64_t P = 0, ldx = 0;
  float lr = 0.f, mom = 0.f;
  int variant = NB_ALLREDUCE, norm = NB_NORM_MEAN, order = NB_ORDER_MIX_THEN_UPDATE, kernel = NB_KERNEL_AUTO;
  nb::Mixing mx;
  float *X = nullptr, *V = nullptr, *acc = nullptr, *d_mean = nullptr;
  // X, V and acc sit between guard bands (kGuardBytes of a fixed byte pattern before and after);
  // nb_check_guards verifies that no kernel wrote outside its arrays.
  unsigned char *X_base = nullptr, *V_base = nullptr, *acc_base = nullptr;
  size_t model_bytes = 0, acc_bytes = 0;
  nb::MixTable *d_mix = nullptr;
  int32_t *d_partner = nullptr;
  int *d_err = nullptr;  // device word a kernel sets when one of its bounded waits runs out
  void *staging = nullptr;
  size_t staging_bytes = 0;
  // nb_step_fused_host overlaps the copies of one column chunk with the kernels of the previous one
  static constexpr int kHostChunks = 8;
  cudaStream_t s_copy = nullptr, s_out = nullptr;
  cudaEvent_t ev_start = nullptr, ev_h2d[kHostChunks] = {nullptr}, ev_done[kHostChunks] = {nullptr};
  int64_t step = 0;
  bool acc_fresh = false, device_mix_valid = false;
  int32_t n_acc[NB_MAX_K] = {0};
  bool streaming = false, terminal = false;  // nb_begin_iteration / nb_accumulate_minibatch state
  int streaming_mode = NB_STREAMING_ACCUMULATE;
  bool holding = false;                      // this iteration's deliveries were recorded, not accumulated
  int hold_dtype = NB_F32;
  std::vector<const void *> h_rows;          // [K*M] row pointers of the held deliveries (host mirror)
  const void **d_rows = nullptr;             // the same table on the device
  int acc_esize = 4;
  int64_t sum_finished = 0, launches = 0;
  double alg_bytes = 0.0;
  nb::PipePlan last_plan{};  // shape of the pipeline kernel of the most recent step (zeros: not used)
  int sticky = NB_OK;
  std::string err;
};

namespace {

thread_local std::string g_create_err;

constexpr size_t kGuardBytes = 1024;
constexpr int kGuardPattern = 0xA5;

// One array with a guard band on each side; *data is 1024-byte aligned.
cudaError_t alloc_guarded(unsigned char **base, float **data, size_t bytes) {
  cudaError_t e = cudaMalloc(base, bytes + 2 * kGuardBytes);
  if (e != cudaSuccess) return e;
  if ((e = cudaMemset(*base, kGuardPattern, kGuardBytes)) != cudaSuccess) return e;
  if ((e = cudaMemset(*base + kGuardBytes, 0, bytes)) != cudaSuccess) return e;
  if ((e = cudaMemset(*base + kGuardBytes + bytes, kGuardPattern, kGuardBytes)) != cudaSuccess) return e;
  *data = reinterpret_cast<float *>(*base + kGuardBytes);
  return cudaSuccess;
}

struct DeviceGuard {
  int prev = -1;
  bool switched = false;
  explicit DeviceGuard(int dev) {
    if (cudaGetDevice(&prev) == cudaSuccess && prev != dev) switched = cudaSetDevice(dev) == cudaSuccess;
  }
  ~DeviceGuard() {
    if (switched) cudaSetDevice(prev);
  }
};

}  // namespace

namespace nb {
void set_global_error(const std::string &msg) { g_create_err = msg; }
}  // namespace nb

namespace {

int fail(nb_ctx *c, int code, const std::string &msg) {
  if (c) {
    c->err = msg;
    if (code == NB_ERR_CUDA) c->sticky = NB_ERR_CUDA;
  } else {
    g_create_err = msg;
  }
  return code;
}

int cuda_fail(nb_ctx *c, cudaError_t e, const char *what) {
  return fail(c, e == cudaErrorMemoryAllocation ? NB_ERR_NOMEM : NB_ERR_CUDA,
              std::string(what) + ": " + cudaGetErrorString(e));
}

#define NB_CUDA(c, call)                                       \
  do {                                                         \
    cudaError_t e__ = (call);                                  \
    if (e__ != cudaSuccess) return cuda_fail((c), e__, #call); \
  } while (0)

#define NB_ENTER(c)                                                       \
  if (!(c)) return NB_ERR_ARG;                                            \
  if ((c)->sticky != NB_OK) return (c)->sticky;                           \
  DeviceGuard guard__((c)->device)

bool is_device_pointer(const void *p) {
  cudaPointerAttributes at;
  if (cudaPointerGetAttributes(&at, p) != cudaSuccess) {
    cudaGetLastError();
    return false;
  }
  return at.type == cudaMemoryTypeDevice || at.type == cudaMemoryTypeManaged;
}

// Where the context's arrays begin and end (and, when given, the caller's gradient stream): what the
// bounds-checked build compares every address with.
nb::bounds::Extents extents_of(const nb_ctx *c, const void *grads, int64_t ld_m, int64_t ld_k, int es) {
  nb::bounds::Extents e;
  e.x_lo = (uintptr_t)c->X;
  e.x_hi = e.x_lo + c->model_bytes;
  e.v_lo = (uintptr_t)c->V;
  e.v_hi = e.v_lo + c->model_bytes;
  e.acc_lo = (uintptr_t)c->acc;
  e.acc_hi = e.acc_lo + c->acc_bytes;
  e.g_lo = (uintptr_t)grads;
  e.g_hi = grads ? e.g_lo + (size_t)((int64_t)(c->K - 1) * ld_k + (int64_t)(c->M - 1) * ld_m + c->P) * (size_t)es : 0;
  return e;
}

// Validates the gradient-stream description and the finished counts; fills the step arguments.
int fill_step_args(nb_ctx *c, const void *grads, int dtype, int64_t ld_m, int64_t ld_k, const int32_t *finished,
                   nb::StepArgs *a, int *esize) {
  if (!grads) return fail(c, NB_ERR_ARG, "grads is NULL");
  if (!finished) return fail(c, NB_ERR_ARG, "finished is NULL");
  if (dtype != NB_F32 && dtype != NB_BF16) return fail(c, NB_ERR_ARG, "dtype must be NB_F32 or NB_BF16");
  const int es = dtype == NB_F32 ? 4 : 2;
  if (ld_m == 0) ld_m = c->P;
  if (ld_k == 0) ld_k = (int64_t)c->M * ld_m;
  if ((uintptr_t)grads % (size_t)es != 0) return fail(c, NB_ERR_ARG, "grads is not aligned to its element size");
  if (ld_m < c->P) return fail(c, NB_ERR_ARG, "ld_m is smaller than P");
  if (ld_k < (int64_t)(c->M - 1) * ld_m + c->P) return fail(c, NB_ERR_ARG, "ld_k is too small for M rows of pitch ld_m");
  for (int i = 0; i < c->K; ++i) {
    if (finished[i] < 0 || finished[i] > c->M)
      return fail(c, NB_ERR_ARG, "finished[" + std::to_string(i) + "] is outside [0, M]");
  }
  std::memset(a, 0, sizeof(*a));
  a->X = c->X;
  a->V = c->V;
  a->acc = c->acc;
  a->G = grads;
  a->mix = c->d_mix;
  a->ldx = c->ldx;
  a->ld_m = ld_m;
  a->ld_k = ld_k;
  a->P = c->P;
  a->K = c->K;
  a->M = c->M;
  a->g_aligned = ((uintptr_t)grads % (size_t)(4 * es) == 0) && (ld_m % 4 == 0) && (ld_k % 4 == 0);
  for (int i = 0; i < c->K; ++i) a->n[i] = finished[i];
  a->ext = extents_of(c, grads, ld_m, ld_k, es);
  a->err = c->d_err;
  *esize = es;
  return NB_OK;
}

// Scalars, scale factors and mixing mode: the part of the arguments the step (not the accumulate) needs.
void fill_update_args(nb_ctx *c, nb::StepArgs *a) {
  a->lr = c->lr;
  a->mom = c->mom;
  a->inv_K = 1.0f / (float)c->K;
  a->order = c->order;
  a->mean_mode = (c->variant == NB_ALLREDUCE) ? 1 : 0;
  a->mix_slots = 0;
  if (c->variant == NB_DPSGD) a->mix_slots = (int32_t)c->mx.col.size();
  if (c->variant == NB_MATCHA) a->mix_slots = c->K * (1 + c->mx.n_matchings);
  for (int i = 0; i < c->K; ++i) {
    const int n = a->n[i];
    if (c->norm == NB_NORM_MEAN) a->s[i] = n > 0 ? 1.0f / (float)n : 0.0f;
    else a->s[i] = (float)n / (float)c->M;
  }
}

void record_stats(nb_ctx *c, const nb::StepArgs &a, int esize) {
  int64_t sum = 0;
  for (int i = 0; i < c->K; ++i) sum += a.n[i];
  c->sum_finished = sum;
  c->alg_bytes = (double)c->P * ((double)esize * (double)sum + 16.0 * (double)c->rows);
}

// MATCHA: rebuild W on the device for the current step (K3), ahead of the step kernel in `st`.
int build_device_mixing(nb_ctx *c, cudaStream_t st) {
  if (c->variant != NB_MATCHA) return NB_OK;
  nb::MatchaArgs m;
  m.mix = c->d_mix;
  m.partner = c->d_partner;
  m.seed = c->mx.seed;
  for (int j = 0; j < c->mx.n_matchings; ++j) m.thr[j] = c->mx.thr[j];
  m.step = c->step;
  m.K = c->K;
  m.n_matchings = c->mx.n_matchings;
  m.alpha = c->mx.alpha;
  m.err = c->d_err;
  NB_CUDA(c, nb::launch_matcha_build(m, st));
  c->launches++;
  c->device_mix_valid = true;
  return NB_OK;
}

// The step kernels on the columns `a` describes (all of them, or one chunk); the mixing matrix of
// the current step must already be on the device.
int launch_update(nb_ctx *c, const nb::StepArgs &a, int src, cudaStream_t st) {
  int n_launched = 0;
  const bool pipeline = c->kernel == NB_KERNEL_AUTO;
  cudaError_t e;
  if (c->variant == NB_CENTRALIZED) e = nb::launch_centralized(a, src, pipeline, c->d_err, &n_launched, &c->last_plan, st);
  else e = nb::launch_step(a, src, pipeline, c->d_err, &n_launched, &c->last_plan, st);
  c->launches += n_launched;
  if (e != cudaSuccess) return cuda_fail(c, e, "launch_step");
  return NB_OK;
}

int run_update(nb_ctx *c, nb::StepArgs *a, int src, cudaStream_t st) {
  fill_update_args(c, a);
  int rc = build_device_mixing(c, st);
  if (rc != NB_OK) return rc;
  rc = launch_update(c, *a, src, st);
  if (rc != NB_OK) return rc;
  c->step++;
  c->acc_fresh = false;
  return NB_OK;
}

// Reads the device error word (the stream is drained first).  A kernel sets it when one of its
// bounded waits ran out; that is a defect, reported as a sticky NB_ERR_CUDA.
int check_device_error(nb_ctx *c, cudaStream_t st) {
  int h = 0;
  NB_CUDA(c, cudaMemcpyAsync(&h, c->d_err, sizeof(int), cudaMemcpyDeviceToHost, st));
  NB_CUDA(c, cudaStreamSynchronize(st));
  if (h != 0) return fail(c, NB_ERR_CUDA, "device-side wait timed out (code " + std::to_string(h) + ")");
  return NB_OK;
}

// dense [rows, P] <-> pitched [rows, ldx]
int copy_rows_out(nb_ctx *c, float *dst, const float *src, int rows, cudaStream_t st) {
  if (!dst) return fail(c, NB_ERR_ARG, "dst is NULL");
  for (int r = 0; r < rows; ++r)
    NB_CUDA(c, cudaMemcpyAsync(dst + (int64_t)r * c->P, src + (int64_t)r * c->ldx, sizeof(float) * (size_t)c->P,
                               cudaMemcpyDefault, st));
  if (!is_device_pointer(dst)) return check_device_error(c, st);
  return NB_OK;
}
int copy_rows_in(nb_ctx *c, float *dst, const float *src, int rows, cudaStream_t st) {
  for (int r = 0; r < rows; ++r)
    NB_CUDA(c, cudaMemcpyAsync(dst + (int64_t)r * c->ldx, src + (int64_t)r * c->P, sizeof(float) * (size_t)c->P,
                               cudaMemcpyDefault, st));
  if (!is_device_pointer(src)) NB_CUDA(c, cudaStreamSynchronize(st));
  return NB_OK;
}

}  // namespace

extern "C" {

const char *nb_last_error(const nb_ctx *c) { return c ? c->err.c_str() : g_create_err.c_str(); }

int nb_create(nb_ctx **out, int K, int64_t P, int M, float lr, float mom, int variant, const nb_topology *topo) {
  if (!out) return NB_ERR_ARG;
  *out = nullptr;
  if (K < 1) return fail(nullptr, NB_ERR_ARG, "K must be >= 1");
  if (P < 1) return fail(nullptr, NB_ERR_ARG, "P must be >= 1");
  if (M < 1) return fail(nullptr, NB_ERR_ARG, "M must be >= 1");
  if (variant < NB_ALLREDUCE || variant > NB_CENTRALIZED) return fail(nullptr, NB_ERR_ARG, "unknown variant");
  nb::Mixing mx;
  std::string err;
  int rc = nb::build_mixing(topo, variant, K, &mx, &err);
  if (rc != NB_OK) return fail(nullptr, rc, err);

  nb_ctx *c = new (std::nothrow) nb_ctx;
  if (!c) return fail(nullptr, NB_ERR_NOMEM, "host allocation failed");
  c->K = K;
  c->P = P;
  c->M = M;
  c->lr = lr;
  c->mom = mom;
  c->variant = variant;
  c->rows = variant == NB_CENTRALIZED ? 1 : K;
  // Row pitch of X, V and acc: a multiple of the 512-column tile (2 KB), so that every row segment a
  // tile copies starts on a 2 KB boundary (measured: 2-3 % more bandwidth than 128-byte multiples).
  c->ldx = (P + 511) / 512 * 512;
#ifdef NB_TUNING
  if (const char *pad = std::getenv("NB_LDX_PAD")) c->ldx += 512 * (int64_t)std::atoi(pad);  // sweeps of the row pitch
#endif
  c->mx = mx;

  auto bail = [&](cudaError_t e, const char *what) {
    int code = cuda_fail(nullptr, e, what);
    cudaGetLastError();
    nb_destroy(c);
    return code;
  };
  cudaError_t e;
  if ((e = cudaGetDevice(&c->device)) != cudaSuccess) return bail(e, "cudaGetDevice");
  if ((e = nb::configure_kernels()) != cudaSuccess) return bail(e, "cudaFuncSetAttribute");
  const size_t model_bytes = sizeof(float) * (size_t)c->rows * (size_t)c->ldx;
  const size_t acc_bytes = sizeof(float) * (size_t)K * (size_t)c->ldx;
  c->model_bytes = model_bytes;
  c->acc_bytes = acc_bytes;
  if ((e = alloc_guarded(&c->X_base, &c->X, model_bytes)) != cudaSuccess) return bail(e, "cudaMalloc(X)");
  if ((e = alloc_guarded(&c->V_base, &c->V, model_bytes)) != cudaSuccess) return bail(e, "cudaMalloc(V)");
  if ((e = alloc_guarded(&c->acc_base, &c->acc, acc_bytes)) != cudaSuccess) return bail(e, "cudaMalloc(acc)");
  if ((e = cudaMalloc(&c->d_err, 2 * sizeof(int))) != cudaSuccess) return bail(e, "cudaMalloc(err)");
  if ((e = cudaMemset(c->d_err, 0, 2 * sizeof(int))) != cudaSuccess) return bail(e, "cudaMemset(err)");
  if (variant == NB_DPSGD || variant == NB_MATCHA) {
    if ((e = cudaMalloc(&c->d_mix, sizeof(nb::MixTable))) != cudaSuccess) return bail(e, "cudaMalloc(mix)");
    nb::MixTable *h = new (std::nothrow) nb::MixTable;
    if (!h) { nb_destroy(c); return fail(nullptr, NB_ERR_NOMEM, "host allocation failed"); }
    std::memset(h, 0, sizeof(*h));
    if (variant == NB_DPSGD) {
      for (int i = 0; i < K; ++i) { h->row_beg[i] = mx.row_ptr[i]; h->row_end[i] = mx.row_ptr[i + 1]; }
      for (size_t q = 0; q < mx.col.size(); ++q) { h->col[q] = mx.col[q]; h->val[q] = mx.val[q]; }
      h->n_slots = (int32_t)mx.col.size();
    }
    e = cudaMemcpy(c->d_mix, h, sizeof(*h), cudaMemcpyHostToDevice);
    delete h;
    if (e != cudaSuccess) return bail(e, "cudaMemcpy(mix)");
  }
  if (variant == NB_MATCHA && mx.n_matchings > 0) {
    const size_t pb = sizeof(int32_t) * mx.partner.size();
    if ((e = cudaMalloc(&c->d_partner, pb)) != cudaSuccess) return bail(e, "cudaMalloc(partner)");
    if ((e = cudaMemcpy(c->d_partner, mx.partner.data(), pb, cudaMemcpyHostToDevice)) != cudaSuccess)
      return bail(e, "cudaMemcpy(partner)");
  }
  *out = c;
  return NB_OK;
}

int nb_destroy(nb_ctx *c) {
  if (!c) return NB_OK;
  DeviceGuard guard(c->device);
  cudaDeviceSynchronize();
  cudaFree(c->X_base);
  cudaFree(c->V_base);
  cudaFree(c->acc_base);
  cudaFree(c->d_mean);
  cudaFree(c->d_mix);
  cudaFree(c->d_partner);
  cudaFree(c->d_err);
  cudaFree(c->d_rows);
  cudaFree(c->staging);
  if (c->s_copy) cudaStreamDestroy(c->s_copy);
  if (c->s_out) cudaStreamDestroy(c->s_out);
  if (c->ev_start) cudaEventDestroy(c->ev_start);
  for (int q = 0; q < nb_ctx::kHostChunks; ++q) {
    if (c->ev_h2d[q]) cudaEventDestroy(c->ev_h2d[q]);
    if (c->ev_done[q]) cudaEventDestroy(c->ev_done[q]);
  }
  cudaGetLastError();
  delete c;
  return NB_OK;
}

int nb_set_option(nb_ctx *c, int key, int64_t value) {
  NB_ENTER(c);
  if (key == NB_OPT_NORM) {
    if (value != NB_NORM_MEAN && value != NB_NORM_PAPER) return fail(c, NB_ERR_ARG, "unknown norm");
    c->norm = (int)value;
    return NB_OK;
  }
  if (key == NB_OPT_ORDER) {
    if (value != NB_ORDER_MIX_THEN_UPDATE && value != NB_ORDER_UPDATE_THEN_MIX) return fail(c, NB_ERR_ARG, "unknown order");
    c->order = (int)value;
    return NB_OK;
  }
  if (key == NB_OPT_STREAMING) {
    if (value != NB_STREAMING_ACCUMULATE && value != NB_STREAMING_HOLD) return fail(c, NB_ERR_ARG, "unknown streaming mode");
    if (c->streaming) return fail(c, NB_ERR_STATE, "the streaming mode cannot change inside an iteration");
    c->streaming_mode = (int)value;
    return NB_OK;
  }
  if (key == NB_OPT_KERNEL) {
    if (value != NB_KERNEL_AUTO && value != NB_KERNEL_DIRECT) return fail(c, NB_ERR_ARG, "unknown kernel choice");
    c->kernel = (int)value;
    return NB_OK;
  }
  return fail(c, NB_ERR_ARG, "unknown option key");
}

int nb_set_lr(nb_ctx *c, float lr) {
  NB_ENTER(c);
  c->lr = lr;
  return NB_OK;
}

int nb_set_params(nb_ctx *c, const float *x0, int per_learner, void *stream) {
  NB_ENTER(c);
  cudaStream_t st = (cudaStream_t)stream;
  if (!x0) return fail(c, NB_ERR_ARG, "x0 is NULL");
  if (per_learner != 0 && per_learner != 1) return fail(c, NB_ERR_ARG, "per_learner must be 0 or 1");
  if (per_learner && c->variant == NB_CENTRALIZED) return fail(c, NB_ERR_ARG, "NB_CENTRALIZED holds one model");
  if (per_learner) {
    int rc = copy_rows_in(c, c->X, x0, c->rows, st);
    if (rc != NB_OK) return rc;
  } else {
    int rc = copy_rows_in(c, c->X, x0, 1, st);
    if (rc != NB_OK) return rc;
    for (int r = 1; r < c->rows; ++r)
      NB_CUDA(c, cudaMemcpyAsync(c->X + (int64_t)r * c->ldx, c->X, sizeof(float) * (size_t)c->P, cudaMemcpyDeviceToDevice, st));
  }
  NB_CUDA(c, cudaMemsetAsync(c->V, 0, sizeof(float) * (size_t)c->rows * (size_t)c->ldx, st));
  c->step = 0;
  c->acc_fresh = false;
  return NB_OK;
}

int nb_accumulate(nb_ctx *c, const void *grads, int dtype, int64_t ld_m, int64_t ld_k, const int32_t *finished,
                  void *stream) {
  NB_ENTER(c);
  nb::StepArgs a;
  int es = 4;
  int rc = fill_step_args(c, grads, dtype, ld_m, ld_k, finished, &a, &es);
  if (rc != NB_OK) return rc;
  int n_launched = 0;
  cudaError_t e = nb::launch_accumulate(a, dtype == NB_F32 ? nb::kSrcF32 : nb::kSrcBF16, c->kernel == NB_KERNEL_AUTO,
                                        c->d_err, &n_launched, (cudaStream_t)stream);
  c->launches += n_launched;
  if (e != cudaSuccess) return cuda_fail(c, e, "launch_accumulate");
  std::memcpy(c->n_acc, a.n, sizeof(c->n_acc));
  c->acc_esize = es;
  c->acc_fresh = true;
  c->streaming = false;
  return NB_OK;
}

int nb_begin_iteration(nb_ctx *c) {
  NB_ENTER(c);
  std::memset(c->n_acc, 0, sizeof(c->n_acc));
  c->streaming = true;
  c->terminal = false;
  c->acc_fresh = true;
  c->acc_esize = 4;
  c->holding = c->streaming_mode == NB_STREAMING_HOLD;
  if (c->holding) {
    c->h_rows.assign((size_t)c->K * (size_t)c->M, nullptr);
    if (!c->d_rows) NB_CUDA(c, cudaMalloc(&c->d_rows, sizeof(void *) * (size_t)c->K * (size_t)c->M));
  }
  return NB_OK;
}

int nb_accumulate_minibatch(nb_ctx *c, int learner, const void *grad, int dtype, void *stream) {
  NB_ENTER(c);
  if (!c->streaming) return fail(c, NB_ERR_STATE, "nb_accumulate_minibatch needs nb_begin_iteration first");
  if (learner < 0 || learner >= c->K) return fail(c, NB_ERR_ARG, "learner index out of range");
  if (!grad) return fail(c, NB_ERR_ARG, "grad is NULL");
  if (dtype != NB_F32 && dtype != NB_BF16) return fail(c, NB_ERR_ARG, "dtype must be NB_F32 or NB_BF16");
  if (c->terminal) return NB_ABANDONED;  // the first finisher has ended the iteration
  const int es = dtype == NB_F32 ? 4 : 2;
  const bool aligned = (uintptr_t)grad % (size_t)(4 * es) == 0;
  if ((uintptr_t)grad % (size_t)es != 0) return fail(c, NB_ERR_ARG, "grad is not aligned to its element size");
  if (c->holding) {  // record the vector; nb_step reads it in place
    if ((uintptr_t)grad % 16 != 0) return fail(c, NB_ERR_ARG, "NB_STREAMING_HOLD needs 16-byte aligned gradient vectors");
    bool first = true;
    for (int i = 0; i < c->K; ++i) first = first && c->n_acc[i] == 0;
    if (first) c->hold_dtype = dtype;
    else if (dtype != c->hold_dtype) return fail(c, NB_ERR_ARG, "NB_STREAMING_HOLD needs one dtype per iteration");
    c->h_rows[(size_t)learner * (size_t)c->M + (size_t)c->n_acc[learner]] = grad;
    c->acc_esize = es;
    if (++c->n_acc[learner] == c->M) c->terminal = true;
    return NB_OK;
  }
  NB_CUDA(c, nb::launch_add_minibatch(c->acc + (int64_t)learner * c->ldx, grad, dtype == NB_F32 ? nb::kSrcF32 : nb::kSrcBF16,
                                      aligned, c->P, c->n_acc[learner] == 0, extents_of(c, nullptr, 0, 0, es), c->d_err,
                                      (cudaStream_t)stream));
  c->launches++;
  c->acc_esize = es;
  if (++c->n_acc[learner] == c->M) c->terminal = true;
  return NB_OK;
}

int nb_get_finished(const nb_ctx *c, int32_t *finished, int32_t *terminal) {
  if (!c || !finished) return NB_ERR_ARG;
  for (int i = 0; i < c->K; ++i) finished[i] = c->n_acc[i];
  if (terminal) *terminal = c->terminal ? 1 : 0;
  return NB_OK;
}

int nb_step(nb_ctx *c, void *stream) {
  NB_ENTER(c);
  if (!c->acc_fresh) return fail(c, NB_ERR_STATE, "nb_step needs an nb_accumulate since the last step");
  nb::StepArgs a;
  std::memset(&a, 0, sizeof(a));
  a.X = c->X;
  a.V = c->V;
  a.acc = c->acc;
  a.mix = c->d_mix;
  a.ldx = c->ldx;
  a.P = c->P;
  a.K = c->K;
  a.M = c->M;
  a.g_aligned = 1;
  a.ext = extents_of(c, nullptr, 0, 0, 4);
  a.err = c->d_err;
  std::memcpy(a.n, c->n_acc, sizeof(a.n));
  record_stats(c, a, c->acc_esize);
  if (c->streaming && c->holding) {
    // the recorded vectors are the gradient stream: the fused step reads them where they lie
    NB_CUDA(c, cudaMemcpyAsync(c->d_rows, c->h_rows.data(), sizeof(void *) * c->h_rows.size(), cudaMemcpyHostToDevice,
                               (cudaStream_t)stream));
    c->streaming = false;
    c->holding = false;
    a.row_ptrs = c->d_rows;
    // (g_aligned stays 1: the vectors are 16-byte aligned and every thread starts at a multiple of 4 columns)
    return run_update(c, &a, c->hold_dtype == NB_F32 ? nb::kSrcF32 : nb::kSrcBF16, (cudaStream_t)stream);
  }
  if (c->streaming) {  // learners that delivered nothing contribute a zero accumulator
    for (int i = 0; i < c->K; ++i)
      if (c->n_acc[i] == 0)
        NB_CUDA(c, cudaMemsetAsync(c->acc + (int64_t)i * c->ldx, 0, sizeof(float) * (size_t)c->ldx, (cudaStream_t)stream));
    c->streaming = false;
  }
  return run_update(c, &a, nb::kSrcAcc, (cudaStream_t)stream);
}

int nb_step_fused(nb_ctx *c, const void *grads, int dtype, int64_t ld_m, int64_t ld_k, const int32_t *finished,
                  void *stream) {
  NB_ENTER(c);
  nb::StepArgs a;
  int es = 4;
  int rc = fill_step_args(c, grads, dtype, ld_m, ld_k, finished, &a, &es);
  if (rc != NB_OK) return rc;
  record_stats(c, a, es);
  return run_update(c, &a, dtype == NB_F32 ? nb::kSrcF32 : nb::kSrcBF16, (cudaStream_t)stream);
}

int nb_step_fused_host(nb_ctx *c, const void *grads_host, int dtype, int64_t ld_m, int64_t ld_k,
                       const int32_t *finished, float *mean_out, void *stream) {
  NB_ENTER(c);
  cudaStream_t st = (cudaStream_t)stream;
  if (!grads_host) return fail(c, NB_ERR_ARG, "grads_host is NULL");
  if (!finished) return fail(c, NB_ERR_ARG, "finished is NULL");
  if (dtype != NB_F32 && dtype != NB_BF16) return fail(c, NB_ERR_ARG, "dtype must be NB_F32 or NB_BF16");
  const size_t es = dtype == NB_F32 ? 4 : 2;
  if (ld_m == 0) ld_m = c->P;
  if (ld_k == 0) ld_k = (int64_t)c->M * ld_m;
  if ((uintptr_t)grads_host % es != 0) return fail(c, NB_ERR_ARG, "grads_host is not aligned to its element size");
  if (ld_m < c->P) return fail(c, NB_ERR_ARG, "ld_m is smaller than P");
  if (ld_k < (int64_t)(c->M - 1) * ld_m + c->P) return fail(c, NB_ERR_ARG, "ld_k is too small for M rows of pitch ld_m");
  for (int i = 0; i < c->K; ++i)
    if (finished[i] < 0 || finished[i] > c->M) return fail(c, NB_ERR_ARG, "finished count outside [0, M]");
  const int64_t ldg = (c->P + 511) / 512 * 512;  // staging pitch, elements: rows start on 2 KB boundaries
  const size_t need = (size_t)c->K * (size_t)c->M * (size_t)ldg * es;
  if (c->staging_bytes < need) {
    NB_CUDA(c, cudaStreamSynchronize(st));
    cudaFree(c->staging);
    c->staging = nullptr;
    c->staging_bytes = 0;
    NB_CUDA(c, cudaMalloc(&c->staging, need));
    c->staging_bytes = need;
  }
  if (mean_out && !c->d_mean) NB_CUDA(c, cudaMalloc(&c->d_mean, sizeof(float) * (size_t)c->P));
  if (!c->s_copy) {
    NB_CUDA(c, cudaStreamCreateWithFlags(&c->s_copy, cudaStreamNonBlocking));
    NB_CUDA(c, cudaStreamCreateWithFlags(&c->s_out, cudaStreamNonBlocking));
    NB_CUDA(c, cudaEventCreateWithFlags(&c->ev_start, cudaEventDisableTiming));
    for (int q = 0; q < nb_ctx::kHostChunks; ++q) {
      NB_CUDA(c, cudaEventCreateWithFlags(&c->ev_h2d[q], cudaEventDisableTiming));
      NB_CUDA(c, cudaEventCreateWithFlags(&c->ev_done[q], cudaEventDisableTiming));
    }
  }
  nb::StepArgs a;
  int esz = 4;
  int rc = fill_step_args(c, c->staging, dtype, ldg, (int64_t)c->M * ldg, finished, &a, &esz);
  if (rc != NB_OK) return rc;
  record_stats(c, a, esz);
  fill_update_args(c, &a);
  rc = build_device_mixing(c, st);
  if (rc != NB_OK) return rc;
  const int src_kind = dtype == NB_F32 ? nb::kSrcF32 : nb::kSrcBF16;
  // Column chunks (multiples of the 512-column tile, at least 64K columns each): the copy stream
  // brings chunk q+1 over the bus while `stream` runs the kernels of chunk q and the output stream
  // returns chunk q-1's mean model; the three directions overlap because columns are independent.
  int n_chunks = (int)(c->P / 65536);
  if (n_chunks > nb_ctx::kHostChunks) n_chunks = nb_ctx::kHostChunks;
  if (n_chunks < 1) n_chunks = 1;
  const int64_t per_chunk = ((c->P / n_chunks) + 511) / 512 * 512;
  NB_CUDA(c, cudaEventRecord(c->ev_start, st));
  NB_CUDA(c, cudaStreamWaitEvent(c->s_copy, c->ev_start, 0));  // the staging buffer is free once `stream` got here
  for (int q = 0; q < n_chunks; ++q) {
    const int64_t c0 = (int64_t)q * per_chunk;
    const int64_t cols = (q == n_chunks - 1) ? c->P - c0 : per_chunk;
    if (cols <= 0) break;
    // only the finished mini-batches cross the bus: the abandoned ones are never needed.  One
    // pitched copy per learner moves its n_i row segments (row by row when the pitch is too large).
    for (int i = 0; i < c->K; ++i) {
      if (finished[i] == 0) continue;
      const char *src = (const char *)grads_host + ((size_t)i * (size_t)ld_k + (size_t)c0) * es;
      char *dst = (char *)c->staging + ((size_t)i * (size_t)c->M * (size_t)ldg + (size_t)c0) * es;
      const size_t spitch = (size_t)ld_m * es, dpitch = (size_t)ldg * es;
      if (spitch < (size_t)2147483647 && dpitch < (size_t)2147483647) {
        NB_CUDA(c, cudaMemcpy2DAsync(dst, dpitch, src, spitch, (size_t)cols * es, (size_t)finished[i],
                                     cudaMemcpyHostToDevice, c->s_copy));
      } else {
        for (int m = 0; m < finished[i]; ++m)
          NB_CUDA(c, cudaMemcpyAsync(dst + (size_t)m * dpitch, src + (size_t)m * spitch, (size_t)cols * es,
                                     cudaMemcpyHostToDevice, c->s_copy));
      }
    }
    NB_CUDA(c, cudaEventRecord(c->ev_h2d[q], c->s_copy));
    NB_CUDA(c, cudaStreamWaitEvent(st, c->ev_h2d[q], 0));
    rc = launch_update(c, nb::column_range(a, c0, cols, esz), src_kind, st);
    if (rc != NB_OK) return rc;
    if (mean_out) {
      NB_CUDA(c, nb::launch_mean(c->X + c0, c->ldx, c->rows, cols, c->d_mean + c0, a.ext, c->d_err, st));
      c->launches++;
      NB_CUDA(c, cudaEventRecord(c->ev_done[q], st));
      NB_CUDA(c, cudaStreamWaitEvent(c->s_out, c->ev_done[q], 0));
      NB_CUDA(c, cudaMemcpyAsync(mean_out + c0, c->d_mean + c0, sizeof(float) * (size_t)cols, cudaMemcpyDeviceToHost, c->s_out));
    }
  }
  c->step++;
  c->acc_fresh = false;
  NB_CUDA(c, cudaStreamSynchronize(c->s_out));
  return check_device_error(c, st);
}

int nb_get_params(nb_ctx *c, float *dst, void *stream) {
  NB_ENTER(c);
  return copy_rows_out(c, dst, c->X, c->rows, (cudaStream_t)stream);
}

int nb_get_momentum(nb_ctx *c, float *dst, void *stream) {
  NB_ENTER(c);
  return copy_rows_out(c, dst, c->V, c->rows, (cudaStream_t)stream);
}

int nb_get_accumulator(nb_ctx *c, float *dst, void *stream) {
  NB_ENTER(c);
  return copy_rows_out(c, dst, c->acc, c->K, (cudaStream_t)stream);
}

int nb_get_mean_params(nb_ctx *c, float *dst, void *stream) {
  NB_ENTER(c);
  cudaStream_t st = (cudaStream_t)stream;
  if (!dst) return fail(c, NB_ERR_ARG, "dst is NULL");
  const bool dev = is_device_pointer(dst);
  float *out = dst;
  if (!dev) {
    if (!c->d_mean) NB_CUDA(c, cudaMalloc(&c->d_mean, sizeof(float) * (size_t)c->P));
    out = c->d_mean;
  }
  NB_CUDA(c, nb::launch_mean(c->X, c->ldx, c->rows, c->P, out, extents_of(c, nullptr, 0, 0, 4), c->d_err, st));
  c->launches++;
  if (!dev) {
    NB_CUDA(c, cudaMemcpyAsync(dst, out, sizeof(float) * (size_t)c->P, cudaMemcpyDeviceToHost, st));
    return check_device_error(c, st);
  }
  return NB_OK;
}

int nb_set_state(nb_ctx *c, int64_t step, const float *X, const float *V, void *stream) {
  NB_ENTER(c);
  if (step < 0 || !X || !V) return fail(c, NB_ERR_ARG, "nb_set_state: step >= 0 and X, V required");
  int rc = copy_rows_in(c, c->X, X, c->rows, (cudaStream_t)stream);
  if (rc != NB_OK) return rc;
  rc = copy_rows_in(c, c->V, V, c->rows, (cudaStream_t)stream);
  if (rc != NB_OK) return rc;
  c->step = step;
  c->acc_fresh = false;
  return NB_OK;
}

int nb_get_step(const nb_ctx *c, int64_t *step) {
  if (!c || !step) return NB_ERR_ARG;
  *step = c->step;
  return NB_OK;
}

int nb_get_W(nb_ctx *c, int64_t step, float *W_dense) {
  if (!c) return NB_ERR_ARG;
  if (!W_dense || step < 0) return fail(c, NB_ERR_ARG, "nb_get_W: W_dense and step >= 0 required");
  nb::dense_W(c->mx, step, W_dense, nullptr);
  return NB_OK;
}

int nb_get_matcha_activation(nb_ctx *c, int64_t step, uint32_t *bits) {
  if (!c) return NB_ERR_ARG;
  if (!bits || step < 0) return fail(c, NB_ERR_ARG, "bits and step >= 0 required");
  if (c->variant != NB_MATCHA) return fail(c, NB_ERR_STATE, "not a MATCHA context");
  *bits = nb::matcha_bits(c->mx.seed, step, c->mx.n_matchings, c->mx.thr.data());
  return NB_OK;
}

int nb_get_device_mixing(nb_ctx *c, uint32_t *bits, float *W_dense, void *stream) {
  NB_ENTER(c);
  if (c->variant != NB_MATCHA) return fail(c, NB_ERR_STATE, "not a MATCHA context");
  if (!c->device_mix_valid) return fail(c, NB_ERR_STATE, "no step has run yet");
  nb::MixTable *h = new (std::nothrow) nb::MixTable;
  if (!h) return fail(c, NB_ERR_NOMEM, "host allocation failed");
  cudaError_t e = cudaMemcpyAsync(h, c->d_mix, sizeof(*h), cudaMemcpyDeviceToHost, (cudaStream_t)stream);
  if (e == cudaSuccess) e = cudaStreamSynchronize((cudaStream_t)stream);
  if (e != cudaSuccess) {
    delete h;
    return cuda_fail(c, e, "cudaMemcpyAsync(mix)");
  }
  if (bits) *bits = h->bits;
  if (W_dense) {
    const int K = c->K;
    for (size_t q = 0; q < (size_t)K * K; ++q) W_dense[q] = 0.f;
    for (int i = 0; i < K; ++i)
      for (int e2 = h->row_beg[i]; e2 < h->row_end[i]; ++e2)
        if (e2 >= 0 && e2 < NB_MAX_NNZ && h->col[e2] >= 0 && h->col[e2] < K) W_dense[(size_t)i * K + h->col[e2]] += h->val[e2];
  }
  delete h;
  return NB_OK;
}

int nb_check_guards(nb_ctx *c, void *stream) {
  NB_ENTER(c);
  cudaStream_t st = (cudaStream_t)stream;
  unsigned char h[2 * kGuardBytes];
  struct Arr { const char *name; unsigned char *base; size_t bytes; };
  const Arr arrs[3] = {{"X", c->X_base, c->model_bytes}, {"V", c->V_base, c->model_bytes}, {"acc", c->acc_base, c->acc_bytes}};
  for (const Arr &a : arrs) {
    if (!a.base) continue;
    NB_CUDA(c, cudaMemcpyAsync(h, a.base, kGuardBytes, cudaMemcpyDeviceToHost, st));
    NB_CUDA(c, cudaMemcpyAsync(h + kGuardBytes, a.base + kGuardBytes + a.bytes, kGuardBytes, cudaMemcpyDeviceToHost, st));
    NB_CUDA(c, cudaStreamSynchronize(st));
    for (size_t q = 0; q < 2 * kGuardBytes; ++q)
      if (h[q] != kGuardPattern)
        return fail(c, NB_ERR_STATE, std::string("guard band of ") + a.name + " overwritten at byte " +
                                         std::to_string(q < kGuardBytes ? (long long)q - (long long)kGuardBytes
                                                                        : (long long)(q - kGuardBytes)) +
                                         (q < kGuardBytes ? " before the array" : " after the array"));
  }
  return check_device_error(c, st);
}

int nb_selftest_wait_timeout(nb_ctx *c, void *stream) {
  NB_ENTER(c);
  cudaStream_t st = (cudaStream_t)stream;
  int rc = check_device_error(c, st);  // start from a clean error word
  if (rc != NB_OK) return rc;
  int *gave_up = c->d_err + 1;
  NB_CUDA(c, cudaMemsetAsync(gave_up, 0, sizeof(int), st));
  NB_CUDA(c, nb::launch_wait_selftest(c->d_err, 9, 2000000ll /* ~1 ms */, gave_up, st));
  c->launches++;
  int h[2] = {0, 0};
  NB_CUDA(c, cudaMemcpyAsync(h, c->d_err, 2 * sizeof(int), cudaMemcpyDeviceToHost, st));
  NB_CUDA(c, cudaStreamSynchronize(st));
  // the wait must have run out in every lane and reported its code; then the word is cleared again
  NB_CUDA(c, cudaMemsetAsync(c->d_err, 0, 2 * sizeof(int), st));
  NB_CUDA(c, cudaStreamSynchronize(st));
  if (h[0] != 9 || h[1] != 32)
    return fail(c, NB_ERR_STATE, "wait self-test: error word " + std::to_string(h[0]) + ", lanes that gave up " + std::to_string(h[1]));
  return NB_OK;
}

int64_t nb_recommended_pitch(int64_t P, int dtype) {
  if (P < 1 || (dtype != NB_F32 && dtype != NB_BF16)) return 0;
  const int64_t per_block = 2048 / (dtype == NB_F32 ? 4 : 2);
  return (P + per_block - 1) / per_block * per_block;
}

int nb_debug_build(void) {
#ifdef NB_DEBUG
  return 1;
#else
  return 0;
#endif
}

int nb_debug_span_code(uint64_t addr, uint64_t bytes, uint64_t lo, uint64_t hi) {
  return nb::bounds::span_code((uintptr_t)addr, bytes, (uintptr_t)lo, (uintptr_t)hi, nb::bounds::kStateAddress);
}

int nb_debug_index_code(int64_t index, int64_t count) {
  return nb::bounds::index_inside(index, count) ? nb::bounds::kOk : nb::bounds::kLearnerIndex;
}

int nb_get_kernel_plan(const nb_ctx *c, int32_t *plan) {
  if (!c || !plan) return NB_ERR_ARG;
  const nb::PipePlan &p = c->last_plan;
  plan[0] = p.n_tiles > 0 ? 1 : 0;
  plan[1] = p.T;
  plan[2] = p.n_groups;
  plan[3] = p.n_slots;
  plan[4] = p.rows_per_item;
  plan[5] = p.grid;
  plan[6] = p.smem_bytes;
  plan[7] = p.n_tiles;
  plan[8] = p.row_copies;
  plan[9] = p.head;
  plan[10] = p.x_stages;
  plan[11] = p.n_tiles > 0 ? 4 * p.quads_per_thread : 0;
  return NB_OK;
}

int nb_get_stats(const nb_ctx *c, int64_t *sum_finished, double *algorithmic_bytes, int64_t *kernel_launches) {
  if (!c) return NB_ERR_ARG;
  if (sum_finished) *sum_finished = c->sum_finished;
  if (algorithmic_bytes) *algorithmic_bytes = c->alg_bytes;
  if (kernel_launches) *kernel_launches = c->launches;
  return NB_OK;
}

}  // extern "C"
