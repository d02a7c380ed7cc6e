// nb_step_static: the accumulate -> step pair for callers that must not allocate device memory.
//
// Some users of this library cannot call cudaMalloc once they are running: processes that gave the
// whole GPU to a framework's memory pool at start-up and have no budget left outside it, serving
// loops for which the implicit device-wide synchronisation of an allocation is a latency fault, and
// deployments whose policy forbids allocation after initialisation.  For them the one piece of
// scratch memory the unfused path needs - the fp32 accumulator acc[K, ld] between the masked
// accumulate and the update - lives in a fixed array that is part of the library image.  Every GPU
// that loads the library carries this array (NB_STATIC_MAX_ELEMS floats) until the process exits.
#include <cuda_runtime.h>

#include <cstring>
#include <mutex>
#include <string>

#include "nb_internal.h"
#include "nb_kernels.h"

namespace {

// The scratch accumulator.  In host code this name is only a handle for the runtime's symbol
// look-up, never a device address; kernels receive the address cudaGetSymbolAddress returns.
static __device__ __align__(256) float nb_static_acc[NB_STATIC_MAX_ELEMS];

constexpr int kMaxDevices = 64;
std::mutex g_setup_mutex;
float *g_acc_addr[kMaxDevices] = {nullptr};

// Once per device, with that device current: resolve the array's device address.
cudaError_t static_acc_address(float **out) {
  int dev = -1;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return e;
  if (dev < 0 || dev >= kMaxDevices) return cudaErrorInvalidDevice;
  std::lock_guard<std::mutex> lock(g_setup_mutex);
  if (!g_acc_addr[dev]) {
    float *p = nullptr;
    e = cudaGetSymbolAddress(reinterpret_cast<void **>(&p), nb_static_acc);
    if (e != cudaSuccess) return e;
    g_acc_addr[dev] = p;
  }
  *out = g_acc_addr[dev];
  return cudaSuccess;
}

}  // namespace

namespace nb {
void set_global_error(const std::string &msg);  // text returned by nb_last_error(NULL)
}

extern "C" int nb_step_static(int K, int64_t P, int M, float lr, float mom, float *X, float *V, int64_t ld,
                              const void *grads, int dtype, int64_t ld_m, int64_t ld_k, const int32_t *finished,
                              void *stream) {
  auto fail = [](int code, const std::string &msg) {
    nb::set_global_error(msg);
    return code;
  };
  if (K < 1 || P < 1 || M < 1) return fail(NB_ERR_ARG, "nb_step_static: K, P and M must be >= 1");
  if (K > NB_MAX_K) return fail(NB_ERR_UNSUPPORTED, "nb_step_static: K exceeds NB_MAX_K");
  if (!X || !V || !grads || !finished) return fail(NB_ERR_ARG, "nb_step_static: NULL pointer argument");
  if (dtype != NB_F32 && dtype != NB_BF16) return fail(NB_ERR_ARG, "nb_step_static: dtype must be NB_F32 or NB_BF16");
  if (ld < P || ld % 4 != 0) return fail(NB_ERR_ARG, "nb_step_static: ld must be >= P and a multiple of 4");
  if ((uintptr_t)X % 16 != 0 || (uintptr_t)V % 16 != 0) return fail(NB_ERR_ARG, "nb_step_static: X and V must be 16-byte aligned");
  if ((int64_t)K * ld > (int64_t)NB_STATIC_MAX_ELEMS)
    return fail(NB_ERR_UNSUPPORTED, "nb_step_static: K*ld = " + std::to_string((long long)K * ld) +
                                        " floats exceeds the static accumulator (NB_STATIC_MAX_ELEMS = " +
                                        std::to_string((long long)NB_STATIC_MAX_ELEMS) + ")");
  const int es = dtype == NB_F32 ? 4 : 2;
  if (ld_m == 0) ld_m = P;
  if (ld_k == 0) ld_k = (int64_t)M * ld_m;
  if (ld_m < P || ld_k < (int64_t)(M - 1) * ld_m + P) return fail(NB_ERR_ARG, "nb_step_static: ld_m / ld_k too small");
  for (int i = 0; i < K; ++i)
    if (finished[i] < 0 || finished[i] > M) return fail(NB_ERR_ARG, "nb_step_static: finished count outside [0, M]");

  float *acc = nullptr;
  cudaError_t e = static_acc_address(&acc);
  if (e != cudaSuccess) return fail(NB_ERR_CUDA, std::string("nb_step_static: cudaGetSymbolAddress: ") + cudaGetErrorString(e));

  nb::StepArgs a;
  std::memset(&a, 0, sizeof(a));
  a.X = X;
  a.V = V;
  a.acc = acc;
  a.G = grads;
  a.ldx = ld;
  a.ld_m = ld_m;
  a.ld_k = ld_k;
  a.P = P;
  a.K = K;
  a.M = M;
  a.g_aligned = ((uintptr_t)grads % (size_t)(4 * es) == 0) && (ld_m % 4 == 0) && (ld_k % 4 == 0);
  a.lr = lr;
  a.mom = mom;
  a.inv_K = 1.0f / (float)K;
  a.order = NB_ORDER_MIX_THEN_UPDATE;
  a.mean_mode = 1;
  for (int i = 0; i < K; ++i) {
    a.n[i] = finished[i];
    a.s[i] = finished[i] > 0 ? 1.0f / (float)finished[i] : 0.0f;
  }
  // extents for the bounds-checked build (there is no context, hence no error word: a failed check
  // there only skips the access)
  a.ext.x_lo = (uintptr_t)X;
  a.ext.x_hi = a.ext.x_lo + sizeof(float) * (size_t)K * (size_t)ld;
  a.ext.v_lo = (uintptr_t)V;
  a.ext.v_hi = a.ext.v_lo + sizeof(float) * (size_t)K * (size_t)ld;
  a.ext.acc_lo = (uintptr_t)acc;
  a.ext.acc_hi = a.ext.acc_lo + sizeof(float) * (size_t)NB_STATIC_MAX_ELEMS;
  a.ext.g_lo = (uintptr_t)grads;
  a.ext.g_hi = a.ext.g_lo + (size_t)((int64_t)(K - 1) * ld_k + (int64_t)(M - 1) * ld_m + P) * (size_t)es;
  a.err = nullptr;
  cudaStream_t st = (cudaStream_t)stream;
  // the accumulate kernel writes every element of acc[K, 0:round_up(P,4)) that the step kernel reads,
  // so nothing of the previous call's contents survives into this one
  e = nb::launch_accumulate_direct_only(a, dtype == NB_F32 ? nb::kSrcF32 : nb::kSrcBF16, st);
  if (e == cudaSuccess) e = nb::launch_step_direct_only(a, nb::kSrcAcc, st);
  if (e != cudaSuccess) return fail(NB_ERR_CUDA, std::string("nb_step_static: launch: ") + cudaGetErrorString(e));
  return NB_OK;
}
