"""Thin ctypes binding of the C-ABI library (include/nb.h): argument marshalling only.

Every step of the path runs inside libnb.so's CUDA kernels; nothing here computes.  Tensors are
torch tensors (device memory and streams come from torch); their raw pointers cross the boundary.
If the library is missing or fails to load, importing this module raises: there is no fallback.
"""
import ctypes as C
import os

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.environ.get("NB_LIB_PATH") or os.path.join(_HERE, "libnb.so")

NB_OK, NB_ERR_ARG, NB_ERR_STATE, NB_ERR_CUDA, NB_ERR_NOMEM, NB_ERR_UNSUPPORTED = 0, -1, -2, -3, -4, -5
NB_ALLREDUCE, NB_DPSGD, NB_MATCHA, NB_CENTRALIZED = 0, 1, 2, 3
NB_F32, NB_BF16 = 0, 1
NB_TOPO_FULL, NB_TOPO_RING, NB_TOPO_CSR, NB_TOPO_MATCHINGS, NB_TOPO_RANDOM_REGULAR = 0, 1, 2, 3, 4
NB_OPT_NORM, NB_OPT_ORDER, NB_OPT_KERNEL, NB_OPT_STREAMING = 0, 1, 2, 3
NB_STREAMING_ACCUMULATE, NB_STREAMING_HOLD = 0, 1
NB_KERNEL_AUTO, NB_KERNEL_DIRECT = 0, 1
NB_NORM_MEAN, NB_NORM_PAPER = 0, 1
NB_ORDER_MIX_THEN_UPDATE, NB_ORDER_UPDATE_THEN_MIX = 0, 1
NB_STRAG_UNIFORM_COUNT, NB_STRAG_SHIFTED_EXP, NB_STRAG_SHIFTED_EXP_SLOWSET = 0, 1, 2
NB_MAX_K, NB_MAX_MATCHINGS, NB_MAX_NNZ = 64, 32, 1024
NB_STATIC_MAX_ELEMS = 1 << 22
NB_ABANDONED = 1

VARIANTS = {"allreduce": NB_ALLREDUCE, "dpsgd": NB_DPSGD, "matcha": NB_MATCHA, "centralized": NB_CENTRALIZED}
STRAGGLER_MODELS = {"uniform_count": NB_STRAG_UNIFORM_COUNT, "shifted_exp": NB_STRAG_SHIFTED_EXP,
                    "shifted_exp_slowset": NB_STRAG_SHIFTED_EXP_SLOWSET}


class nb_topology(C.Structure):
    _fields_ = [("kind", C.c_int32), ("degree", C.c_int32), ("seed", C.c_uint64),
                ("row_ptr", C.POINTER(C.c_int32)), ("col_idx", C.POINTER(C.c_int32)), ("val", C.POINTER(C.c_float)),
                ("n_matchings", C.c_int32), ("partner", C.POINTER(C.c_int32)),
                ("alpha", C.c_float), ("act_prob", C.c_float), ("act_probs", C.POINTER(C.c_float))]


class nb_runtime_report(C.Structure):
    _fields_ = [("mean_t_nonblocking", C.c_double), ("mean_t_blocking", C.c_double), ("ratio", C.c_double),
                ("mean_throughput_ratio", C.c_double), ("mean_fractional_data", C.c_double),
                ("mean_finished_fraction", C.c_double), ("mean_min_tau", C.c_double), ("mean_max_tau", C.c_double),
                ("steps", C.c_int64)]


class nb_straggler(C.Structure):
    _fields_ = [("model", C.c_int32), ("seed", C.c_uint64), ("params", C.c_double * 4)]


class NbError(RuntimeError):
    def __init__(self, code, msg):
        super().__init__("nb error %d: %s" % (code, msg))
        self.code = code


def _load():
    if not os.path.exists(LIB_PATH):
        raise ImportError("libnb.so is not built (run: python -m paper_2211_00889_b200.build); "
                          "there is no CPU or PyTorch fallback for this path")
    lib = C.CDLL(LIB_PATH)
    vp, i32, i64, f32 = C.c_void_p, C.c_int, C.c_int64, C.c_float
    P = C.POINTER
    sig = {
        "nb_straggler_sample": [P(nb_straggler), i32, i32, i64, P(C.c_int32), P(C.c_uint8), P(C.c_double)],
        "nb_topology_matchings": [P(nb_topology), i32, P(C.c_int32), P(C.c_int32), P(C.c_int32)],
        "nb_matcha_optimize": [P(nb_topology), i32, f32, i32, P(C.c_float), P(C.c_float), P(C.c_float), P(C.c_float)],
        "nb_mixing_matrix": [P(nb_topology), i32, i32, i64, P(C.c_float), P(C.c_uint32)],
        "nb_create": [P(vp), i32, i64, i32, f32, f32, i32, P(nb_topology)],
        "nb_destroy": [vp],
        "nb_set_option": [vp, i32, i64],
        "nb_set_lr": [vp, f32],
        "nb_set_params": [vp, vp, i32, vp],
        "nb_accumulate": [vp, vp, i32, i64, i64, P(C.c_int32), vp],
        "nb_step": [vp, vp],
        "nb_step_fused": [vp, vp, i32, i64, i64, P(C.c_int32), vp],
        "nb_step_fused_host": [vp, vp, i32, i64, i64, P(C.c_int32), vp, vp],
        "nb_get_params": [vp, vp, vp],
        "nb_get_momentum": [vp, vp, vp],
        "nb_get_accumulator": [vp, vp, vp],
        "nb_get_mean_params": [vp, vp, vp],
        "nb_set_state": [vp, i64, vp, vp, vp],
        "nb_get_step": [vp, P(i64)],
        "nb_get_W": [vp, i64, P(C.c_float)],
        "nb_get_matcha_activation": [vp, i64, P(C.c_uint32)],
        "nb_get_device_mixing": [vp, P(C.c_uint32), P(C.c_float), vp],
        "nb_get_stats": [vp, P(i64), P(C.c_double), P(i64)],
        "nb_begin_iteration": [vp],
        "nb_accumulate_minibatch": [vp, i32, vp, i32, vp],
        "nb_get_finished": [vp, P(C.c_int32), P(C.c_int32)],
        "nb_runtime_report_compute": [P(nb_straggler), i32, i32, i64, i64, P(nb_runtime_report)],
        "nb_get_kernel_plan": [vp, P(C.c_int32)],
        "nb_check_guards": [vp, vp],
        "nb_selftest_wait_timeout": [vp, vp],
        "nb_step_static": [i32, i64, i32, f32, f32, vp, vp, i64, vp, i32, i64, i64, P(C.c_int32), vp],
        "nb_debug_build": [],
        "nb_debug_span_code": [C.c_uint64, C.c_uint64, C.c_uint64, C.c_uint64],
        "nb_debug_index_code": [i64, i64],
    }
    for name, args in sig.items():
        fn = getattr(lib, name)
        fn.argtypes = args
        fn.restype = C.c_int
    lib.nb_recommended_pitch.argtypes = [i64, i32]
    lib.nb_recommended_pitch.restype = i64
    lib.nb_last_error.argtypes = [vp]
    lib.nb_last_error.restype = C.c_char_p
    return lib


lib = _load()
EXPORTED = ["nb_straggler_sample", "nb_topology_matchings", "nb_mixing_matrix", "nb_create", "nb_destroy",
            "nb_last_error", "nb_set_option", "nb_set_lr", "nb_set_params", "nb_accumulate", "nb_step",
            "nb_step_fused", "nb_step_fused_host", "nb_get_params", "nb_get_momentum", "nb_get_accumulator",
            "nb_get_mean_params", "nb_set_state", "nb_get_step", "nb_get_W", "nb_get_matcha_activation",
            "nb_get_device_mixing", "nb_get_stats", "nb_step_static", "nb_get_kernel_plan", "nb_check_guards", "nb_selftest_wait_timeout",
            "nb_matcha_optimize", "nb_begin_iteration", "nb_accumulate_minibatch", "nb_get_finished", "nb_runtime_report_compute",
            "nb_debug_build", "nb_debug_span_code", "nb_debug_index_code", "nb_recommended_pitch"]


def _i32p(a):
    return a.ctypes.data_as(C.POINTER(C.c_int32))


def make_topology(kind="full", K=0, degree=0, seed=0, csr=None, partner=None, alpha=0.0, act_prob=0.0,
                  act_probs=None):
    """Returns (nb_topology, keepalive) for the named kind."""
    t = nb_topology()
    keep = []
    kinds = {"full": NB_TOPO_FULL, "ring": NB_TOPO_RING, "csr": NB_TOPO_CSR, "matchings": NB_TOPO_MATCHINGS,
             "random_regular": NB_TOPO_RANDOM_REGULAR}
    t.kind = kinds[kind]
    t.degree = degree
    t.seed = seed
    t.alpha = alpha
    t.act_prob = act_prob
    if csr is not None:
        rp = np.ascontiguousarray(csr[0], dtype=np.int32)
        ci = np.ascontiguousarray(csr[1], dtype=np.int32)
        va = np.ascontiguousarray(csr[2], dtype=np.float32)
        keep += [rp, ci, va]
        t.row_ptr, t.col_idx = _i32p(rp), _i32p(ci)
        t.val = va.ctypes.data_as(C.POINTER(C.c_float))
    if act_probs is not None:
        ap = np.ascontiguousarray(act_probs, dtype=np.float32)
        keep.append(ap)
        t.act_probs = ap.ctypes.data_as(C.POINTER(C.c_float))
    if partner is not None:
        pt = np.ascontiguousarray(partner, dtype=np.int32)
        keep.append(pt)
        t.n_matchings = pt.shape[0]
        t.partner = _i32p(pt)
    return t, keep


def straggler_sample(model, seed, step, K, M, params=()):
    """Finished counts n[K], mask[K,M] and mini-batch times tau[K] of one step (host simulator)."""
    cfg = nb_straggler()
    cfg.model = STRAGGLER_MODELS[model] if isinstance(model, str) else model
    cfg.seed = seed
    for q, v in enumerate(params):
        cfg.params[q] = float(v)
    n = np.zeros(K, dtype=np.int32)
    mask = np.zeros((K, M), dtype=np.uint8)
    tau = np.zeros(K, dtype=np.float64)
    rc = lib.nb_straggler_sample(C.byref(cfg), K, M, step, _i32p(n), mask.ctypes.data_as(C.POINTER(C.c_uint8)),
                                 tau.ctypes.data_as(C.POINTER(C.c_double)))
    if rc != NB_OK:
        raise NbError(rc, "nb_straggler_sample")
    return n, mask, tau


def runtime_report(model, seed, K, M, steps, params=(), step0=0):
    """nb_runtime_report_compute as a dict (host only)."""
    cfg = nb_straggler()
    cfg.model = STRAGGLER_MODELS[model] if isinstance(model, str) else model
    cfg.seed = seed
    for q, v in enumerate(params):
        cfg.params[q] = float(v)
    rep = nb_runtime_report()
    rc = lib.nb_runtime_report_compute(C.byref(cfg), K, M, step0, steps, C.byref(rep))
    if rc != NB_OK:
        raise NbError(rc, "nb_runtime_report_compute")
    return {name: getattr(rep, name) for name, _ in nb_runtime_report._fields_}


def topology_matchings(topo, K):
    partner = np.full((NB_MAX_MATCHINGS, K), -1, dtype=np.int32)
    n = C.c_int32(0)
    att = C.c_int32(0)
    rc = lib.nb_topology_matchings(C.byref(topo), K, _i32p(partner), C.byref(n), C.byref(att))
    if rc != NB_OK:
        raise NbError(rc, "nb_topology_matchings")
    return partner[:n.value].copy(), att.value


def matcha_optimize(topo, K, budget, iters=0):
    """Activation probabilities (fp32 array [m]), alpha, lambda_2 and rho of MATCHA's design problem."""
    m = topology_matchings(topo, K)[0].shape[0]
    probs = np.zeros(m, dtype=np.float32)
    a, l2, rho = C.c_float(0), C.c_float(0), C.c_float(0)
    rc = lib.nb_matcha_optimize(C.byref(topo), K, budget, iters, probs.ctypes.data_as(C.POINTER(C.c_float)),
                                C.byref(a), C.byref(l2), C.byref(rho))
    if rc != NB_OK:
        raise NbError(rc, "nb_matcha_optimize")
    return probs, a.value, l2.value, rho.value


def mixing_matrix(topo, variant, K, step):
    W = np.zeros((K, K), dtype=np.float32)
    bits = C.c_uint32(0)
    rc = lib.nb_mixing_matrix(C.byref(topo) if topo is not None else None, variant, K, step,
                              W.ctypes.data_as(C.POINTER(C.c_float)), C.byref(bits))
    if rc != NB_OK:
        raise NbError(rc, "nb_mixing_matrix")
    return W, bits.value


def _ptr(t):
    """Raw address of a torch tensor or NumPy array (None -> NULL)."""
    if t is None:
        return None
    if isinstance(t, np.ndarray):
        return C.c_void_p(t.ctypes.data)
    return C.c_void_p(t.data_ptr())


def _stream():
    import torch
    return C.c_void_p(torch.cuda.current_stream().cuda_stream)


def _dtype_code(t):
    import torch
    if t.dtype == torch.float32:
        return NB_F32
    if t.dtype == torch.bfloat16:
        return NB_BF16
    raise TypeError("gradient stream must be float32 or bfloat16")


class NbContext:
    """Owns one nb_ctx.  Methods mirror the C entry points one to one."""

    def __init__(self, K, P, M, lr, mom, variant, topo=None):
        self.K, self.P, self.M = K, P, M
        self.variant = VARIANTS[variant] if isinstance(variant, str) else variant
        self.rows = 1 if self.variant == NB_CENTRALIZED else K
        self._keep = None
        if isinstance(topo, tuple):
            topo, self._keep = topo
        self._h = C.c_void_p()
        rc = lib.nb_create(C.byref(self._h), K, P, M, lr, mom, self.variant,
                           C.byref(topo) if topo is not None else None)
        if rc != NB_OK:
            self._h = None
            raise NbError(rc, lib.nb_last_error(None).decode())

    def _ck(self, rc):
        if rc != NB_OK:
            raise NbError(rc, lib.nb_last_error(self._h).decode())

    def close(self):
        if getattr(self, "_h", None):
            if lib is not None:          # (None while the interpreter is shutting down: the process frees the GPU itself)
                lib.nb_destroy(self._h)
            self._h = None

    __del__ = close

    def __enter__(self):
        return self

    def __exit__(self, *a):
        self.close()

    def set_option(self, key, value):
        self._ck(lib.nb_set_option(self._h, key, value))

    def set_lr(self, lr):
        self._ck(lib.nb_set_lr(self._h, lr))

    def set_params(self, x0, per_learner=False):
        self._ck(lib.nb_set_params(self._h, _ptr(x0), 1 if per_learner else 0, _stream()))

    @staticmethod
    def _finished(n):
        return np.ascontiguousarray(n, dtype=np.int32)

    @staticmethod
    def _pitches(grads, ld_m, ld_k):
        """Element strides of a [K, M, P] gradient tensor: the caller's, else the tensor's own (a view
        whose rows are contiguous is passed as it is, never copied)."""
        if hasattr(grads, "stride") and grads.dim() == 3:
            if grads.stride(2) != 1 and grads.shape[2] > 1:
                raise ValueError("gradient rows must be contiguous (stride 1 along the parameter axis)")
            if not ld_m:
                ld_m = grads.stride(1) if grads.shape[1] > 1 else 0
            if not ld_k:
                ld_k = grads.stride(0) if grads.shape[0] > 1 else 0
        return ld_m, ld_k

    def accumulate(self, grads, finished, ld_m=0, ld_k=0):
        n = self._finished(finished)
        ld_m, ld_k = self._pitches(grads, ld_m, ld_k)
        self._ck(lib.nb_accumulate(self._h, _ptr(grads), _dtype_code(grads), ld_m, ld_k, _i32p(n), _stream()))

    def begin_iteration(self):
        self._ck(lib.nb_begin_iteration(self._h))

    def accumulate_minibatch(self, learner, grad):
        """True if the mini-batch was accumulated, False if it was abandoned (terminal signal raised)."""
        rc = lib.nb_accumulate_minibatch(self._h, learner, _ptr(grad), _dtype_code(grad), _stream())
        if rc == NB_ABANDONED:
            return False
        self._ck(rc)
        return True

    def get_finished(self):
        n = np.zeros(self.K, dtype=np.int32)
        term = C.c_int32(0)
        self._ck(lib.nb_get_finished(self._h, _i32p(n), C.byref(term)))
        return n, bool(term.value)

    def step(self):
        self._ck(lib.nb_step(self._h, _stream()))

    def step_fused(self, grads, finished, ld_m=0, ld_k=0):
        n = self._finished(finished)
        ld_m, ld_k = self._pitches(grads, ld_m, ld_k)
        self._ck(lib.nb_step_fused(self._h, _ptr(grads), _dtype_code(grads), ld_m, ld_k, _i32p(n), _stream()))

    def step_fused_host(self, grads_host, finished, mean_out=None, ld_m=0, ld_k=0):
        n = self._finished(finished)
        ld_m, ld_k = self._pitches(grads_host, ld_m, ld_k)
        self._ck(lib.nb_step_fused_host(self._h, _ptr(grads_host), _dtype_code(grads_host), ld_m, ld_k, _i32p(n),
                                        _ptr(mean_out), _stream()))

    def _out(self, fn, rows, device):
        import torch
        shape = (rows, self.P) if rows > 1 or self.variant != NB_CENTRALIZED else (self.P,)
        dst = torch.empty(shape, dtype=torch.float32, device=device)
        self._ck(fn(self._h, _ptr(dst), _stream()))
        return dst

    def get_params(self, device="cpu"):
        return self._out(lib.nb_get_params, self.rows, device)

    def get_momentum(self, device="cpu"):
        return self._out(lib.nb_get_momentum, self.rows, device)

    def get_accumulator(self, device="cpu"):
        import torch
        dst = torch.empty((self.K, self.P), dtype=torch.float32, device=device)
        self._ck(lib.nb_get_accumulator(self._h, _ptr(dst), _stream()))
        return dst

    def get_mean_params(self, device="cpu"):
        import torch
        dst = torch.empty(self.P, dtype=torch.float32, device=device)
        self._ck(lib.nb_get_mean_params(self._h, _ptr(dst), _stream()))
        return dst

    def set_state(self, step, X, V):
        self._ck(lib.nb_set_state(self._h, step, _ptr(X), _ptr(V), _stream()))

    def get_step(self):
        s = C.c_int64(0)
        self._ck(lib.nb_get_step(self._h, C.byref(s)))
        return s.value

    def get_W(self, step):
        W = np.zeros((self.K, self.K), dtype=np.float32)
        self._ck(lib.nb_get_W(self._h, step, W.ctypes.data_as(C.POINTER(C.c_float))))
        return W

    def get_matcha_activation(self, step):
        b = C.c_uint32(0)
        self._ck(lib.nb_get_matcha_activation(self._h, step, C.byref(b)))
        return b.value

    def get_device_mixing(self):
        W = np.zeros((self.K, self.K), dtype=np.float32)
        b = C.c_uint32(0)
        self._ck(lib.nb_get_device_mixing(self._h, C.byref(b), W.ctypes.data_as(C.POINTER(C.c_float)), _stream()))
        return b.value, W

    def selftest_wait_timeout(self):
        self._ck(lib.nb_selftest_wait_timeout(self._h, _stream()))

    def check_guards(self):
        self._ck(lib.nb_check_guards(self._h, _stream()))

    def get_kernel_plan(self):
        a = np.zeros(12, dtype=np.int32)
        self._ck(lib.nb_get_kernel_plan(self._h, _i32p(a)))
        keys = ("pipeline", "tile", "groups", "slots", "rows_per_item", "grid", "smem_bytes", "tiles", "row_copies",
                "head", "x_buffers", "columns_per_thread")
        return dict(zip(keys, (int(v) for v in a)))

    def get_stats(self):
        s, b, l = C.c_int64(0), C.c_double(0), C.c_int64(0)
        self._ck(lib.nb_get_stats(self._h, C.byref(s), C.byref(b), C.byref(l)))
        return {"sum_finished": s.value, "algorithmic_bytes": b.value, "kernel_launches": l.value}


def recommended_pitch(P, dtype):
    """Row pitch in elements at which a [K, M, P] gradient stream of torch dtype `dtype` streams fastest."""
    import torch
    return int(lib.nb_recommended_pitch(P, NB_F32 if dtype == torch.float32 else NB_BF16))


def step_static(X, V, grads, finished, P, M, lr, mom, ld_m=0, ld_k=0):
    """nb_step_static: one all-reduce-variant iteration on caller-owned X[K, ld], V[K, ld] (device
    tensors, updated in place) for callers that cannot allocate device memory; the accumulator
    lives in a fixed array inside the library.  Raises NbError (NB_ERR_UNSUPPORTED) when K*ld
    exceeds NB_STATIC_MAX_ELEMS."""
    K, ld = X.shape
    n = np.ascontiguousarray(finished, dtype=np.int32)
    rc = lib.nb_step_static(K, P, M, lr, mom, _ptr(X), _ptr(V), ld, _ptr(grads), _dtype_code(grads), ld_m, ld_k,
                            _i32p(n), _stream())
    if rc != NB_OK:
        raise NbError(rc, lib.nb_last_error(None).decode())


def context_for(w, P=None):
    """NbContext for a workloads.Workload (optionally on a narrower column range)."""
    P = w.P if P is None else P
    topo = None
    if w.topology == "ring":
        topo = make_topology("ring")
    elif w.topology == "random_regular":
        topo = make_topology("random_regular", degree=w.degree, seed=w.seed, alpha=w.alpha, act_prob=w.act_prob)
    return NbContext(w.K, P, w.M, w.lr, w.mom, w.variant, topo)
