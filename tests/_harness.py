"""Shared helpers of the GPU parity tests: drive the library and the oracle on the same seeded
inputs and compare.  Not a test module."""
import numpy as np

from oracle import nb_oracle as O
from paper_2211_00889_b200 import workloads as WL

TOL_SAME_INPUT = 1e-5     # GPU fp32 path vs fp64 oracle fed the same input values
TOL_BF16_ROUNDING = 2e-3  # GPU on bf16 gradients vs oracle fed the un-rounded fp32 gradients


def oracle_for(w, P, norm="mean", order="mix_then_update"):
    """Oracle whose topology comes from the oracle's own generators."""
    if w.variant == "allreduce":
        return O.Oracle(w.K, P, w.M, w.lr, w.mom, "allreduce", norm=norm, order=order)
    if w.variant == "dpsgd":
        W = O.ring_W(w.K) if w.topology == "ring" else O.full_W(w.K)
        return O.Oracle(w.K, P, w.M, w.lr, w.mom, "dpsgd", W=W, norm=norm, order=order)
    if w.variant == "matcha":
        edges, _ = O.random_regular_graph(w.seed, w.K, w.degree)
        partner = O.greedy_matchings(edges, w.K)
        return O.Oracle(w.K, P, w.M, w.lr, w.mom, "matcha", partner=partner, alpha=w.alpha, prob=w.act_prob,
                        seed=w.seed, norm=norm, order=order)
    raise ValueError(w.variant)


def to_device(payload, device="cuda"):
    """NumPy payload (float32 or uint16 bf16 bits) -> torch tensor of the library's dtype."""
    import torch
    t = torch.from_numpy(np.ascontiguousarray(payload))
    if payload.dtype == np.uint16:
        t = t.view(torch.bfloat16)
    return t.to(device)


def rel_errors(x_gpu, x_ref):
    """(norm-wise, max-wise) relative errors over learners."""
    x_gpu = np.asarray(x_gpu, dtype=np.float64)
    x_ref = np.asarray(x_ref, dtype=np.float64)
    if x_ref.ndim == 1:
        x_gpu, x_ref = x_gpu[None], x_ref[None]
    nrm = max(np.linalg.norm(x_gpu[i] - x_ref[i]) / max(np.linalg.norm(x_ref[i]), 1e-300)
              for i in range(x_ref.shape[0]))
    mx = np.abs(x_gpu - x_ref).max() / max(np.abs(x_ref).max(), 1e-300)
    return nrm, mx


def assert_close(x_gpu, x_ref, tol, what=""):
    nrm, mx = rel_errors(x_gpu, x_ref)
    assert nrm <= tol and mx <= tol, "%s: norm-wise %.3e, max-wise %.3e > %.1e" % (what, nrm, mx, tol)
    return nrm, mx


def lib_counts(B, w, t):
    n, mask, _ = B.straggler_sample(w.straggler_model, w.seed, t, w.K, w.M, w.straggler_params)
    want = O.straggler_counts(w.straggler_model, w.seed, t, w.K, w.M, w.straggler_params)
    assert n.tolist() == want                       # bit-exact finished counts
    assert np.array_equal(mask, O.finished_mask(want, w.M))
    return n
