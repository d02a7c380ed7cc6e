"""Seeded synthetic inputs and the named workload configurations.

This module is the only one that both the CUDA-path tests and the CPU oracle tests use.  It holds
no arithmetic of the method: it only describes workloads (sizes, dtypes, straggler-model
parameters, hyper-parameters) and draws seeded Gaussian gradient streams and initial parameters.
Finished counts, masks, topologies and MATCHA activations are NOT produced here: the library and
the oracle each generate them independently and the tests compare the two bit for bit.

The gradient streams stand in for the mini-batch gradients of the paper's CIFAR-10/100 image
classifiers (Sec. 6.1), which need datasets and trained networks that are not available: flat
vectors of the stated parameter counts with i.i.d. N(0, sigma) entries.
"""
from dataclasses import dataclass, field
from typing import Tuple

import numpy as np

BASE_SEED = 221100889


@dataclass(frozen=True)
class Workload:
    name: str
    variant: str                 # "allreduce" | "dpsgd" | "matcha"
    topology: str                # "full" | "ring" | "random_regular"
    K: int                       # learners
    P: int                       # parameters per learner
    M: int                       # mini-batches per batch
    grad_dtype: str              # "f32" | "bf16"
    grad_sigma: float            # standard deviation of the synthetic gradients
    init_sigma: float            # standard deviation of the initial parameters
    straggler_model: str         # "uniform_count" | "shifted_exp" | "shifted_exp_slowset"
    straggler_params: Tuple[float, ...]
    lr: float
    mom: float
    steps: int
    seed: int
    degree: int = 0              # random_regular only
    alpha: float = 0.0           # MATCHA only
    act_prob: float = 0.0        # MATCHA only


def _w(idx, **kw):
    return Workload(seed=BASE_SEED + idx, **kw)


WORKLOADS = {
    "cfg1_tiny_allreduce": _w(
        1, name="cfg1_tiny_allreduce", variant="allreduce", topology="full", K=4, P=4096, M=4,
        grad_dtype="f32", grad_sigma=1.0, init_sigma=0.01, straggler_model="uniform_count",
        straggler_params=(), lr=0.1, mom=0.9, steps=10),
    "cfg2_allreduce_resnet18": _w(
        2, name="cfg2_allreduce_resnet18", variant="allreduce", topology="full", K=8, P=11_200_000,
        M=8, grad_dtype="f32", grad_sigma=0.01, init_sigma=0.01, straggler_model="shifted_exp",
        straggler_params=(0.5,), lr=0.1, mom=0.9, steps=50),
    "cfg3_dpsgd_ring_resnet50": _w(
        3, name="cfg3_dpsgd_ring_resnet50", variant="dpsgd", topology="ring", K=16, P=25_600_000,
        M=8, grad_dtype="bf16", grad_sigma=0.01, init_sigma=0.01, straggler_model="shifted_exp",
        straggler_params=(1.0,), lr=0.05, mom=0.9, steps=50),
    "cfg4_matcha_vgg16": _w(
        4, name="cfg4_matcha_vgg16", variant="matcha", topology="random_regular", K=16,
        P=138_000_000, M=4, grad_dtype="bf16", grad_sigma=0.01, init_sigma=0.01,
        straggler_model="shifted_exp", straggler_params=(0.5,), lr=0.05, mom=0.9, steps=20,
        degree=3, alpha=0.2, act_prob=0.5),
    "cfg5_scale_allreduce": _w(
        5, name="cfg5_scale_allreduce", variant="allreduce", topology="full", K=32, P=124_000_000,
        M=8, grad_dtype="bf16", grad_sigma=0.01, init_sigma=0.01,
        straggler_model="shifted_exp_slowset", straggler_params=(0.25, 2.0, 0.1), lr=0.05, mom=0.9,
        steps=20),
    "cfg5_scale_ring": _w(
        5, name="cfg5_scale_ring", variant="dpsgd", topology="ring", K=32, P=124_000_000,
        M=8, grad_dtype="bf16", grad_sigma=0.01, init_sigma=0.01,
        straggler_model="shifted_exp_slowset", straggler_params=(0.25, 2.0, 0.1), lr=0.05, mom=0.9,
        steps=20),
}


def scaled(w: Workload, P: int, steps: int = None) -> Workload:
    """The same workload on a narrower parameter vector (every step of the path is independent per
    column, so a column slice is the same computation)."""
    from dataclasses import replace
    return replace(w, P=P, steps=w.steps if steps is None else steps)


# ---------------------------------------------------------------------------------------------
# Seeded draws (CPU, NumPy).  Used at sizes a CPU handles; the GPU-resident generator below is
# for full-size streams.
# ---------------------------------------------------------------------------------------------
def _np_rng(seed: int, stream: int, step: int) -> np.random.Generator:
    return np.random.Generator(np.random.Philox(key=[(seed << 8) ^ stream, step]))


def init_params(w: Workload) -> np.ndarray:
    """x0[P] fp32, i.i.d. N(0, init_sigma); replicated to every learner by the caller."""
    g = _np_rng(w.seed, 0, 0)
    return (g.standard_normal(w.P, dtype=np.float32) * np.float32(w.init_sigma)).astype(np.float32)


def round_to_bf16_bits(a: np.ndarray) -> np.ndarray:
    """fp32 -> bf16 storage bits (uint16) with round-to-nearest-even; input has no NaN/Inf."""
    u = np.ascontiguousarray(a, dtype=np.float32).view(np.uint32)
    bias = ((u >> np.uint32(16)) & np.uint32(1)) + np.uint32(0x7FFF)
    return ((u + bias) >> np.uint32(16)).astype(np.uint16)


def bf16_bits_to_f32(b: np.ndarray) -> np.ndarray:
    """bf16 storage bits (uint16) -> the exact fp32 values they denote."""
    return (b.astype(np.uint32) << np.uint32(16)).view(np.float32)


def gradients_np(w: Workload, step: int, with_unrounded: bool = False):
    """One step's mini-batch gradient stream G[K, M, P] drawn on the CPU.

    Returns (payload, values): `payload` is the array handed to the library (float32, or uint16
    bf16 storage bits); `values` is a float32 array holding exactly the numbers the payload
    denotes (what the oracle consumes).  with_unrounded adds the fp32 draws before bf16 rounding."""
    g = _np_rng(w.seed, 1, step)
    a = g.standard_normal((w.K, w.M, w.P), dtype=np.float32) * np.float32(w.grad_sigma)
    if w.grad_dtype == "f32":
        return (a, a, a) if with_unrounded else (a, a)
    bits = round_to_bf16_bits(a)
    vals = bf16_bits_to_f32(bits)
    return (bits, vals, a) if with_unrounded else (bits, vals)


def gradients_torch(w: Workload, step: int, device):
    """One step's gradient stream drawn on `device` with torch's seeded generator; returns a
    tensor [K, M, P] of dtype float32 or bfloat16.  Full-size streams never exist on the host:
    callers copy the column slices they want checked."""
    import torch
    gen = torch.Generator(device=device)
    gen.manual_seed((w.seed << 20) + step)
    dt = torch.float32 if w.grad_dtype == "f32" else torch.bfloat16
    out = torch.empty((w.K, w.M, w.P), dtype=dt, device=device)
    # draw learner by learner to bound the fp32 temporary
    for i in range(w.K):
        tmp = torch.randn((w.M, w.P), generator=gen, device=device, dtype=torch.float32)
        tmp.mul_(w.grad_sigma)
        out[i].copy_(tmp)
        del tmp
    return out
