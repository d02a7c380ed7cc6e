"""Randomised configurations of the whole step against the oracle: learner count, mini-batch count,
column count (aligned or not), gradient dtype, variant and topology, normalisation, order, fused or
unfused entry, padded or dense gradient rows, arbitrary finished counts (zeros included)."""
from dataclasses import replace

import numpy as np
import pytest

from oracle import nb_oracle as O
from paper_2211_00889_b200 import workloads as WL
from tests import _harness as H

pytestmark = pytest.mark.gpu


def _random_case(rng):
    variant = rng.choice(["allreduce", "ring", "identity_csr", "matcha", "centralized"])
    K = int(rng.integers(1, 41))
    if variant == "matcha":
        K = int(rng.choice([4, 6, 8, 10, 16, 24]))
    M = int(rng.integers(1, 13))
    P = int(rng.choice([rng.integers(1, 600), 512 * rng.integers(1, 6), 512 * rng.integers(1, 6) + 8 * rng.integers(1, 60),
                        512 * rng.integers(1, 4) + rng.integers(1, 512)]))
    dtype = str(rng.choice(["bf16", "f32"]))
    norm = str(rng.choice(["mean", "paper"]))
    order = str(rng.choice(["mix_then_update", "update_then_mix"]))
    fused = bool(rng.integers(0, 2))
    pad = int(rng.choice([0, 0, 8, 24]))
    return dict(variant=variant, K=K, M=M, P=P, dtype=dtype, norm=norm, order=order, fused=fused, pad=pad,
                seed=int(rng.integers(0, 2 ** 40)))


@pytest.mark.parametrize("case_id", range(48))
def test_random_configuration(case_id):
    import torch
    from paper_2211_00889_b200.build import build_library
    build_library()
    from paper_2211_00889_b200 import binding as B
    rng = np.random.default_rng(7000 + case_id)
    c = _random_case(rng)
    K, M, P = c["K"], c["M"], c["P"]
    lr, mom = 0.05, 0.9
    if c["variant"] == "allreduce":
        ctx = B.NbContext(K, P, M, lr, mom, "allreduce")
        orc = O.Oracle(K, P, M, lr, mom, "allreduce", norm=c["norm"], order=c["order"])
    elif c["variant"] == "ring":
        ctx = B.NbContext(K, P, M, lr, mom, "dpsgd", B.make_topology("ring"))
        orc = O.Oracle(K, P, M, lr, mom, "dpsgd", W=O.ring_W(K), norm=c["norm"], order=c["order"])
    elif c["variant"] == "identity_csr":
        csr = (np.arange(K + 1), np.arange(K), np.ones(K))
        ctx = B.NbContext(K, P, M, lr, mom, "dpsgd", B.make_topology("csr", csr=csr))
        orc = O.Oracle(K, P, M, lr, mom, "dpsgd", W=O.identity_W(K), norm=c["norm"], order=c["order"])
    elif c["variant"] == "matcha":
        d = 3 if K > 4 else 2
        topo = B.make_topology("random_regular", degree=d, seed=c["seed"], alpha=0.2, act_prob=0.6)
        ctx = B.NbContext(K, P, M, lr, mom, "matcha", topo)
        partner = O.greedy_matchings(O.random_regular_graph(c["seed"], K, d)[0], K)
        orc = O.Oracle(K, P, M, lr, mom, "matcha", partner=partner, alpha=0.2, prob=0.6, seed=c["seed"],
                       norm=c["norm"], order=c["order"])
    else:
        ctx = B.NbContext(K, P, M, lr, mom, "centralized")
        orc = None
    ctx.set_option(B.NB_OPT_NORM, B.NB_NORM_MEAN if c["norm"] == "mean" else B.NB_NORM_PAPER)
    ctx.set_option(B.NB_OPT_ORDER, B.NB_ORDER_MIX_THEN_UPDATE if c["order"] == "mix_then_update" else B.NB_ORDER_UPDATE_THEN_MIX)
    x0 = (rng.standard_normal(P) * 0.01).astype(np.float32)
    ctx.set_params(torch.from_numpy(x0).cuda())
    if orc is not None:
        orc.set_params(x0)
    x_ps, v_ps = x0.astype(np.float64), np.zeros(P)
    tdt = torch.bfloat16 if c["dtype"] == "bf16" else torch.float32
    for t in range(3):
        G = (torch.from_numpy(rng.standard_normal((K, M, P)).astype(np.float32)) * 0.01).to(tdt)
        n = rng.integers(0, M + 1, K)
        if c["pad"]:
            wide = torch.zeros((K, M, P + c["pad"]), dtype=tdt)
            wide[:, :, :P] = G
            g = wide.cuda()[:, :, :P]
            ld = dict(ld_m=P + c["pad"], ld_k=M * (P + c["pad"]))
        else:
            g, ld = G.cuda(), {}
        if c["fused"]:
            ctx.step_fused(g, n, **ld)
        else:
            ctx.accumulate(g, n, **ld)
            ctx.step()
        vals = G.float().numpy()
        if orc is not None:
            orc.step(vals, n.tolist())
        else:
            x_ps, v_ps = O.step_centralized(x_ps, v_ps, vals, n.tolist(), lr, mom, norm=c["norm"])
    X = ctx.get_params().numpy()
    V = ctx.get_momentum().numpy()
    if orc is not None:
        H.assert_close(X, orc.X, H.TOL_SAME_INPUT, str(c))
        H.assert_close(V, orc.V, H.TOL_SAME_INPUT, str(c))
    else:
        H.assert_close(X, x_ps, H.TOL_SAME_INPUT, str(c))
        H.assert_close(V, v_ps, H.TOL_SAME_INPUT, str(c))
    ctx.check_guards()
    ctx.close()


@pytest.mark.parametrize("case_id", range(100))
def test_random_differential_between_kernel_families(case_id):
    """The same random problem through the default kernels (bulk-copy pipeline in whichever shape the
    planner picks - box or per-row copies, one to three X buffers, either mixing order - plus the
    short-range kernel on what is left) and through the direct-load kernels alone: identical bits.
    Learner counts up to NB_MAX_K, streams shifted off their 16-byte boundary, padded rows."""
    import torch
    from paper_2211_00889_b200.build import build_library
    build_library()
    from paper_2211_00889_b200 import binding as B
    rng = np.random.default_rng(9000 + case_id)
    variant = str(rng.choice(["allreduce", "ring", "matcha", "centralized"]))
    K = int(rng.choice([1, 2, 3, 7, 16, 17, 25, 33, 48, 64])) if variant != "matcha" else int(rng.choice([4, 8, 16, 24]))
    M = int(rng.integers(1, 21))
    P = int(rng.choice([rng.integers(1, 512), 512 * rng.integers(1, 10), 512 * rng.integers(1, 10) + rng.integers(1, 512)]))
    dtype = torch.bfloat16 if rng.integers(0, 2) else torch.float32
    order = int(rng.integers(0, 2))
    shift = int(rng.choice([0, 0, 1, 3]))
    pad = int(rng.choice([0, 0, 8, 5]))
    fused = bool(rng.integers(0, 2))
    seed = int(rng.integers(0, 2 ** 40))

    def make():
        if variant == "allreduce":
            return B.NbContext(K, P, M, 0.05, 0.9, "allreduce")
        if variant == "ring":
            return B.NbContext(K, P, M, 0.05, 0.9, "dpsgd", B.make_topology("ring"))
        if variant == "matcha":
            topo = B.make_topology("random_regular", degree=3 if K > 4 else 2, seed=seed, alpha=0.2, act_prob=0.6)
            return B.NbContext(K, P, M, 0.05, 0.9, "matcha", topo)
        return B.NbContext(K, P, M, 0.05, 0.9, "centralized")

    a, d = make(), make()
    d.set_option(B.NB_OPT_KERNEL, B.NB_KERNEL_DIRECT)
    x0 = torch.from_numpy((rng.standard_normal(P) * 0.01).astype(np.float32)).cuda()
    for c in (a, d):
        if variant != "centralized":
            c.set_option(B.NB_OPT_ORDER, order)
        c.set_params(x0)
    for t in range(2):
        G = (torch.from_numpy(rng.standard_normal((K, M, P)).astype(np.float32)) * 0.01).to(dtype).cuda()
        flat = torch.zeros(K * M * (P + pad) + shift, dtype=dtype, device="cuda")
        g = flat[shift:].view(K, M, P + pad)[:, :, :P]          # rows P + pad apart, `shift` elements off the allocation
        g.copy_(G)
        n = rng.integers(0, M + 1, K)
        for c in (a, d):
            if fused:
                c.step_fused(g, n)
            else:
                c.accumulate(g, n)
                c.step()
    case = dict(variant=variant, K=K, M=M, P=P, dtype=str(dtype), order=order, shift=shift, pad=pad, fused=fused,
                plan=a.get_kernel_plan())
    assert torch.equal(a.get_params(), d.get_params()), case
    assert torch.equal(a.get_momentum(), d.get_momentum()), case
    a.check_guards(); d.check_guards()
    a.close(); d.close()


@pytest.mark.parametrize("case_id", range(48))
def test_random_differential_with_many_tiles_per_cta(case_id):
    """The differential test in the persistent regime: about 4100 tiles, so that every CTA of every
    kernel shape (up to nine CTAs per SM) takes three or more tiles - ring phases wrap, X buffers are
    reused, the old-models-in-the-ring buffer is handed on from tile to tile - and the default kernels
    must still give the bits of the direct-load kernels."""
    import torch
    from paper_2211_00889_b200.build import build_library
    build_library()
    from paper_2211_00889_b200 import binding as B
    rng = np.random.default_rng(77000 + case_id)
    variant = str(rng.choice(["allreduce", "ring", "matcha", "centralized"]))
    K = int(rng.choice([1, 2, 3, 5, 8, 16, 24, 33, 40, 48, 64])) if variant != "matcha" else int(rng.choice([4, 8, 16, 24]))
    M = int(rng.integers(1, 7 if K >= 33 else 13))
    P = 512 * int(rng.integers(4100, 4300)) + int(rng.choice([0, 8, rng.integers(1, 512)]))
    dtype = torch.bfloat16 if rng.integers(0, 2) else torch.float32
    order = int(rng.integers(0, 2))
    shift = int(rng.choice([0, 0, 1]))
    fused = bool(rng.integers(0, 2))
    seed = int(rng.integers(0, 2 ** 40))

    def make():
        if variant == "allreduce":
            return B.NbContext(K, P, M, 0.05, 0.9, "allreduce")
        if variant == "ring":
            return B.NbContext(K, P, M, 0.05, 0.9, "dpsgd", B.make_topology("ring"))
        if variant == "matcha":
            topo = B.make_topology("random_regular", degree=3 if K > 4 else 2, seed=seed, alpha=0.2, act_prob=0.6)
            return B.NbContext(K, P, M, 0.05, 0.9, "matcha", topo)
        return B.NbContext(K, P, M, 0.05, 0.9, "centralized")

    a, d = make(), make()
    d.set_option(B.NB_OPT_KERNEL, B.NB_KERNEL_DIRECT)
    gen = torch.Generator(device="cuda")
    gen.manual_seed(seed)
    x0 = torch.randn(P, generator=gen, device="cuda") * 0.01
    for c in (a, d):
        if variant != "centralized":
            c.set_option(B.NB_OPT_ORDER, order)
        c.set_params(x0)
    flat = torch.empty(K * M * P + shift, dtype=dtype, device="cuda")
    g = flat[shift:].view(K, M, P)                       # `shift` elements off the allocation's 16-byte boundary
    plan = None
    for t in range(3):
        for i in range(K):                               # drawn learner by learner: no fp32 copy of the whole stream
            g[i].copy_(torch.randn((M, P), generator=gen, device="cuda") * 0.01)
        n = rng.integers(0, M + 1, K)
        for c in (a, d):
            if fused:
                c.step_fused(g, n)
            else:
                c.accumulate(g, n)
                c.step()
        plan = a.get_kernel_plan()
    case = dict(variant=variant, K=K, M=M, P=P, dtype=str(dtype), order=order, shift=shift, fused=fused, plan=plan)
    assert plan["pipeline"] == 1 and plan["tiles"] >= 3 * plan["grid"], case
    assert torch.equal(a.get_params(device="cuda"), d.get_params(device="cuda")), case
    assert torch.equal(a.get_momentum(device="cuda"), d.get_momentum(device="cuda")), case
    a.check_guards(); d.check_guards()
    a.close(); d.close()
    del flat, g
    torch.cuda.empty_cache()
