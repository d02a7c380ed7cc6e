"""Parity at the full sizes of the named configurations, in the launch configuration bench.py
times (dense, aligned gradient stream resident in HBM; nb_step_fused): the computation is
independent per column, so the oracle recomputes a fixed set of column windows exactly - the first
and last tiles, windows across tile boundaries and random windows - from the same input values."""
import numpy as np
import pytest

from oracle import nb_oracle as O
from paper_2211_00889_b200 import workloads as WL
from tests import _harness as H

pytestmark = pytest.mark.gpu


def _windows(P, rng, n_random=24, width=48):
    wins = [(0, min(P, 1040)), (max(0, P - 1040), P)]
    for t in (1, 2, 1000):                                   # straddle 1024-column tile boundaries
        c = t * 1024
        if c + 8 < P:
            wins.append((c - 8, c + 8))
    for _ in range(n_random):
        c = int(rng.integers(0, max(1, P - width)))
        wins.append((c, min(P, c + width)))
    cols = np.unique(np.concatenate([np.arange(a, b) for a, b in wins]))
    return cols


@pytest.mark.parametrize("name,steps", [
    ("cfg2_allreduce_resnet18", 10),
    ("cfg3_dpsgd_ring_resnet50", 10),
    ("cfg4_matcha_vgg16", 4),
    ("cfg5_scale_allreduce", 2),
    ("cfg5_scale_ring", 2),
])
def test_full_size_sampled_columns(name, steps):
    _full_size(WL.WORKLOADS[name], steps)


def test_full_size_rows_not_16_byte_aligned():
    """The benchmark workload with one more column: a dense stream whose rows all start at different
    byte offsets, on the per-row bulk-copy path, in the launch configuration bench.py times."""
    from dataclasses import replace
    w = WL.WORKLOADS["cfg3_dpsgd_ring_resnet50"]
    _full_size(replace(w, P=w.P + 1, name="cfg3 with P + 1 columns"), 4, expect_row_copies=1)


def test_mid_size_every_column():
    """About 600 thousand columns, sixteen learners: every CTA of the persistent kernel takes several
    tiles (stage reuse, ring phase wrap), and EVERY column is compared with the oracle."""
    import torch
    from paper_2211_00889_b200.build import build_library
    build_library()
    from paper_2211_00889_b200 import binding as B
    w = WL.scaled(WL.WORKLOADS["cfg3_dpsgd_ring_resnet50"], 1200 * 512 + 24, steps=3)
    ctx = B.context_for(w)
    orc = H.oracle_for(w, w.P)
    x0 = WL.init_params(w)
    ctx.set_params(torch.from_numpy(x0).cuda())
    orc.set_params(x0)
    for t in range(w.steps):
        n = H.lib_counts(B, w, t)
        payload, values = WL.gradients_np(w, t)
        ctx.step_fused(H.to_device(payload), n)
        orc.step(values, n.tolist())
        del payload, values
    plan = ctx.get_kernel_plan()
    assert plan["pipeline"] == 1 and plan["tiles"] == 1200 and plan["tiles"] >= 3 * plan["grid"]
    H.assert_close(ctx.get_params().numpy(), orc.X, H.TOL_SAME_INPUT, "X")
    H.assert_close(ctx.get_momentum().numpy(), orc.V, H.TOL_SAME_INPUT, "V")
    ctx.check_guards()
    ctx.close()


@pytest.mark.parametrize("dtype,tiles", [("bf16", 3600), ("f32", 1800)])
def test_mid_size_every_column_centralized(dtype, tiles):
    """Alg. 3 on enough tiles that every CTA of the persistent no-stage kernel takes three or more
    (ring phase wrap, the tile loop), every column compared with the oracle; and the same sizes through
    nb_accumulate + nb_step (the masked-accumulate kernel in its persistent regime), and from a stream
    whose rows are not 16-byte aligned (one bulk copy per row), bit for bit."""
    import torch
    from paper_2211_00889_b200.build import build_library
    build_library()
    from paper_2211_00889_b200 import binding as B
    K, M, P = 8, 8, tiles * 512 + 24
    rng = np.random.default_rng(tiles)
    x0 = (rng.standard_normal(P) * 0.01).astype(np.float32)
    fused = B.NbContext(K, P, M, 0.1, 0.9, "centralized")
    unfused = B.NbContext(K, P, M, 0.1, 0.9, "centralized")
    shifted = B.NbContext(K, P, M, 0.1, 0.9, "centralized")   # the same values one element off 16-byte alignment
    for c in (fused, unfused, shifted):
        c.set_params(torch.from_numpy(x0).cuda())
    x, v = x0.astype(np.float64), np.zeros(P)
    tdt = torch.bfloat16 if dtype == "bf16" else torch.float32
    gen = torch.Generator(device="cuda")
    gen.manual_seed(tiles)
    for t in range(3):
        G = (torch.randn((K, M, P), generator=gen, device="cuda", dtype=torch.float32) * 0.01).to(tdt)
        n = rng.integers(0, M + 1, K)
        fused.step_fused(G, n)
        plan = fused.get_kernel_plan()
        unfused.accumulate(G, n)
        unfused.step()
        flat = torch.empty(G.numel() + 1, dtype=G.dtype, device=G.device)
        Gs = flat[1:].view_as(G)
        Gs.copy_(G)
        if t % 2:
            shifted.step_fused(Gs, n)
            assert shifted.get_kernel_plan()["row_copies"] == 1
        else:
            shifted.accumulate(Gs, n)
            shifted.step()
        del Gs, flat
        x, v = O.step_centralized(x, v, G.float().cpu().numpy(), n.tolist(), 0.1, 0.9)
        del G
    assert plan["pipeline"] == 1 and plan["tiles"] == tiles and plan["tiles"] >= 3 * plan["grid"]
    H.assert_close(fused.get_params().numpy(), x, H.TOL_SAME_INPUT, "x")
    H.assert_close(fused.get_momentum().numpy(), v, H.TOL_SAME_INPUT, "v")
    for c in (unfused, shifted):
        assert torch.equal(fused.get_params(), c.get_params())
        assert torch.equal(fused.get_momentum(), c.get_momentum())
    for c in (fused, unfused, shifted):
        c.check_guards()
        c.close()


@pytest.mark.parametrize("K,M,tiles,x_buffers", [(16, 8, 1200, 3), (32, 8, 600, 2), (40, 4, 600, 1)])
def test_mid_size_every_column_update_then_mix(K, M, tiles, x_buffers):
    """Eq. 4-6's order on several tiles per CTA, every column: the deferred averaging pass over three X
    buffers (K = 16), the half-deferred pass over two (K = 32), and the single buffer whose old model
    rows travel in the ring items (K = 40)."""
    import torch
    from dataclasses import replace
    from paper_2211_00889_b200.build import build_library
    build_library()
    from paper_2211_00889_b200 import binding as B
    w = replace(WL.scaled(WL.WORKLOADS["cfg3_dpsgd_ring_resnet50"], tiles * 512 + 24, steps=3), K=K, M=M)
    ctx = B.context_for(w)
    ctx.set_option(B.NB_OPT_ORDER, B.NB_ORDER_UPDATE_THEN_MIX)
    orc = H.oracle_for(w, w.P, order="update_then_mix")
    x0 = WL.init_params(w)
    ctx.set_params(torch.from_numpy(x0).cuda())
    orc.set_params(x0)
    for t in range(w.steps):
        n = H.lib_counts(B, w, t)
        payload, values = WL.gradients_np(w, t)
        ctx.step_fused(H.to_device(payload), n)
        orc.step(values, n.tolist())
        del payload, values
    plan = ctx.get_kernel_plan()
    assert plan["pipeline"] == 1 and plan["x_buffers"] == x_buffers and plan["tiles"] >= 3 * plan["grid"]
    H.assert_close(ctx.get_params().numpy(), orc.X, H.TOL_SAME_INPUT, "X")
    H.assert_close(ctx.get_momentum().numpy(), orc.V, H.TOL_SAME_INPUT, "V")
    ctx.check_guards()
    ctx.close()


@pytest.mark.parametrize("K,M,order", [(2, 2, "mix_then_update"), (3, 8, "mix_then_update"), (5, 3, "update_then_mix")])
def test_mid_size_every_column_few_learners(K, M, order):
    """Few learners run four CTAs per SM of one consumer group each; 2400 tiles give every CTA four or
    more of them, and every column is compared with the oracle."""
    import torch
    from dataclasses import replace
    from paper_2211_00889_b200.build import build_library
    build_library()
    from paper_2211_00889_b200 import binding as B
    w = replace(WL.scaled(WL.WORKLOADS["cfg3_dpsgd_ring_resnet50"], 2400 * 512 + 24, steps=3), K=K, M=M)
    ctx = B.context_for(w)
    if order == "update_then_mix":
        ctx.set_option(B.NB_OPT_ORDER, B.NB_ORDER_UPDATE_THEN_MIX)
    orc = H.oracle_for(w, w.P, order=order)
    x0 = WL.init_params(w)
    ctx.set_params(torch.from_numpy(x0).cuda())
    orc.set_params(x0)
    for t in range(w.steps):
        n = H.lib_counts(B, w, t)
        payload, values = WL.gradients_np(w, t)
        ctx.step_fused(H.to_device(payload), n)
        orc.step(values, n.tolist())
        del payload, values
    plan = ctx.get_kernel_plan()
    assert plan["pipeline"] == 1 and plan["groups"] == 1 and plan["tiles"] >= 4 * plan["grid"]
    H.assert_close(ctx.get_params().numpy(), orc.X, H.TOL_SAME_INPUT, "X")
    H.assert_close(ctx.get_momentum().numpy(), orc.V, H.TOL_SAME_INPUT, "V")
    ctx.check_guards()
    ctx.close()


def test_more_than_two_to_the_31_columns():
    """Column indices beyond 32 bits: one learner pair, 2^31 + 1544 columns (the last window the
    oracle checks lies entirely above 2^31)."""
    from dataclasses import replace
    w = replace(WL.WORKLOADS["cfg3_dpsgd_ring_resnet50"], K=2, M=2, P=2 ** 31 + 3 * 512 + 8, name="two_to_31_columns")
    _full_size(w, 2)


def _full_size(w, steps, expect_row_copies=0):
    import torch
    from paper_2211_00889_b200.build import build_library
    build_library()
    from paper_2211_00889_b200 import binding as B
    name = w.name
    es = 4 if w.grad_dtype == "f32" else 2
    need = w.K * w.M * w.P * es + 4 * w.K * w.P * 4 + w.M * w.P * 4 + (2 << 30)
    torch.cuda.empty_cache()
    free, _ = torch.cuda.mem_get_info()
    if free < need:
        pytest.skip("needs %.0f GB of free device memory" % (need / 1e9))
    cols = _windows(w.P, np.random.default_rng(w.seed))
    cols_dev = torch.from_numpy(cols).cuda()
    gen = torch.Generator(device="cuda")
    gen.manual_seed(w.seed)
    x0 = torch.randn(w.P, generator=gen, device="cuda", dtype=torch.float32) * w.init_sigma
    ctx = B.context_for(w)
    ctx.set_params(x0)
    orc = H.oracle_for(w, len(cols))
    orc.set_params(x0[cols_dev].cpu().numpy())
    del x0
    for t in range(steps):
        n = H.lib_counts(B, w, t)
        G = WL.gradients_torch(w, t, "cuda")
        ctx.step_fused(G, n)
        Gs = G[:, :, cols_dev].float().cpu().numpy()          # exact values of the sampled columns
        torch.cuda.synchronize()
        del G
        orc.step(Gs, n.tolist())
        if w.variant == "matcha":
            bits, Wdev = ctx.get_device_mixing()
            assert bits == O.matcha_activation(w.seed, t, len(orc.partner), w.act_prob)
    torch.cuda.empty_cache()
    plan = ctx.get_kernel_plan()
    assert plan["pipeline"] == 1 and plan["row_copies"] == expect_row_copies
    X = ctx.get_params(device="cuda")[:, cols_dev].cpu().numpy()
    V = ctx.get_momentum(device="cuda")[:, cols_dev].cpu().numpy()
    ctx.check_guards()
    ctx.close()
    torch.cuda.empty_cache()
    H.assert_close(X, orc.X, H.TOL_SAME_INPUT, name + " X")
    H.assert_close(V, orc.V, H.TOL_SAME_INPUT, name + " V")
