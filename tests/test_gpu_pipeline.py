"""Edge cases of the bulk-copy pipeline kernel and of its hand-over to the direct-load kernel:
sizes around one tile, many learners, more mini-batches than one ring item holds, learners with
nothing finished, and bitwise agreement between the two kernels on the same values."""
from dataclasses import replace

import numpy as np
import pytest

from oracle import nb_oracle as O
from paper_2211_00889_b200 import workloads as WL
from tests import _harness as H

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def B():
    from paper_2211_00889_b200.build import build_library
    build_library()
    from paper_2211_00889_b200 import binding
    return binding


def _against_oracle(B, w, steps, counts=None, fused=True):
    import torch
    ctx = B.context_for(w)
    orc = H.oracle_for(w, w.P)
    x0 = WL.init_params(w)
    ctx.set_params(torch.from_numpy(x0).cuda())
    orc.set_params(x0)
    launches = []
    for t in range(steps):
        n = counts[t] if counts is not None else H.lib_counts(B, w, t)
        payload, values = WL.gradients_np(w, t)
        before = ctx.get_stats()["kernel_launches"]
        if fused:
            ctx.step_fused(H.to_device(payload), n)
        else:
            ctx.accumulate(H.to_device(payload), n)
            ctx.step()
        launches.append(ctx.get_stats()["kernel_launches"] - before)
        orc.step(values, [int(v) for v in n])
    H.assert_close(ctx.get_params().numpy(), orc.X, H.TOL_SAME_INPUT, w.name)
    H.assert_close(ctx.get_momentum().numpy(), orc.V, H.TOL_SAME_INPUT, w.name)
    ctx.check_guards()
    ctx.close()
    return launches


@pytest.mark.parametrize("P,expected_launches", [
    (512, 1),            # exactly one tile: pipeline kernel only
    (512 + 8, 2),        # one tile + an 8-column tail for the direct kernel
    (3 * 512, 1),
    (511, 1),            # below one tile (and unaligned): direct kernel only
    (256, 1),
    (2 * 512 + 1, 2),    # odd row length: one tile of per-row bulk copies (the second would read past
                         # the end of the last row) + a 513-column tail
    (2 * 512 + 8, 2),    # rows are 16-byte multiples again: two tiles of box copies + 8 columns
    (512 + 7, 1),        # odd and shorter than one tile plus the 16 bytes a row copy may over-read
])
def test_sizes_around_one_tile(B, P, expected_launches):
    w = WL.scaled(WL.WORKLOADS["cfg3_dpsgd_ring_resnet50"], P, steps=3)
    launches = _against_oracle(B, w, w.steps)
    assert launches == [expected_launches] * w.steps


def test_bench_workload_runs_on_the_pipeline_kernel(B):
    """The shape the planner picks for the benchmark workload (a narrow slice of it is enough)."""
    import torch
    w = WL.scaled(WL.WORKLOADS["cfg3_dpsgd_ring_resnet50"], 8 * 512, steps=1)
    ctx = B.context_for(w)
    ctx.set_params(torch.from_numpy(WL.init_params(w)).cuda())
    assert ctx.get_kernel_plan()["pipeline"] == 0                      # nothing has run yet
    ctx.step_fused(H.to_device(WL.gradients_np(w, 0)[0]), H.lib_counts(B, w, 0))
    plan = ctx.get_kernel_plan()
    assert plan["pipeline"] == 1 and plan["tile"] == 512 and plan["tiles"] == 8
    assert plan["groups"] >= 1 and plan["slots"] >= 2 * plan["groups"] and plan["smem_bytes"] <= 227 * 1024
    ctx.close()


@pytest.mark.parametrize("K", [2, 3, 17, 33, 64])
@pytest.mark.parametrize("variant", ["dpsgd", "allreduce"])
def test_learner_counts(B, K, variant):
    base = WL.WORKLOADS["cfg3_dpsgd_ring_resnet50" if variant == "dpsgd" else "cfg2_allreduce_resnet18"]
    w = replace(WL.scaled(base, 2 * 512 + 24, steps=3), K=K)
    _against_oracle(B, w, w.steps)
    _against_oracle(B, w, w.steps, fused=False)


@pytest.mark.parametrize("dtype", ["bf16", "f32"])
@pytest.mark.parametrize("M", [1, 9, 20])
def test_more_minibatches_than_one_ring_item(B, dtype, M):
    w = replace(WL.scaled(WL.WORKLOADS["cfg3_dpsgd_ring_resnet50"], 3 * 512 + 16, steps=3), M=M, grad_dtype=dtype, K=6)
    _against_oracle(B, w, w.steps)
    rng = np.random.default_rng(M)
    counts = [rng.integers(0, M + 1, w.K) for _ in range(w.steps)]      # includes learners with nothing finished
    counts[1][:] = 0
    counts[2][:] = M
    _against_oracle(B, w, w.steps, counts=counts)


def test_matcha_and_options_on_pipeline_sizes(B):
    import torch
    w = WL.scaled(WL.WORKLOADS["cfg4_matcha_vgg16"], 4 * 512, steps=4)
    for norm, order in ((B.NB_NORM_PAPER, B.NB_ORDER_UPDATE_THEN_MIX), (B.NB_NORM_MEAN, B.NB_ORDER_UPDATE_THEN_MIX)):
        ctx = B.context_for(w)
        ctx.set_option(B.NB_OPT_NORM, norm)
        ctx.set_option(B.NB_OPT_ORDER, order)
        orc = H.oracle_for(w, w.P, "paper" if norm == B.NB_NORM_PAPER else "mean", "update_then_mix")
        x0 = WL.init_params(w)
        ctx.set_params(torch.from_numpy(x0).cuda()); orc.set_params(x0)
        for t in range(w.steps):
            n = H.lib_counts(B, w, t)
            payload, values = WL.gradients_np(w, t)
            ctx.step_fused(H.to_device(payload), n)
            orc.step(values, n.tolist())
        H.assert_close(ctx.get_params().numpy(), orc.X, H.TOL_SAME_INPUT)
        ctx.close()


def _shifted_view(g, by=1):
    """The same values `by` elements further into a fresh buffer: rows lose their 16-byte alignment."""
    import torch
    flat = torch.empty(g.numel() + by, dtype=g.dtype, device=g.device)
    out = flat[by:].view_as(g)
    out.copy_(g)
    return out


@pytest.mark.parametrize("name", ["cfg2_allreduce_resnet18", "cfg3_dpsgd_ring_resnet50", "cfg4_matcha_vgg16",
                                  "cfg5_scale_ring"])
@pytest.mark.parametrize("order", [0, 1])
@pytest.mark.parametrize("P", [5 * 512 + 40, 5 * 512 + 41, 5 * 512 + 44])
def test_pipeline_and_direct_kernels_agree_bitwise(B, name, order, P):
    """The same values reach the library four ways: as a 16-byte aligned dense stream (for P = 5*512+40
    every row is a 16-byte multiple: box copies; for the odd P and for P = 4 mod 8 in bf16 the rows
    are not: one bulk copy per row), shifted by one element (the stream itself starts off a 16-byte
    boundary: the first tile goes to the direct-load kernel), shifted by three, and through the
    direct-load kernels alone.  Identical bits every time."""
    import torch
    w = WL.scaled(WL.WORKLOADS[name], P, steps=3)
    es = 2 if w.grad_dtype == "bf16" else 4
    rows_aligned = (P * es) % 16 == 0
    ctxs = [B.context_for(w) for _ in range(4)]
    a, b, b3, d = ctxs
    d.set_option(B.NB_OPT_KERNEL, B.NB_KERNEL_DIRECT)
    for c in ctxs:
        c.set_option(B.NB_OPT_ORDER, order)
        c.set_params(torch.from_numpy(WL.init_params(w)).cuda())
    extra = 1 if w.variant == "matcha" else 0
    for t in range(w.steps):
        n = H.lib_counts(B, w, t)
        g = H.to_device(WL.gradients_np(w, t)[0])
        streams = (g, _shifted_view(g, 1), _shifted_view(g, 3), g)
        want_launches = (2, 3, 3, 1)       # pipeline + tail; head + pipeline + tail; the same; direct only
        want_row_copies = (0 if rows_aligned else 1, 1, 1, 0)
        for c, gs, wl, wr in zip(ctxs, streams, want_launches, want_row_copies):
            before = c.get_stats()["kernel_launches"]
            c.step_fused(gs, n)
            assert c.get_stats()["kernel_launches"] - before == wl + extra
            plan = c.get_kernel_plan()
            assert plan["pipeline"] == (0 if c is d else 1)
            if c is not d:
                assert plan["row_copies"] == wr and plan["head"] == (512 if c in (b, b3) else 0)
                assert plan["head"] + plan["tiles"] * plan["tile"] <= P
    for c in (b, b3, d):
        assert torch.equal(a.get_params(), c.get_params())
        assert torch.equal(a.get_momentum(), c.get_momentum())
    for c in ctxs:
        c.check_guards()
        c.close()


@pytest.mark.parametrize("dtype", ["bf16", "f32"])
@pytest.mark.parametrize("variant", ["dpsgd", "allreduce"])
def test_unaligned_rows_against_the_oracle(B, dtype, variant):
    """Odd row length on the per-row bulk-copy path, several tiles per CTA's worth of columns, every
    row at a different byte shift, checked against the oracle (not only against the other kernels)."""
    base = WL.WORKLOADS["cfg3_dpsgd_ring_resnet50" if variant == "dpsgd" else "cfg2_allreduce_resnet18"]
    w = replace(WL.scaled(base, 7 * 512 + 5, steps=4), grad_dtype=dtype, K=5, M=11)
    rng = np.random.default_rng(5)
    counts = [rng.integers(0, w.M + 1, w.K) for _ in range(w.steps)]
    counts[0][:] = w.M
    _against_oracle(B, w, w.steps, counts=counts)
    _against_oracle(B, w, w.steps, counts=counts, fused=False)


@pytest.mark.parametrize("dtype,P", [("bf16", 4 * 512 + 40), ("f32", 3 * 512 + 12), ("bf16", 512)])
@pytest.mark.parametrize("fused", [True, False])
def test_centralized_step_on_pipeline_sizes(B, dtype, P, fused):
    """Alg. 3 through the no-stage pipeline kernel: oracle parity, and the same bits from box copies
    (aligned rows), per-row bulk copies (the stream shifted by one element) and the direct-load kernel."""
    import torch
    K, M = 8, 8
    rng = np.random.default_rng(11)
    x0 = (rng.standard_normal(P) * 0.01).astype(np.float32)
    a = B.NbContext(K, P, M, 0.1, 0.9, "centralized")
    b = B.NbContext(K, P, M, 0.1, 0.9, "centralized")
    d = B.NbContext(K, P, M, 0.1, 0.9, "centralized")
    d.set_option(B.NB_OPT_KERNEL, B.NB_KERNEL_DIRECT)
    for c in (a, b, d):
        c.set_params(torch.from_numpy(x0).cuda())
    x, v = x0.astype(np.float64), np.zeros(P)
    tdt = torch.bfloat16 if dtype == "bf16" else torch.float32
    for t in range(4):
        G = (torch.from_numpy(rng.standard_normal((K, M, P)).astype(np.float32)) * 0.01).to(tdt).cuda()
        n = rng.integers(0, M + 1, K)
        shifted = _shifted_view(G)
        if fused:
            a.step_fused(G, n); b.step_fused(shifted, n); d.step_fused(G, n)
        else:
            a.accumulate(G, n); a.step()
            b.accumulate(shifted, n); b.step()
            d.accumulate(G, n); d.step()
        x, v = O.step_centralized(x, v, G.float().cpu().numpy(), n.tolist(), 0.1, 0.9)
    H.assert_close(a.get_params().numpy(), x, H.TOL_SAME_INPUT)
    H.assert_close(a.get_momentum().numpy(), v, H.TOL_SAME_INPUT)
    assert torch.equal(a.get_params(), b.get_params()) and torch.equal(a.get_momentum(), b.get_momentum())
    assert torch.equal(a.get_params(), d.get_params()) and torch.equal(a.get_momentum(), d.get_momentum())
    a.close(); b.close(); d.close()


@pytest.mark.parametrize("dtype", ["bf16", "f32"])
@pytest.mark.parametrize("M", [3, 8, 19])
def test_accumulate_on_pipeline_sizes(B, dtype, M):
    import torch
    K, P = 7, 3 * 512 + 24
    rng = np.random.default_rng(M)
    tdt = torch.bfloat16 if dtype == "bf16" else torch.float32
    a = B.NbContext(K, P, M, 0.1, 0.9, "allreduce")
    b = B.NbContext(K, P, M, 0.1, 0.9, "allreduce")
    d = B.NbContext(K, P, M, 0.1, 0.9, "allreduce")
    d.set_option(B.NB_OPT_KERNEL, B.NB_KERNEL_DIRECT)
    G = torch.from_numpy(rng.standard_normal((K, M, P)).astype(np.float32)).to(tdt).cuda()
    n = rng.integers(0, M + 1, K)
    n[0], n[1] = 0, M
    shifted = _shifted_view(G)
    la = a.get_stats()["kernel_launches"]
    a.accumulate(G, n)
    assert a.get_stats()["kernel_launches"] - la == 2            # pipeline kernel + 24-column tail
    lb = b.get_stats()["kernel_launches"]
    b.accumulate(shifted, n)
    assert b.get_stats()["kernel_launches"] - lb == 3            # first tile + per-row bulk copies + tail
    ld = d.get_stats()["kernel_launches"]
    d.accumulate(G, n)
    assert d.get_stats()["kernel_launches"] - ld == 1            # direct-load kernel only
    acc = a.get_accumulator()
    assert torch.equal(acc, b.get_accumulator()) and torch.equal(acc, d.get_accumulator())
    H.assert_close(acc.numpy(), O.accumulate(G.float().cpu().numpy(), n.tolist()), 2e-6)
    assert float(acc[0].abs().max()) == 0.0
    a.close(); b.close(); d.close()


@pytest.mark.parametrize("K", [1, 2, 5, 31, 64])
@pytest.mark.parametrize("variant,order", [("dpsgd", 0), ("dpsgd", 1), ("allreduce", 0), ("allreduce", 1),
                                           ("centralized", 0)])   # one shared model has no mixing order
def test_short_range_kernel_agrees_with_the_direct_kernel_bitwise(B, K, variant, order):
    """Column ranges of a few hundred columns (ragged tails, problems narrower than a tile) run on the
    learner-parallel kernel (a thread owns one learner's 4 columns); NB_KERNEL_DIRECT runs the same
    problem on the column-per-thread kernel.  Same bits, any learner count up to NB_MAX_K, both
    orders, all mixing modes, aligned and unaligned rows, fused and unfused."""
    import torch
    for P, dtype in ((300, "bf16"), (515, "f32"), (7, "bf16"), (512 + 129, "bf16")):
        rng = np.random.default_rng(1000 * K + P)
        M = 5
        topo = B.make_topology("ring") if variant == "dpsgd" else None
        ctxs = [B.NbContext(K, P, M, 0.05, 0.9, variant, topo) for _ in range(3)]
        a, u, d = ctxs                                   # fused, unfused, direct kernels only
        d.set_option(B.NB_OPT_KERNEL, B.NB_KERNEL_DIRECT)
        x0 = (rng.standard_normal(P) * 0.01).astype(np.float32)
        for c in ctxs:
            if variant != "centralized":
                c.set_option(B.NB_OPT_ORDER, order)
            c.set_params(torch.from_numpy(x0).cuda())
        tdt = torch.bfloat16 if dtype == "bf16" else torch.float32
        for t in range(3):
            G = (torch.from_numpy(rng.standard_normal((K, M, P)).astype(np.float32)) * 0.01).to(tdt).cuda()
            n = rng.integers(0, M + 1, K)
            a.step_fused(G, n)
            u.accumulate(G, n); u.step()
            d.step_fused(G, n)
            assert d.get_kernel_plan()["pipeline"] == 0
        for c in (u, d):
            assert torch.equal(a.get_params(), c.get_params()) and torch.equal(a.get_momentum(), c.get_momentum())
        for c in ctxs:
            c.check_guards()
            c.close()


def test_aligned_and_unaligned_streams_interleave(B):
    """A context may see aligned streams (box copies) and unaligned ones (per-row bulk copies plus a
    first tile on the direct-load kernel) in any order; state and results must be those of a context
    that only ever saw aligned streams."""
    import torch
    w = WL.scaled(WL.WORKLOADS["cfg5_scale_ring"], 4 * 512 + 40, steps=6)
    ref, mix = B.context_for(w), B.context_for(w)
    x0 = torch.from_numpy(WL.init_params(w)).cuda()
    ref.set_params(x0); mix.set_params(x0)
    for t in range(w.steps):
        n = H.lib_counts(B, w, t)
        g = H.to_device(WL.gradients_np(w, t)[0])
        ref.step_fused(g, n)
        if t in (1, 2, 4):                                   # unaligned view of the same values
            mix.step_fused(_shifted_view(g), n)
            assert mix.get_kernel_plan()["row_copies"] == 1 and mix.get_kernel_plan()["head"] == 512
        else:
            mix.step_fused(g, n)
            assert mix.get_kernel_plan()["row_copies"] == 0 and mix.get_kernel_plan()["head"] == 0
        if t == 2:                                           # checkpoint in between
            X, V, step = mix.get_params(), mix.get_momentum(), mix.get_step()
            mix.set_state(step, X, V)
        assert torch.equal(ref.get_params(), mix.get_params())
    assert torch.equal(ref.get_momentum(), mix.get_momentum())
    assert torch.equal(ref.get_mean_params(), mix.get_mean_params())
    mix.check_guards()
    ref.close(); mix.close()


def test_a_wait_that_runs_out_is_reported_and_the_context_stays_usable(B):
    """The kernels' barrier waits are bounded.  The self-test makes one run out on purpose (a barrier
    phase that nothing completes, limit ~1 ms): the lanes give up, the error word carries the code,
    the kernel returns, and the context then steps normally."""
    import torch
    w = WL.scaled(WL.WORKLOADS["cfg3_dpsgd_ring_resnet50"], 2 * 512, steps=2)
    ctx = B.context_for(w)
    orc = H.oracle_for(w, w.P)
    x0 = WL.init_params(w)
    ctx.set_params(torch.from_numpy(x0).cuda()); orc.set_params(x0)
    ctx.selftest_wait_timeout()
    for t in range(w.steps):
        n = H.lib_counts(B, w, t)
        payload, values = WL.gradients_np(w, t)
        ctx.step_fused(H.to_device(payload), n)
        orc.step(values, n.tolist())
        if t == 0:
            ctx.selftest_wait_timeout()                     # between steps as well
    H.assert_close(ctx.get_params().numpy(), orc.X, H.TOL_SAME_INPUT)
    ctx.check_guards()                                      # also reads the (cleared) device error word
    ctx.close()
