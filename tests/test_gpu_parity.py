"""GPU parity: the CUDA path, called through the C ABI, against the fp64 CPU oracle on the same
seeded inputs.  Bit-exact for finished counts, masks and MATCHA activations; norm-wise 1e-5 on
parameters against the oracle fed the same input values; 2e-3 for bf16 gradient inputs against
the oracle fed the un-rounded fp32 gradients."""
from dataclasses import replace

import numpy as np
import pytest

from oracle import nb_oracle as O
from paper_2211_00889_b200 import workloads as WL
from tests import _harness as H

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def B():
    import torch
    assert torch.cuda.is_available()
    from paper_2211_00889_b200.build import build_library
    build_library()
    from paper_2211_00889_b200 import binding
    return binding


def _run(B, w, steps, fused=True, norm="mean", order="mix_then_update", check_steps=(10,), with_unrounded=False,
         pad=0):
    """Runs library and oracle side by side; returns per-check-step errors."""
    import torch
    ctx = B.context_for(w)
    ctx.set_option(B.NB_OPT_NORM, B.NB_NORM_MEAN if norm == "mean" else B.NB_NORM_PAPER)
    ctx.set_option(B.NB_OPT_ORDER, B.NB_ORDER_MIX_THEN_UPDATE if order == "mix_then_update" else B.NB_ORDER_UPDATE_THEN_MIX)
    orc = H.oracle_for(w, w.P, norm, order)
    orc_unr = H.oracle_for(w, w.P, norm, order) if with_unrounded else None
    x0 = WL.init_params(w)
    ctx.set_params(torch.from_numpy(x0).cuda())
    orc.set_params(x0)
    if orc_unr:
        orc_unr.set_params(x0)
    out = {}
    for t in range(steps):
        n = H.lib_counts(B, w, t)
        payload, values, unr = WL.gradients_np(w, t, with_unrounded=True)
        if pad:
            buf = np.zeros((w.K, w.M, w.P + pad), dtype=payload.dtype)
            buf[:, :, :w.P] = payload
            g = H.to_device(buf)
            ld = dict(ld_m=w.P + pad, ld_k=w.M * (w.P + pad))
        else:
            g = H.to_device(payload)
            ld = {}
        g_before = g.clone()
        if fused:
            ctx.step_fused(g, n, **ld)
        else:
            ctx.accumulate(g, n, **ld)
            ctx.step()
        assert torch.equal(g.view(torch.int16) if g.dtype == torch.bfloat16 else g,
                           g_before.view(torch.int16) if g.dtype == torch.bfloat16 else g_before)   # G is read-only
        orc.step(values, n.tolist())
        if orc_unr:
            orc_unr.step(unr, n.tolist())
        if w.variant == "matcha":
            bits, Wdev = ctx.get_device_mixing()
            want = O.matcha_activation(w.seed, t, len(orc.partner), w.act_prob)
            assert bits == want == ctx.get_matcha_activation(t)          # bit-exact activation word
            assert np.array_equal(Wdev, ctx.get_W(t))                     # device builder == host builder
            assert np.abs(Wdev - O.matcha_W(orc.partner, want, w.alpha, w.K)).max() < 1e-7
        if (t + 1) in check_steps or t == steps - 1:
            X = ctx.get_params().numpy()
            V = ctx.get_momentum().numpy()
            e = H.assert_close(X, orc.X, H.TOL_SAME_INPUT, "%s step %d X" % (w.name, t + 1))
            H.assert_close(V, orc.V, H.TOL_SAME_INPUT, "%s step %d V" % (w.name, t + 1))
            H.assert_close(ctx.get_mean_params().numpy(), O.mean_params(orc.X), H.TOL_SAME_INPUT, "mean model")
            if orc_unr:
                H.assert_close(X, orc_unr.X, H.TOL_BF16_ROUNDING, "%s step %d X vs un-rounded" % (w.name, t + 1))
            out[t + 1] = e
    assert ctx.get_step() == steps
    ctx.check_guards()            # no kernel wrote outside X, V or the accumulator
    ctx.close()
    return out


# ----------------------------------------------------------------------------------------------
# The five configurations, at sizes the oracle finishes in seconds that span several column
# tiles and a ragged tail (cfg1 is run at its real size).
# ----------------------------------------------------------------------------------------------
def test_cfg1_tiny_allreduce_exact_size(B):
    w = WL.WORKLOADS["cfg1_tiny_allreduce"]
    _run(B, w, w.steps, fused=True)
    _run(B, w, w.steps, fused=False)


@pytest.mark.parametrize("name,P", [
    ("cfg2_allreduce_resnet18", 5 * 1024 + 260),
    ("cfg3_dpsgd_ring_resnet50", 4 * 1024 + 520),
    ("cfg4_matcha_vgg16", 3 * 1024 + 8),
    ("cfg5_scale_allreduce", 2 * 1024 + 36),
    ("cfg5_scale_ring", 2 * 1024 + 36),
])
@pytest.mark.parametrize("fused", [True, False])
def test_configs_scaled_columns(B, name, P, fused):
    w = WL.scaled(WL.WORKLOADS[name], P, steps=12)
    _run(B, w, w.steps, fused=fused, check_steps=(10,), with_unrounded=(w.grad_dtype == "bf16"))


@pytest.mark.parametrize("name", ["cfg2_allreduce_resnet18", "cfg3_dpsgd_ring_resnet50", "cfg4_matcha_vgg16",
                                  "cfg5_scale_allreduce", "cfg5_scale_ring"])
def test_configs_for_their_full_number_of_steps(B, name):
    """Every configuration for as many steps as it names (50, 50, 20, 20, 20), on a column range of a
    few tiles: the tolerance holds after 10 steps (where the contract states it) and still at the end."""
    w = WL.scaled(WL.WORKLOADS[name], 2 * 1024 + 72)
    assert w.steps in (20, 50)
    errs = _run(B, w, w.steps, fused=True, check_steps=(10, w.steps), with_unrounded=(w.grad_dtype == "bf16"))
    assert set(errs) == {10, w.steps}


@pytest.mark.parametrize("name", ["cfg2_allreduce_resnet18", "cfg3_dpsgd_ring_resnet50", "cfg4_matcha_vgg16"])
@pytest.mark.parametrize("P", [1, 3, 7, 4099, 1025])
def test_ragged_and_unaligned_sizes(B, name, P):
    # P not a multiple of 4: rows of the dense stream are not 16-byte aligned -> scalar-load kernels
    w = WL.scaled(WL.WORKLOADS[name], P, steps=4)
    _run(B, w, w.steps, fused=True)
    _run(B, w, w.steps, fused=False)


@pytest.mark.parametrize("name", ["cfg2_allreduce_resnet18", "cfg3_dpsgd_ring_resnet50"])
def test_padded_rows_take_the_vector_path_with_a_partial_last_vector(B, name):
    # P = 4099 with row pitch 4104: aligned rows, last vector has 3 valid columns
    w = WL.scaled(WL.WORKLOADS[name], 4099, steps=3)
    _run(B, w, w.steps, fused=True, pad=5)
    _run(B, w, w.steps, fused=False, pad=5)


@pytest.mark.parametrize("name", ["cfg1_tiny_allreduce", "cfg3_dpsgd_ring_resnet50", "cfg4_matcha_vgg16"])
@pytest.mark.parametrize("norm,order", [("paper", "mix_then_update"), ("mean", "update_then_mix"),
                                        ("paper", "update_then_mix")])
def test_norm_and_order_options(B, name, norm, order):
    w = WL.scaled(WL.WORKLOADS[name], 2 * 1024 + 100, steps=6)
    _run(B, w, w.steps, fused=True, norm=norm, order=order)
    _run(B, w, w.steps, fused=False, norm=norm, order=order)


# ----------------------------------------------------------------------------------------------
# Self-consistency of the CUDA path (bitwise)
# ----------------------------------------------------------------------------------------------
@pytest.mark.parametrize("name", ["cfg2_allreduce_resnet18", "cfg3_dpsgd_ring_resnet50", "cfg4_matcha_vgg16",
                                  "cfg5_scale_ring"])
def test_fused_equals_unfused_bitwise(B, name):
    import torch
    w = WL.scaled(WL.WORKLOADS[name], 3 * 1024 + 404, steps=5)
    a, b = B.context_for(w), B.context_for(w)
    x0 = torch.from_numpy(WL.init_params(w)).cuda()
    a.set_params(x0)
    b.set_params(x0)
    for t in range(w.steps):
        n = H.lib_counts(B, w, t)
        g = H.to_device(WL.gradients_np(w, t)[0])
        a.step_fused(g, n)
        b.accumulate(g, n)
        b.step()
    assert torch.equal(a.get_params(), b.get_params())
    assert torch.equal(a.get_momentum(), b.get_momentum())
    a.close(); b.close()


@pytest.mark.parametrize("name", ["cfg3_dpsgd_ring_resnet50", "cfg4_matcha_vgg16", "cfg2_allreduce_resnet18"])
def test_column_subset_equals_full_run_bitwise(B, name):
    """Columns never interact: running a column slice alone gives the same bits as the full run."""
    import torch
    P, c0, c1 = 4 * 1024 + 96, 1024 + 8, 3 * 1024 + 40
    w = WL.scaled(WL.WORKLOADS[name], P, steps=4)
    ws = replace(w, P=c1 - c0)
    full, part = B.context_for(w), B.context_for(ws)
    x0 = WL.init_params(w)
    full.set_params(torch.from_numpy(x0).cuda())
    part.set_params(torch.from_numpy(x0[c0:c1].copy()).cuda())
    for t in range(w.steps):
        n = H.lib_counts(B, w, t)
        payload = WL.gradients_np(w, t)[0]
        full.step_fused(H.to_device(payload), n)
        part.step_fused(H.to_device(payload[:, :, c0:c1]), n)
    assert torch.equal(full.get_params()[:, c0:c1], part.get_params())
    full.close(); part.close()


def test_strided_view_of_a_wider_stream_equals_dense(B):
    """ld_m / ld_k: a column window of a wider gradient buffer, addressed in place."""
    import torch
    P, c0, c1 = 3 * 1024, 512, 2 * 1024 + 512
    w = WL.scaled(WL.WORKLOADS["cfg3_dpsgd_ring_resnet50"], P, steps=3)
    ws = replace(w, P=c1 - c0)
    a, b = B.context_for(ws), B.context_for(ws)
    x0 = torch.from_numpy(WL.init_params(ws)).cuda()
    a.set_params(x0); b.set_params(x0)
    for t in range(w.steps):
        n = H.lib_counts(B, w, t)
        g = H.to_device(WL.gradients_np(w, t)[0])
        view = g[:, :, c0:c1]                      # not contiguous
        a.step_fused(view, n, ld_m=P, ld_k=w.M * P)
        b.step_fused(view.contiguous(), n)
    assert torch.equal(a.get_params(), b.get_params())
    a.close(); b.close()


def test_checkpoint_resume_is_bitwise(B):
    import torch
    w = WL.scaled(WL.WORKLOADS["cfg4_matcha_vgg16"], 2 * 1024 + 12, steps=10)
    x0 = torch.from_numpy(WL.init_params(w)).cuda()
    straight = B.context_for(w)
    straight.set_params(x0)
    first = B.context_for(w)
    first.set_params(x0)
    for t in range(10):
        n = H.lib_counts(B, w, t)
        g = H.to_device(WL.gradients_np(w, t)[0])
        straight.step_fused(g, n)
        if t < 5:
            first.step_fused(g, n)
    X, V, step = first.get_params(), first.get_momentum(), first.get_step()
    first.close()
    second = B.context_for(w)
    second.set_state(step, X, V)                     # host tensors in
    for t in range(5, 10):
        n = H.lib_counts(B, w, t)
        second.step_fused(H.to_device(WL.gradients_np(w, t)[0]), n)
    assert torch.equal(second.get_params(), straight.get_params())
    assert torch.equal(second.get_momentum(), straight.get_momentum())
    straight.close(); second.close()


# ----------------------------------------------------------------------------------------------
# Exact-arithmetic cases: every fp32 operation is exact, so GPU == oracle bit for bit
# ----------------------------------------------------------------------------------------------
@pytest.mark.parametrize("variant", ["allreduce", "dpsgd_identity", "matcha"])
def test_exact_arithmetic_matches_oracle_bit_for_bit(B, variant):
    import torch
    K, P, M = 4, 1024 + 36, 4
    lr, mom = 0.25, 0.5
    rng = np.random.default_rng(17)
    x0 = (rng.integers(-64, 65, P) / 4.0).astype(np.float32)
    if variant == "allreduce":
        ctx = B.NbContext(K, P, M, lr, mom, "allreduce")
        orc = O.Oracle(K, P, M, lr, mom, "allreduce")
    elif variant == "dpsgd_identity":
        csr = (np.arange(K + 1), np.arange(K), np.ones(K))
        ctx = B.NbContext(K, P, M, lr, mom, "dpsgd", B.make_topology("csr", csr=csr))
        orc = O.Oracle(K, P, M, lr, mom, "dpsgd", W=O.identity_W(K))
    else:
        partner = [[1, 0, 3, 2], [2, 3, 0, 1]]
        ctx = B.NbContext(K, P, M, lr, mom, "matcha",
                          B.make_topology("matchings", partner=np.array(partner), seed=5, alpha=0.25, act_prob=0.5))
        orc = O.Oracle(K, P, M, lr, mom, "matcha", partner=partner, alpha=0.25, prob=0.5, seed=5)
    ctx.set_params(torch.from_numpy(x0).cuda())
    orc.set_params(x0)
    for t in range(3):
        G = rng.integers(-8, 9, (K, M, P)).astype(np.float32)
        n = [int(v) for v in rng.choice([1, 2, 4], K)]
        ctx.step_fused(torch.from_numpy(G).cuda(), n)
        orc.step(G, n)
        X = ctx.get_params().numpy()
        assert np.array_equal(X.astype(np.float64), orc.X), (variant, t)
        assert np.array_equal(ctx.get_momentum().numpy().astype(np.float64), orc.V)
    ctx.close()


# ----------------------------------------------------------------------------------------------
# Degenerate cases and the other entry points
# ----------------------------------------------------------------------------------------------
def test_zero_finished_learner_and_single_learner(B):
    import torch
    # n_i = 0: no gradient contribution; momentum decays, mixing still happens
    w = WL.scaled(WL.WORKLOADS["cfg3_dpsgd_ring_resnet50"], 1024 + 4, steps=3)
    w = replace(w, K=5)
    ctx = B.context_for(w)
    orc = H.oracle_for(w, w.P)
    x0 = WL.init_params(w)
    ctx.set_params(torch.from_numpy(x0).cuda()); orc.set_params(x0)
    for t in range(3):
        payload, values = WL.gradients_np(w, t)
        n = [0, w.M, 1, 0, 3] if t != 1 else [0] * 5
        ctx.step_fused(H.to_device(payload), n)
        orc.step(values, n)
    H.assert_close(ctx.get_params().numpy(), orc.X, H.TOL_SAME_INPUT)
    ctx.close()
    # K = 1, M = 1
    w1 = replace(WL.scaled(WL.WORKLOADS["cfg2_allreduce_resnet18"], 77, steps=2), K=1, M=1)
    ctx = B.context_for(w1); orc = H.oracle_for(w1, 77)
    x0 = WL.init_params(w1)
    ctx.set_params(torch.from_numpy(x0).cuda()); orc.set_params(x0)
    for t in range(2):
        payload, values = WL.gradients_np(w1, t)
        ctx.step_fused(H.to_device(payload), [1]); orc.step(values, [1])
    H.assert_close(ctx.get_params().numpy(), orc.X, H.TOL_SAME_INPUT)
    ctx.close()


def test_masked_accumulate_alone(B):
    """nb_accumulate's output against the oracle's prefix sums; abandoned rows are never read
    (they hold NaN here)."""
    import torch
    w = WL.scaled(WL.WORKLOADS["cfg3_dpsgd_ring_resnet50"], 2 * 1024 + 24, steps=1)
    ctx = B.context_for(w)
    payload, values = WL.gradients_np(w, 0)
    n = H.lib_counts(B, w, 0)
    g = H.to_device(payload)
    for i in range(w.K):
        g[i, int(n[i]):] = float("nan")
    ctx.accumulate(g, n)
    acc = ctx.get_accumulator().numpy()
    assert np.isfinite(acc).all()
    H.assert_close(acc, O.accumulate(values, n.tolist()), 1e-6)
    ctx.close()


def test_per_learner_initialisation_and_large_k(B):
    import torch
    K, P, M = 40, 1024 + 8, 2
    rng = np.random.default_rng(3)
    X0 = rng.standard_normal((K, P)).astype(np.float32)
    ctx = B.NbContext(K, P, M, 0.1, 0.9, "dpsgd", B.make_topology("ring"))
    orc = O.Oracle(K, P, M, 0.1, 0.9, "dpsgd", W=O.ring_W(K))
    ctx.set_params(torch.from_numpy(X0).cuda(), per_learner=True); orc.set_params(X0)
    for t in range(3):
        G = rng.standard_normal((K, M, P)).astype(np.float32)
        n = rng.integers(0, M + 1, K).tolist()
        ctx.step_fused(torch.from_numpy(G).cuda(), n); orc.step(G, n)
    H.assert_close(ctx.get_params().numpy(), orc.X, H.TOL_SAME_INPUT)
    ctx.close()


def test_centralized_variant(B):
    import torch
    K, P, M = 8, 3 * 1024 + 5, 4
    rng = np.random.default_rng(4)
    x0 = (rng.standard_normal(P) * 0.01).astype(np.float32)
    for fused in (True, False):
        ctx = B.NbContext(K, P, M, 0.1, 0.9, "centralized")
        ctx.set_params(torch.from_numpy(x0).cuda())
        x, v = x0.astype(np.float64), np.zeros(P)
        for t in range(6):
            G = (np.random.default_rng(100 + t).standard_normal((K, M, P)) * 0.01).astype(np.float32)
            n = np.random.default_rng(200 + t).integers(1, M + 1, K).tolist()
            if fused:
                ctx.step_fused(torch.from_numpy(G).cuda(), n)
            else:
                ctx.accumulate(torch.from_numpy(G).cuda(), n); ctx.step()
            x, v = O.step_centralized(x, v, G, n, 0.1, 0.9)
        H.assert_close(ctx.get_params().numpy(), x, H.TOL_SAME_INPUT)
        H.assert_close(ctx.get_momentum().numpy(), v, H.TOL_SAME_INPUT)
        H.assert_close(ctx.get_mean_params().numpy(), x, H.TOL_SAME_INPUT)
        ctx.close()


def test_host_buffer_entry_point(B):
    import torch
    w = WL.scaled(WL.WORKLOADS["cfg3_dpsgd_ring_resnet50"], 2 * 1024 + 20, steps=3)
    a, b = B.context_for(w), B.context_for(w)
    x0 = torch.from_numpy(WL.init_params(w)).cuda()
    a.set_params(x0); b.set_params(x0)
    mean = torch.empty(w.P, dtype=torch.float32).pin_memory()
    for t in range(w.steps):
        n = H.lib_counts(B, w, t)
        payload = WL.gradients_np(w, t)[0]
        host = torch.from_numpy(payload).view(torch.bfloat16).pin_memory()
        a.step_fused_host(host, n, mean_out=mean)
        b.step_fused(H.to_device(payload), n)
        assert torch.equal(mean, b.get_mean_params())
    assert torch.equal(a.get_params(), b.get_params())
    a.close(); b.close()


@pytest.mark.parametrize("variant,order,K,P,dtype", [
    ("dpsgd", 0, 16, 3 * 512 + 20, "bf16"), ("dpsgd", 1, 16, 2 * 512 + 7, "bf16"), ("allreduce", 0, 8, 5 * 512, "f32"),
    ("allreduce", 1, 33, 512 + 100, "f32"), ("centralized", 0, 8, 4 * 512 + 9, "bf16"), ("dpsgd", 0, 64, 2 * 512 + 33, "bf16"),
    ("dpsgd", 0, 5, 300, "f32"),
])
def test_streaming_hold_mode_reads_the_delivered_vectors_in_place(B, variant, order, K, P, dtype):
    """NB_STREAMING_HOLD: deliveries are only recorded and nb_step runs the fused step on the vectors
    where they lie (separate allocations, one per mini-batch gradient).  Same terminal-signal
    behaviour as the accumulate mode (Alg. 1 inner loop), the same bits as that mode, oracle parity."""
    import torch
    M = 6
    rng = np.random.default_rng(K * 1000 + P)
    topo = B.make_topology("ring") if variant == "dpsgd" else None
    hold, acc = B.NbContext(K, P, M, 0.05, 0.9, variant, topo), B.NbContext(K, P, M, 0.05, 0.9, variant, topo)
    hold.set_option(B.NB_OPT_STREAMING, B.NB_STREAMING_HOLD)
    x0 = (rng.standard_normal(P) * 0.01).astype(np.float32)
    for c in (hold, acc):
        if variant != "centralized":
            c.set_option(B.NB_OPT_ORDER, order)
        c.set_params(torch.from_numpy(x0).cuda())
    if variant == "centralized":
        orc = None
        x_ps, v_ps = x0.astype(np.float64), np.zeros(P)
    else:
        W = O.ring_W(K) if variant == "dpsgd" else None
        orc = O.Oracle(K, P, M, 0.05, 0.9, "dpsgd" if variant == "dpsgd" else "allreduce", W=W,
                       order="mix_then_update" if order == 0 else "update_then_mix")
        orc.set_params(x0)
    tdt = torch.bfloat16 if dtype == "bf16" else torch.float32
    for t in range(3):
        n = rng.integers(0, M + 1, K)
        n[int(rng.integers(0, K))] = M                               # someone finishes: the terminal signal is raised
        # one separate device allocation per mini-batch gradient (what a learner would hand over)
        vecs = [[(torch.from_numpy(rng.standard_normal(P).astype(np.float32)) * 0.01).to(tdt).cuda() for _ in range(M)]
                for _ in range(K)]
        for c in (hold, acc):
            c.begin_iteration()
        done_first = None
        for m in range(M):                                           # round-robin arrival, as in a real iteration
            for i in range(K):
                if m < n[i]:
                    ra, rb = hold.accumulate_minibatch(i, vecs[i][m]), acc.accumulate_minibatch(i, vecs[i][m])
                    assert ra == rb
        assert hold.get_finished()[0].tolist() == acc.get_finished()[0].tolist()
        got_n = hold.get_finished()[0]
        hold.step(); acc.step()
        torch.cuda.synchronize()                                     # the vectors may be released only now
        G = torch.stack([torch.stack(v) for v in vecs]).float().cpu().numpy()
        if orc is not None:
            orc.step(G, got_n.tolist())
        else:
            x_ps, v_ps = O.step_centralized(x_ps, v_ps, G, got_n.tolist(), 0.05, 0.9)
    assert torch.equal(hold.get_params(), acc.get_params()) and torch.equal(hold.get_momentum(), acc.get_momentum())
    if orc is not None:
        H.assert_close(hold.get_params().numpy(), orc.X, H.TOL_SAME_INPUT)
        H.assert_close(hold.get_momentum().numpy(), orc.V, H.TOL_SAME_INPUT)
    else:
        H.assert_close(hold.get_params().numpy(), x_ps, H.TOL_SAME_INPUT)
    if P >= 1024:
        assert hold.get_kernel_plan()["row_copies"] == 2 or variant == "centralized"
    hold.check_guards()
    # misuse: a vector that is not 16-byte aligned, a second dtype inside one iteration, a mode switch inside one
    hold.begin_iteration()
    flat = torch.zeros(P + 8, dtype=tdt, device="cuda")
    with pytest.raises(B.NbError) as e:
        hold.accumulate_minibatch(0, flat[1:P + 1])
    assert e.value.code == B.NB_ERR_ARG
    assert hold.accumulate_minibatch(0, flat[:P])
    other = torch.zeros(P, dtype=torch.float32 if dtype == "bf16" else torch.bfloat16, device="cuda")
    with pytest.raises(B.NbError) as e:
        hold.accumulate_minibatch(0, other)
    assert e.value.code == B.NB_ERR_ARG
    with pytest.raises(B.NbError) as e:
        hold.set_option(B.NB_OPT_STREAMING, B.NB_STREAMING_ACCUMULATE)
    assert e.value.code == B.NB_ERR_STATE
    hold.step()
    hold.close(); acc.close()


def test_error_reporting(B):
    import torch
    ctx = B.NbContext(4, 100, 4, 0.1, 0.9, "allreduce")
    with pytest.raises(B.NbError) as e:
        ctx.step()
    assert e.value.code == B.NB_ERR_STATE
    g = torch.zeros((4, 4, 100), device="cuda")
    with pytest.raises(B.NbError) as e:
        ctx.step_fused(g, [1, 2, 5, 1])
    assert e.value.code == B.NB_ERR_ARG
    with pytest.raises(B.NbError):
        ctx.step_fused(g, [1, 2, -1, 1])
    with pytest.raises(B.NbError):
        ctx.step_fused(g, [1, 1, 1, 1], ld_m=50)
    # the host-memory entry point validates the caller's strides before it enqueues any copy
    gh = torch.zeros((4, 4, 100))
    for bad in (dict(ld_m=50), dict(ld_k=150), dict(ld_m=-100), dict(ld_m=100, ld_k=-400)):
        with pytest.raises(B.NbError) as e:
            ctx.step_fused_host(gh, [1, 1, 1, 1], **bad)
        assert e.value.code == B.NB_ERR_ARG
    import ctypes
    ones = (ctypes.c_int32 * 4)(1, 1, 1, 1)                  # a pointer that is not element-aligned
    assert B.lib.nb_step_fused(ctx._h, g.data_ptr() + 2, B.NB_F32, 0, 0, ones, None) == B.NB_ERR_ARG
    assert B.lib.nb_accumulate(ctx._h, g.data_ptr() + 2, B.NB_F32, 0, 0, ones, None) == B.NB_ERR_ARG
    with pytest.raises(ValueError):
        ctx.step_fused(g.transpose(1, 2), [1, 1, 1, 1])      # rows must be contiguous: the binding refuses
    assert ctx.get_step() == 0                               # none of the rejected calls ran anything
    wide = torch.zeros((4, 4, 128), device="cuda")
    ctx.accumulate(wide[:, :, :100], [1, 1, 1, 1])           # a view with contiguous rows passes its own strides
    ctx.step()
    with pytest.raises(B.NbError):
        ctx.step()                                   # accumulator already consumed
    st = ctx.get_stats()
    assert st["sum_finished"] == 4 and st["kernel_launches"] == 2
    assert st["algorithmic_bytes"] == 100 * (4 * 4 + 16 * 4)
    ctx.close()


def test_streaming_accumulate_follows_alg1_and_equals_batch_accumulate(B):
    """Mini-batch gradients handed over one at a time (Alg. 1 inner loop): the first learner to deliver
    all M raises the terminal signal, later deliveries are abandoned; sums equal nb_accumulate's bits."""
    import torch
    w = WL.scaled(WL.WORKLOADS["cfg3_dpsgd_ring_resnet50"], 2 * 512 + 20, steps=3)
    a, b = B.context_for(w), B.context_for(w)
    orc = H.oracle_for(w, w.P)
    x0 = WL.init_params(w)
    for c in (a, b):
        c.set_params(torch.from_numpy(x0).cuda())
    orc.set_params(x0)
    with pytest.raises(B.NbError):
        a.accumulate_minibatch(0, torch.zeros(w.P, device="cuda"))          # needs nb_begin_iteration
    for t in range(w.steps):
        payload, values = WL.gradients_np(w, t)
        g = H.to_device(payload)
        n = H.lib_counts(B, w, t)                                            # who finishes how many
        if t == 2:
            n = n.copy(); n[3] = 0                                           # a learner that delivers nothing
        a.begin_iteration()
        # deliver round-robin, mini-batch m of every learner that gets that far; the fastest (n_i = M) last
        for m in range(w.M):
            for i in np.argsort(-n, kind="stable")[::-1]:
                if m < n[i]:
                    assert a.accumulate_minibatch(int(i), g[i, m]) is True
        got, terminal = a.get_finished()
        assert got.tolist() == n.tolist() and terminal == bool((n == w.M).any())
        if terminal:
            assert a.accumulate_minibatch(0, g[0, 0]) is False               # abandoned after the signal
            assert a.get_finished()[0].tolist() == n.tolist()
        b.accumulate(g, n)
        assert torch.equal(a.get_accumulator()[n > 0], b.get_accumulator()[n > 0])
        a.step(); b.step()
        orc.step(values, n.tolist())
        assert torch.equal(a.get_params(), b.get_params())
    H.assert_close(a.get_params().numpy(), orc.X, H.TOL_SAME_INPUT)
    a.close(); b.close()


def test_matcha_with_optimised_per_matching_probabilities(B):
    """MATCHA's designed topology: per-matching activation probabilities under a budget and the
    optimal alpha from nb_matcha_optimize; activation words bit-exact on device, host and oracle."""
    import torch
    K, P, M = 16, 3 * 512 + 40, 4
    seed = 221100893
    base, _ = B.make_topology("random_regular", degree=3, seed=seed)
    probs, alpha, lam2, rho = B.matcha_optimize(base, K, 0.5)
    assert 0 < rho < 1 and lam2 > 0
    partner, _ = B.topology_matchings(base, K)
    topo = B.make_topology("random_regular", degree=3, seed=seed, alpha=alpha, act_probs=probs)
    ctx = B.NbContext(K, P, M, 0.05, 0.9, "matcha", topo)
    orc = O.Oracle(K, P, M, 0.05, 0.9, "matcha", partner=partner.tolist(), alpha=alpha, prob=probs.tolist(), seed=seed)
    rng = np.random.default_rng(1)
    x0 = (rng.standard_normal(P) * 0.01).astype(np.float32)
    ctx.set_params(torch.from_numpy(x0).cuda()); orc.set_params(x0)
    seen = set()
    for t in range(8):
        G = torch.from_numpy((rng.standard_normal((K, M, P)) * 0.01).astype(np.float32)).to(torch.bfloat16).cuda()
        n = rng.integers(1, M + 1, K)
        ctx.step_fused(G, n)
        orc.step(G.float().cpu().numpy(), n.tolist())
        bits, Wdev = ctx.get_device_mixing()
        assert bits == O.matcha_activation_probs(seed, t, probs.tolist()) == ctx.get_matcha_activation(t)
        assert np.array_equal(Wdev, ctx.get_W(t))
        assert np.allclose(Wdev.sum(0), 1.0, atol=1e-6) and np.allclose(Wdev.sum(1), 1.0, atol=1e-6)
        seen.add(bits)
    assert len(seen) > 1
    H.assert_close(ctx.get_params().numpy(), orc.X, H.TOL_SAME_INPUT)
    ctx.close()


def test_work_is_enqueued_on_the_callers_stream(B):
    """Every entry point takes the stream to enqueue on: a run on a side stream (inputs produced on
    that stream, no other synchronisation) equals the run on the default stream bit for bit."""
    import torch
    w = WL.scaled(WL.WORKLOADS["cfg4_matcha_vgg16"], 6 * 512 + 8, steps=4)
    x0 = torch.from_numpy(WL.init_params(w)).cuda()
    ref = B.context_for(w)
    ref.set_params(x0)
    side = torch.cuda.Stream()
    other = B.context_for(w)
    payloads = [WL.gradients_np(w, t)[0] for t in range(w.steps)]
    counts = [H.lib_counts(B, w, t) for t in range(w.steps)]
    for t in range(w.steps):
        ref.step_fused(H.to_device(payloads[t]), counts[t])
    torch.cuda.synchronize()
    with torch.cuda.stream(side):
        other.set_params(x0)
        for t in range(w.steps):
            g = H.to_device(payloads[t]) * 1.0            # produced on the side stream
            other.step_fused(g, counts[t])
        X = other.get_params(device="cuda")
        V = other.get_momentum(device="cuda")
    side.synchronize()
    assert torch.equal(X, ref.get_params(device="cuda")) and torch.equal(V, ref.get_momentum(device="cuda"))
    ref.close(); other.close()


@pytest.mark.parametrize("fused", [True, False])
def test_step_can_be_captured_in_a_cuda_graph(B, fused):
    """The step entry points only enqueue kernels on the caller's stream (no allocation, copy or
    synchronisation once a context has run its first step), so an iteration can be captured in a CUDA
    graph and replayed: three replays equal three plain calls bit for bit."""
    import torch
    w = WL.scaled(WL.WORKLOADS["cfg3_dpsgd_ring_resnet50"], 9 * 512 + 40, steps=4)
    x0 = torch.from_numpy(WL.init_params(w)).cuda()
    G = H.to_device(WL.gradients_np(w, 0)[0])
    n = H.lib_counts(B, w, 0)
    plain, graphed = B.context_for(w), B.context_for(w)

    def step(ctx):
        if fused:
            ctx.step_fused(G, n)
        else:
            ctx.accumulate(G, n)
            ctx.step()

    for ctx in (plain, graphed):
        ctx.set_params(x0)
        step(ctx)                                  # first step outside the capture
    torch.cuda.synchronize()
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph):
        step(graphed)                              # recorded, not run
    for _ in range(3):
        graph.replay()
        step(plain)
    torch.cuda.synchronize()
    assert torch.equal(graphed.get_params(device="cuda"), plain.get_params(device="cuda"))
    assert torch.equal(graphed.get_momentum(device="cuda"), plain.get_momentum(device="cuda"))
    graphed.check_guards()
    del graph
    plain.close(); graphed.close()


@pytest.mark.parametrize("name", ["cfg2_allreduce_resnet18", "cfg3_dpsgd_ring_resnet50", "cfg4_matcha_vgg16",
                                  "cfg5_scale_ring"])
def test_full_step_counts_of_the_configurations(B, name):
    """The configurations' own step counts (50 / 50 / 20 / 20): tolerance checked at step 10 and at the last step."""
    w = WL.WORKLOADS[name]
    ws = WL.scaled(w, 2 * 512 + 72, steps=w.steps)
    errs = _run(B, ws, ws.steps, fused=True, check_steps=(10, ws.steps), with_unrounded=(ws.grad_dtype == "bf16"))
    assert set(errs) == {10, ws.steps}
    assert all(e[0] < H.TOL_SAME_INPUT for e in errs.values())


def test_dense_mixing_matrix_at_the_table_limit(B):
    """D-PSGD with the FULL topology and K = 32 fills the sparse table exactly (1024 non-zeros); it
    must agree with the oracle's dense W (and, up to rounding order, with the all-reduce variant)."""
    import torch
    K, P, M = 32, 2 * 512 + 16, 2
    rng = np.random.default_rng(32)
    X0 = rng.standard_normal((K, P)).astype(np.float32)
    ctx = B.NbContext(K, P, M, 0.1, 0.9, "dpsgd", B.make_topology("full"))
    orc = O.Oracle(K, P, M, 0.1, 0.9, "dpsgd", W=O.full_W(K))
    ctx.set_params(torch.from_numpy(X0).cuda(), per_learner=True); orc.set_params(X0)
    for t in range(3):
        G = rng.standard_normal((K, M, P)).astype(np.float32)
        n = rng.integers(0, M + 1, K).tolist()
        ctx.step_fused(torch.from_numpy(G).cuda(), n); orc.step(G, n)
    H.assert_close(ctx.get_params().numpy(), orc.X, H.TOL_SAME_INPUT)
    ctx.check_guards()
    ctx.close()


@pytest.mark.parametrize("name", ["cfg3_dpsgd_ring_resnet50", "cfg4_matcha_vgg16", "cfg2_allreduce_resnet18"])
def test_host_buffer_entry_point_in_several_chunks(B, name):
    """Enough columns for nb_step_fused_host to split the work into overlapped column chunks: the
    result must equal nb_step_fused on the same values, bit for bit, mean model included."""
    import torch
    w = replace(WL.scaled(WL.WORKLOADS[name], 3 * 65536 + 520, steps=2), K=4, M=3)
    if w.variant == "matcha":
        w = replace(w, degree=3)
    a, b = B.context_for(w), B.context_for(w)
    gen = torch.Generator(device="cuda"); gen.manual_seed(5)
    x0 = torch.randn(w.P, generator=gen, device="cuda") * 0.01
    a.set_params(x0); b.set_params(x0)
    mean = torch.empty(w.P, dtype=torch.float32).pin_memory()
    for t in range(w.steps):
        g = WL.gradients_torch(w, t, "cuda")
        host = torch.empty(g.shape, dtype=g.dtype).pin_memory()
        host.copy_(g)
        n = np.array([3, 1, 0, 2]) if t == 0 else np.array([2, 3, 3, 1])
        a.step_fused_host(host, n, mean_out=mean)
        b.step_fused(g, n)
        assert torch.equal(mean, b.get_mean_params())
    assert a.get_step() == b.get_step() == w.steps
    assert torch.equal(a.get_params(), b.get_params()) and torch.equal(a.get_momentum(), b.get_momentum())
    a.check_guards()
    a.close(); b.close()


def test_learning_rate_can_change_between_steps(B):
    """nb_set_lr (e.g. a decay schedule as in Sec. 6.1): each step uses the rate set before it."""
    import torch
    w = WL.scaled(WL.WORKLOADS["cfg3_dpsgd_ring_resnet50"], 2 * 512 + 8, steps=4)
    ctx = B.context_for(w)
    orc = H.oracle_for(w, w.P)
    x0 = WL.init_params(w)
    ctx.set_params(torch.from_numpy(x0).cuda()); orc.set_params(x0)
    for t, lr in enumerate([0.8, 0.8, 0.08, 0.008]):
        ctx.set_lr(lr)
        orc.lr = lr
        n = H.lib_counts(B, w, t)
        payload, values = WL.gradients_np(w, t)
        ctx.step_fused(H.to_device(payload), n)
        orc.step(values, n.tolist())
    H.assert_close(ctx.get_params().numpy(), orc.X, H.TOL_SAME_INPUT)
    ctx.close()


def test_reported_mixing_matrices(B):
    for name in ("cfg2_allreduce_resnet18", "cfg3_dpsgd_ring_resnet50"):
        w = WL.scaled(WL.WORKLOADS[name], 64, steps=1)
        ctx = B.context_for(w)
        want = O.full_W(w.K) if w.variant == "allreduce" else O.ring_W(w.K)
        assert np.abs(ctx.get_W(0).astype(np.float64) - want).max() < 1e-7
        with pytest.raises(B.NbError):
            ctx.get_matcha_activation(0)           # not a MATCHA context
        ctx.close()
