"""Host logic of the library against the oracle, bit for bit: straggler simulator (finished counts,
masks), random regular graph + matchings, MATCHA activation words, mixing matrices.  CPU only."""
import numpy as np
import pytest

from oracle import nb_oracle as O
from paper_2211_00889_b200.build import build_library

build_library()
from paper_2211_00889_b200 import binding as B  # noqa: E402
from paper_2211_00889_b200.workloads import WORKLOADS  # noqa: E402


@pytest.mark.parametrize("name", list(WORKLOADS))
def test_finished_counts_and_masks_bit_exact(name):
    w = WORKLOADS[name]
    for t in range(300):
        n, mask, tau = B.straggler_sample(w.straggler_model, w.seed, t, w.K, w.M, w.straggler_params)
        want = O.straggler_counts(w.straggler_model, w.seed, t, w.K, w.M, w.straggler_params)
        assert n.tolist() == want, (name, t)
        assert np.array_equal(mask, O.finished_mask(want, w.M))
        assert n.min() >= 1 and n.max() <= w.M
        if w.straggler_model != "uniform_count":
            assert n[int(np.argmin(tau))] == w.M


def test_delays_bit_exact():
    for t in range(200):
        _, _, tau = B.straggler_sample("shifted_exp", 42, t, 16, 8, (1.0,))
        assert tau.tolist() == O.delays_shifted_exp(42, t, 16, [1.0] * 16)


def test_slow_set_bit_exact_through_delays():
    K = 32
    for t in range(200):
        _, _, tau = B.straggler_sample("shifted_exp_slowset", 7, t, K, 8, (0.25, 2.0, 0.1))
        slow = set(O.slow_set(7, t, K, 8))
        want = O.delays_shifted_exp(7, t, K, [2.0 if i in slow else 0.1 for i in range(K)])
        assert tau.tolist() == want


def test_straggler_argument_errors():
    import ctypes as C
    cfg = B.nb_straggler()
    n = np.zeros(4, dtype=np.int32)
    p = n.ctypes.data_as(C.POINTER(C.c_int32))
    cfg.model = 7
    assert B.lib.nb_straggler_sample(C.byref(cfg), 4, 4, 0, p, None, None) == B.NB_ERR_ARG
    cfg.model = B.NB_STRAG_SHIFTED_EXP
    cfg.params[0] = -1.0
    assert B.lib.nb_straggler_sample(C.byref(cfg), 4, 4, 0, p, None, None) == B.NB_ERR_ARG
    cfg.params[0] = 1.0
    assert B.lib.nb_straggler_sample(C.byref(cfg), 0, 4, 0, p, None, None) == B.NB_ERR_ARG
    assert B.lib.nb_straggler_sample(C.byref(cfg), 4, 0, 0, p, None, None) == B.NB_ERR_ARG
    assert B.lib.nb_straggler_sample(C.byref(cfg), 4, 4, 0, p, None, None) == B.NB_OK


@pytest.mark.parametrize("seed,K,d", [(221100893, 16, 3), (1, 16, 3), (2, 8, 3), (3, 32, 3), (4, 10, 4), (5, 6, 5)])
def test_random_regular_graph_and_matchings_bit_exact(seed, K, d):
    topo, _ = B.make_topology("random_regular", degree=d, seed=seed, alpha=0.1, act_prob=0.5)
    partner, attempts = B.topology_matchings(topo, K)
    edges, want_attempts = O.random_regular_graph(seed, K, d)
    want = O.greedy_matchings(edges, K)
    assert attempts == want_attempts
    assert partner.tolist() == want


def test_matcha_activation_and_W_match_oracle():
    w = WORKLOADS["cfg4_matcha_vgg16"]
    topo, _ = B.make_topology("random_regular", degree=w.degree, seed=w.seed, alpha=w.alpha, act_prob=w.act_prob)
    partner, _ = B.topology_matchings(topo, w.K)
    for t in range(500):
        W, bits = B.mixing_matrix(topo, B.NB_MATCHA, w.K, t)
        want_bits = O.matcha_activation(w.seed, t, len(partner), w.act_prob)
        assert bits == want_bits
        Wd = O.matcha_W(partner.tolist(), want_bits, w.alpha, w.K)
        assert np.abs(W.astype(np.float64) - Wd).max() < 1e-7
        assert np.array_equal(W != 0, Wd != 0)


@pytest.mark.parametrize("prob", [0.0, 1.0, 0.25, 0.9])
def test_activation_probability_extremes(prob):
    partner = np.array([[1, 0, 3, 2], [2, 3, 0, 1], [3, 2, 1, 0]], dtype=np.int32)
    topo, _ = B.make_topology("matchings", partner=partner, seed=99, alpha=0.25, act_prob=prob)
    for t in range(200):
        _, bits = B.mixing_matrix(topo, B.NB_MATCHA, 4, t)
        assert bits == O.matcha_activation(99, t, 3, prob)
        if prob == 0.0:
            assert bits == 0
        if prob == 1.0:
            assert bits == 0b111


def test_fixed_mixing_matrices_match_oracle():
    for K in (1, 2, 3, 16, 32):
        topo, _ = B.make_topology("ring")
        W, _ = B.mixing_matrix(topo, B.NB_DPSGD, K, 0)
        assert np.abs(W.astype(np.float64) - O.ring_W(K)).max() < 1e-7
        W, _ = B.mixing_matrix(None, B.NB_ALLREDUCE, K, 0)
        assert np.abs(W.astype(np.float64) - O.full_W(K)).max() < 1e-7      # the library holds fp32(1/K)


def test_topology_validation():
    import ctypes as C
    W = np.zeros((4, 4), dtype=np.float32)
    Wp = W.ctypes.data_as(C.POINTER(C.c_float))
    # CSR whose rows do not sum to one
    topo, keep = B.make_topology("csr", csr=([0, 1, 2, 3, 4], [0, 1, 2, 3], [1.0, 1.0, 0.5, 1.0]))
    assert B.lib.nb_mixing_matrix(C.byref(topo), B.NB_DPSGD, 4, 0, Wp, None) == B.NB_ERR_ARG
    # a good CSR (unsorted columns are accepted and sorted)
    topo, keep = B.make_topology("csr", csr=([0, 2, 4, 5, 6], [1, 0, 0, 1, 2, 3], [0.25, 0.75, 0.25, 0.75, 1.0, 1.0]))
    assert B.lib.nb_mixing_matrix(C.byref(topo), B.NB_DPSGD, 4, 0, Wp, None) == B.NB_OK
    assert W.tolist() == [[0.75, 0.25, 0, 0], [0.25, 0.75, 0, 0], [0, 0, 1, 0], [0, 0, 0, 1]]
    # partner table that is not an involution
    topo, keep = B.make_topology("matchings", partner=np.array([[1, 2, 0, -1]]), alpha=0.1, act_prob=0.5)
    assert B.lib.nb_mixing_matrix(C.byref(topo), B.NB_MATCHA, 4, 0, Wp, None) == B.NB_ERR_ARG
    # edge repeated in two matchings
    topo, keep = B.make_topology("matchings", partner=np.array([[1, 0, -1, -1], [1, 0, 3, 2]]), alpha=0.1, act_prob=0.5)
    assert B.lib.nb_mixing_matrix(C.byref(topo), B.NB_MATCHA, 4, 0, Wp, None) == B.NB_ERR_ARG
    # alpha outside [0, 1]
    topo, keep = B.make_topology("matchings", partner=np.array([[1, 0, 3, 2], [2, 3, 0, 1]]), alpha=1.5, act_prob=0.5)
    assert B.lib.nb_mixing_matrix(C.byref(topo), B.NB_MATCHA, 4, 0, Wp, None) == B.NB_ERR_ARG
    # impossible regular graph (odd K*d)
    topo, keep = B.make_topology("random_regular", degree=3, seed=1, alpha=0.1, act_prob=0.5)
    assert B.lib.nb_mixing_matrix(C.byref(topo), B.NB_MATCHA, 5, 0, Wp, None) == B.NB_ERR_ARG
    # wrong topology for the variant
    topo, keep = B.make_topology("ring")
    assert B.lib.nb_mixing_matrix(C.byref(topo), B.NB_MATCHA, 4, 0, Wp, None) == B.NB_ERR_ARG
    assert B.lib.nb_mixing_matrix(C.byref(topo), B.NB_ALLREDUCE, 4, 0, Wp, None) == B.NB_ERR_ARG


def test_expected_finished_fraction_of_the_bench_workload():
    # documents the size of the timed workload: mean of sum n_i over many steps
    w = WORKLOADS["cfg3_dpsgd_ring_resnet50"]
    tot = sum(int(B.straggler_sample(w.straggler_model, w.seed, t, w.K, w.M, w.straggler_params)[0].sum())
              for t in range(3000))
    assert 70.0 < tot / 3000 < 77.0


@pytest.mark.parametrize("name", ["cfg2_allreduce_resnet18", "cfg3_dpsgd_ring_resnet50", "cfg5_scale_ring"])
def test_runtime_report_matches_oracle(name):
    w = WORKLOADS[name]
    got = B.runtime_report(w.straggler_model, w.seed, w.K, w.M, 400, w.straggler_params, step0=3)
    want = O.runtime_report(w.straggler_model, w.seed, w.K, w.M, 400, w.straggler_params, step0=3)
    assert got["steps"] == want["steps"] == 400
    for k in want:
        assert got[k] == pytest.approx(want[k], rel=1e-13), k
    with pytest.raises(B.NbError) as e:
        B.runtime_report("uniform_count", 1, 4, 4, 10)
    assert e.value.code == B.NB_ERR_UNSUPPORTED


def test_randomised_straggler_configurations_bit_exact():
    """Many random (model, K, M, means, seed, step) draws: counts, masks and times equal the oracle's."""
    rng = np.random.default_rng(2211)
    for _ in range(300):
        K = int(rng.integers(1, 65))
        M = int(rng.integers(1, 33))
        seed = int(rng.integers(0, 2 ** 63))
        t = int(rng.integers(0, 10 ** 9))
        kind = int(rng.integers(0, 3))
        if kind == 0:
            model, params = "uniform_count", ()
        elif kind == 1:
            model, params = "shifted_exp", (float(rng.choice([0.0, 0.1, 0.5, 1.0, 2.0, 7.5])),)
        else:
            model, params = "shifted_exp_slowset", (float(rng.choice([0.0, 0.25, 0.5, 1.0])),
                                                    float(rng.uniform(0, 4)), float(rng.uniform(0, 1)))
        n, mask, tau = B.straggler_sample(model, seed, t, K, M, params)
        want = O.straggler_counts(model, seed, t, K, M, params)
        assert n.tolist() == want, (model, K, M, seed, t, params)
        assert np.array_equal(mask, O.finished_mask(want, M))


def test_randomised_regular_graphs_bit_exact():
    rng = np.random.default_rng(889)
    done = 0
    while done < 16:
        K = int(rng.integers(4, 41))
        d = int(rng.integers(2, min(K - 1, 6) + 1))
        if (K * d) % 2:
            continue
        seed = int(rng.integers(0, 2 ** 62))
        topo, _ = B.make_topology("random_regular", degree=d, seed=seed, alpha=0.05, act_prob=0.5)
        partner, attempts = B.topology_matchings(topo, K)
        edges, want_attempts = O.random_regular_graph(seed, K, d)
        assert attempts == want_attempts and partner.tolist() == O.greedy_matchings(edges, K)
        for t in (0, 1, 12345):
            _, bits = B.mixing_matrix(topo, B.NB_MATCHA, K, t)
            assert bits == O.matcha_activation(seed, t, len(partner), 0.5)
        done += 1


@pytest.mark.parametrize("seed,K,d,budget", [(221100893, 16, 3, 0.5), (7, 12, 3, 0.3), (11, 20, 4, 0.6), (3, 8, 3, 1.0)])
def test_matcha_design_problem_matches_oracle_optimum(seed, K, d, budget):
    """Activation probabilities and alpha from the library solve the same two problems as the
    oracle's routines: compared through the optimal VALUES (the maximiser need not be unique)."""
    topo, _ = B.make_topology("random_regular", degree=d, seed=seed)
    probs, alpha, lam2, rho = B.matcha_optimize(topo, K, budget, iters=1500)
    partner, _ = B.topology_matchings(topo, K)
    m = len(partner)
    Ls = O.matching_laplacians(partner.tolist(), K)
    assert probs.shape == (m,) and np.all(probs >= 0) and np.all(probs <= 1)
    assert probs.sum() <= budget * m + 1e-4                                   # the budget holds
    p_or, lam_or = O.matcha_optimal_probs(Ls, budget, iters=1500)
    assert O.matcha_lambda2(Ls, probs) == pytest.approx(lam2, rel=1e-4, abs=1e-6)
    assert lam2 == pytest.approx(lam_or, rel=2e-3, abs=1e-5)                   # same optimum
    assert lam2 >= O.matcha_lambda2(Ls, [budget] * m) - 1e-6                   # never worse than uniform spending
    a_or, rho_or = O.matcha_optimal_alpha(Ls, probs)                           # oracle's alpha for the library's p
    assert O.matcha_rho(Ls, probs, alpha) == pytest.approx(rho, rel=1e-4)
    assert rho == pytest.approx(rho_or, rel=1e-4) and abs(alpha - a_or) < 2e-3
    assert 0.0 < rho < 1.0
    if budget == 1.0:
        assert np.allclose(probs, 1.0)


def test_per_matching_probabilities_drive_the_activation_words():
    K = 16
    topo, _ = B.make_topology("random_regular", degree=3, seed=221100893)
    probs, alpha, _, _ = B.matcha_optimize(topo, K, 0.5)
    partner, _ = B.topology_matchings(topo, K)
    topo2, keep = B.make_topology("random_regular", degree=3, seed=221100893, alpha=alpha, act_probs=probs)
    freq = np.zeros(len(partner))
    T = 3000
    for t in range(T):
        W, bits = B.mixing_matrix(topo2, B.NB_MATCHA, K, t)
        assert bits == O.matcha_activation_probs(221100893, t, probs.tolist())   # bit-exact
        Wd = O.matcha_W(partner.tolist(), bits, alpha, K)
        assert np.abs(W.astype(np.float64) - Wd).max() < 1e-6
        for j in range(len(partner)):
            freq[j] += (bits >> j) & 1
    assert np.all(np.abs(freq / T - probs) < 0.04)
    # a probability outside [0, 1] is rejected
    import ctypes as C
    bad, keep2 = B.make_topology("random_regular", degree=3, seed=1, alpha=0.1, act_probs=np.array([0.5, 1.5, 0.5, 0.5, 0.5]))
    Wbuf = np.zeros((K, K), dtype=np.float32)
    assert B.lib.nb_mixing_matrix(C.byref(bad), B.NB_MATCHA, K, 0, Wbuf.ctypes.data_as(C.POINTER(C.c_float)), None) == B.NB_ERR_ARG


def test_table_limits_are_reported():
    import ctypes as C
    W = np.zeros((64, 64), dtype=np.float32)
    Wp = W.ctypes.data_as(C.POINTER(C.c_float))
    topo, _ = B.make_topology("full")
    assert B.lib.nb_mixing_matrix(C.byref(topo), B.NB_DPSGD, 32, 0, Wp, None) == B.NB_OK          # 1024 non-zeros: fits
    assert B.lib.nb_mixing_matrix(C.byref(topo), B.NB_DPSGD, 33, 0, Wp, None) == B.NB_ERR_UNSUPPORTED
    assert B.lib.nb_mixing_matrix(None, B.NB_ALLREDUCE, 64, 0, Wp, None) == B.NB_OK               # the mean needs no table
    assert B.lib.nb_mixing_matrix(None, B.NB_ALLREDUCE, 65, 0, Wp, None) == B.NB_ERR_UNSUPPORTED
    # more matchings than activation bits
    K = 4
    partner = np.full((33, K), -1, dtype=np.int32)
    topo, keep = B.make_topology("matchings", partner=partner, alpha=0.1, act_prob=0.5)
    assert B.lib.nb_mixing_matrix(C.byref(topo), B.NB_MATCHA, K, 0, Wp, None) == B.NB_ERR_UNSUPPORTED
