"""Pins for the CPU oracle: every function in oracle/nb_oracle.py is checked against something
other than itself - values the mathematics or the paper fixes, closed forms, special cases that
reduce to textbook updates, exact rational brute force on tiny inputs, and invariants.
CPU only."""
import math
import os
from fractions import Fraction

import numpy as np
import pytest

from oracle import nb_oracle as O

GOLD = os.path.join(os.path.dirname(__file__), "golden")


def _rand(shape, seed, scale=1.0):
    return np.random.default_rng(seed).standard_normal(shape) * scale


# ------------------------------------------------------------------------------------------
# counter generator
# ------------------------------------------------------------------------------------------
def test_mix64_matches_published_splitmix64_vector():
    want = [int(l.strip(), 16) for l in open(os.path.join(GOLD, "splitmix64_seed0.txt"))
            if l.strip() and not l.startswith("#")]
    # SplitMix64 seeded with 0: output k is the finaliser applied to k * increment
    got = [O.mix64(k * O.GOLDEN) for k in (1, 2, 3)]
    assert got == want
    # rng's innermost layer with seed 0 is exactly output 1
    assert O.mix64(0 + O.GOLDEN) == want[0]


def test_rng_is_a_nested_hash_of_its_four_counters():
    # changing any single argument changes the output; same arguments give the same output
    base = O.rng(7, 2, 3, 4)
    assert base == O.rng(7, 2, 3, 4)
    assert len({base, O.rng(8, 2, 3, 4), O.rng(7, 3, 3, 4), O.rng(7, 2, 4, 4), O.rng(7, 2, 3, 5)}) == 5
    assert 0 <= base < 2 ** 64
    # wrap-around of the 64-bit additions is handled
    assert 0 <= O.rng(2 ** 64 - 1, 2 ** 63, 2 ** 64 - 1, 2 ** 64 - 1) < 2 ** 64


def test_rng_uniformity_chi_square():
    n, bins = 200000, 64
    counts = np.zeros(bins)
    for b in range(n):
        counts[O.rng(11, O.STREAM_STRAGGLER, b // 1000, b % 1000) >> 58] += 1
    chi2 = ((counts - n / bins) ** 2 / (n / bins)).sum()
    assert chi2 < 120.0  # 63 dof: mean 63, sd 11.2


def test_uniform01_is_positive_at_most_one_and_centred():
    assert O.uniform01(0) == 0.5 * 2.0 ** -53 > 0.0
    assert O.uniform01(2 ** 64 - 1) == 1.0 and O.uniform01((2 ** 53 - 2) << 11) == 1.0 - 1.5 * 2.0 ** -53 < 1.0
    u = [O.uniform01(O.rng(3, 2, 0, i)) for i in range(50000)]
    assert abs(np.mean(u) - 0.5) < 4 * math.sqrt(1 / 12 / 50000)


# ------------------------------------------------------------------------------------------
# straggler simulator
# ------------------------------------------------------------------------------------------
def _theorem2_table():
    rows = {}
    for l in open(os.path.join(GOLD, "theorem2_runtime.txt")):
        if l.startswith("#") or not l.strip():
            continue
        P, lam, tnb, tdp = l.split()
        rows[(int(P), float(lam))] = (float(tnb), float(tdp))
    return rows


def test_theorem2_closed_form_is_the_harmonic_number():
    # textbook: E[max of P iid Exp(lambda)] = H_P / lambda; the paper's alternating sum must agree
    for (P, lam), (tnb, tdp) in _theorem2_table().items():
        H = sum(1.0 / k for k in range(1, P + 1))
        assert tdp == pytest.approx(H / lam, rel=1e-12)
        assert tnb == pytest.approx(1.0 / (lam * P), rel=1e-15)


@pytest.mark.parametrize("K,delta", [(10, 1.0), (16, 0.5), (4, 1.0)])
def test_exponential_delays_match_theorem2_expectations(K, delta):
    # the paper's own check: P=10 learners, N=10000 draws, sample mean of the maximum
    N = 10000
    lam = 1.0 / delta
    mins, maxs = [], []
    for t in range(N):
        tau = O.delays_shifted_exp(12345, t, K, [delta] * K)
        ex = [x - 1.0 for x in tau]  # the exponential part
        assert min(ex) > 0.0
        mins.append(min(ex))
        maxs.append(max(ex))
    tnb, tdp = _theorem2_table()[(K, lam)]
    # standard errors: sd(min) = delta/K ; var(max) = delta^2 * sum 1/k^2
    se_min = (delta / K) / math.sqrt(N)
    se_max = delta * math.sqrt(sum(1.0 / k ** 2 for k in range(1, K + 1)) / N)
    assert abs(np.mean(mins) - tnb) < 4 * se_min
    assert abs(np.mean(maxs) - tdp) < 4 * se_max


def test_counts_from_delays_invariants():
    M = 8
    for t in range(300):
        tau = O.delays_shifted_exp(99, t, 16, [1.0] * 16)
        n = O.counts_from_delays(tau, M)
        fastest = int(np.argmin(tau))
        assert n[fastest] == M                       # the first finisher did its whole batch
        assert all(1 <= c <= M for c in n)
        order = np.argsort(tau)
        assert all(n[order[a]] >= n[order[a + 1]] for a in range(15))  # slower => not more
        for tau_i, c in zip(tau, n):                 # constant speed: fraction tau_min / tau_i
            assert c == max(1, int(math.floor(M * min(tau) / tau_i + 1e-12))) or \
                abs(M * min(tau) / tau_i - round(M * min(tau) / tau_i)) < 1e-9


def test_counts_hand_worked_example():
    # tau = (1, 2, 1.6, 8.1), M = 8: deadline T = 8; j*tau <= 8 -> 8, 4, 5, 0 -> clamped to 1
    assert O.counts_from_delays([1.0, 2.0, 1.6, 8.1], 8) == [8, 4, 5, 1]
    # ties count as finished
    assert O.counts_from_delays([2.0, 4.0], 4) == [4, 2]


def test_zero_delay_means_everyone_finishes():
    for t in range(20):
        assert O.straggler_counts("shifted_exp", 5, t, 8, 8, (0.0,)) == [8] * 8


def test_uniform_counts_cover_range_evenly():
    M, K = 4, 4
    hist = np.zeros(M + 1)
    for t in range(5000):
        for c in O.counts_uniform(221100890, t, K, M):
            hist[c] += 1
    assert hist[0] == 0
    assert np.all(np.abs(hist[1:] / hist.sum() - 0.25) < 0.01)


def test_slow_set_is_a_uniform_subset_without_repeats():
    K, ns = 32, 8
    freq = np.zeros(K)
    for t in range(4000):
        s = O.slow_set(77, t, K, ns)
        assert len(s) == ns == len(set(s)) and all(0 <= v < K for v in s)
        freq[s] += 1
    assert np.all(np.abs(freq / 4000 - ns / K) < 0.035)
    # the slow learners really are slower on average
    tot_slow, tot_fast, c_slow, c_fast = 0, 0, 0, 0
    for t in range(500):
        slow = set(O.slow_set(77, t, K, ns))
        n = O.straggler_counts("shifted_exp_slowset", 77, t, K, 8, (0.25, 2.0, 0.1))
        for i, c in enumerate(n):
            if i in slow:
                tot_slow += c; c_slow += 1
            else:
                tot_fast += c; c_fast += 1
    assert c_slow == 500 * ns
    assert tot_slow / c_slow < tot_fast / c_fast - 1.0


def test_runtime_report_matches_theorems_1_and_2():
    # tau = 1 + Exp(mean delta): E[min] = 1 + delta/K, E[max] = 1 + delta*H_K (Theorem 2, shifted by 1)
    K, M, delta, steps = 10, 8, 1.0, 20000
    rep = O.runtime_report("shifted_exp", 4242, K, M, steps, (delta,))
    tnb, tdp = _theorem2_table()[(K, 1.0)]
    se_min = (delta / K) / math.sqrt(steps)
    se_max = delta * math.sqrt(sum(1.0 / k ** 2 for k in range(1, K + 1)) / steps)
    assert abs(rep["mean_min_tau"] - (1.0 + tnb)) < 4 * se_min
    assert abs(rep["mean_max_tau"] - (1.0 + tdp)) < 4 * se_max
    assert rep["mean_t_nonblocking"] == pytest.approx(M * rep["mean_min_tau"], rel=1e-12)     # Lemma 1
    assert rep["mean_t_blocking"] == pytest.approx(M * rep["mean_max_tau"], rel=1e-12)
    assert rep["ratio"] == pytest.approx(rep["mean_t_nonblocking"] / rep["mean_t_blocking"], rel=1e-12)  # Theorem 1
    assert rep["ratio"] < 1.0 < rep["mean_throughput_ratio"]                                   # Theorem 5: > 1
    # floor rule never exceeds Corollary 1's fractional data, and is within one mini-batch per learner of it
    assert rep["mean_fractional_data"] - 1.0 / M <= rep["mean_finished_fraction"] <= rep["mean_fractional_data"] + 1e-12
    # no delay spread: everything is 1
    rep0 = O.runtime_report("shifted_exp", 1, 4, 8, 50, (0.0,))
    assert rep0["ratio"] == 1.0 and rep0["mean_throughput_ratio"] == 1.0 and rep0["mean_finished_fraction"] == 1.0


def test_finished_mask_is_a_prefix():
    m = O.finished_mask([0, 1, 3, 4], 4)
    assert m.dtype == np.uint8
    assert m.tolist() == [[0, 0, 0, 0], [1, 0, 0, 0], [1, 1, 1, 0], [1, 1, 1, 1]]


# ------------------------------------------------------------------------------------------
# topologies, MATCHA
# ------------------------------------------------------------------------------------------
def _assert_doubly_stochastic(W, tol=1e-6):
    assert np.allclose(W.sum(0), 1.0, atol=tol) and np.allclose(W.sum(1), 1.0, atol=tol)
    assert np.allclose(W, W.T)


def test_ring_and_full_matrices():
    W = O.ring_W(16)
    _assert_doubly_stochastic(W)
    third = float(np.float32(1 / 3))
    for i in range(16):
        nz = {j: W[i, j] for j in range(16) if W[i, j] != 0}
        assert nz == {i: third, (i + 1) % 16: third, (i - 1) % 16: third}
    _assert_doubly_stochastic(O.full_W(8), 1e-12)
    assert np.all(O.full_W(8) == 0.125)
    assert O.ring_W(1)[0, 0] == pytest.approx(1.0, abs=1e-7)
    _assert_doubly_stochastic(O.ring_W(2))


@pytest.mark.parametrize("seed", [1, 2, 3, 221100893])
def test_random_regular_graph_properties(seed):
    K, d = 16, 3
    edges, attempts = O.random_regular_graph(seed, K, d)
    assert attempts >= 1
    assert len(edges) == K * d // 2 == len(set(edges))
    deg = np.zeros(K, int)
    for (u, v) in edges:
        assert 0 <= u < v < K
        deg[u] += 1; deg[v] += 1
    assert np.all(deg == d)
    # connected: Laplacian has exactly one zero eigenvalue
    L = np.zeros((K, K))
    for (u, v) in edges:
        L[u, u] += 1; L[v, v] += 1; L[u, v] -= 1; L[v, u] -= 1
    ev = np.sort(np.linalg.eigvalsh(L))
    assert abs(ev[0]) < 1e-9 and ev[1] > 1e-6


@pytest.mark.parametrize("seed", [1, 2, 3, 221100893])
def test_matchings_partition_the_edges(seed):
    K, d = 16, 3
    edges, _ = O.random_regular_graph(seed, K, d)
    partner = O.greedy_matchings(edges, K)
    assert d <= len(partner) <= 2 * d - 1
    seen = set()
    for row in partner:
        for u in range(K):
            v = row[u]
            if v >= 0:
                assert row[v] == u and v != u          # involution: vertex-disjoint links
                if u < v:
                    assert (u, v) not in seen           # edge-disjoint across matchings
                    seen.add((u, v))
    assert seen == set(edges)                           # union is the base graph


def test_matcha_W_hand_example():
    # K=4, matchings {0-1, 2-3} and {1-2}; alpha = 0.25 (exact in fp32)
    partner = [[1, 0, 3, 2], [-1, 2, 1, -1]]
    W = O.matcha_W(partner, 0b11, 0.25, 4)
    assert W.tolist() == [[0.75, 0.25, 0, 0], [0.25, 0.5, 0.25, 0], [0, 0.25, 0.5, 0.25], [0, 0, 0.25, 0.75]]
    assert O.matcha_W(partner, 0b00, 0.25, 4).tolist() == np.eye(4).tolist()
    assert O.matcha_W(partner, 0b10, 0.25, 4).tolist() == [[1, 0, 0, 0], [0, 0.75, 0.25, 0], [0, 0.25, 0.75, 0], [0, 0, 0, 1]]


def test_matcha_W_invariants_and_limits():
    K = 16
    edges, _ = O.random_regular_graph(221100893, K, 3)
    partner = O.greedy_matchings(edges, K)
    m = len(partner)
    L = np.zeros((K, K))
    for (u, v) in edges:
        L[u, u] += 1; L[v, v] += 1; L[u, v] -= 1; L[v, u] -= 1
    a = float(np.float32(0.2))
    # probability 1: every matching active in every iteration -> vanilla decentralized SGD (c_b = 1)
    for t in range(5):
        bits = O.matcha_activation(9, t, m, 1.0)
        assert bits == (1 << m) - 1
        assert np.allclose(O.matcha_W(partner, bits, 0.2, K), np.eye(K) - a * L, atol=1e-15)
    # probability 0: nothing active -> W = I
    assert all(O.matcha_activation(9, t, m, 0.0) == 0 for t in range(50))
    # probability 0.5: frequency -> 0.5; E[W] -> I - alpha p L; each W valid
    T = 4000
    Wsum = np.zeros((K, K))
    act = np.zeros(m)
    for t in range(T):
        bits = O.matcha_activation(9, t, m, 0.5)
        W = O.matcha_W(partner, bits, 0.2, K)
        _assert_doubly_stochastic(W, 1e-12)
        assert np.all(W >= 0) and np.all(np.diag(W) >= 1 - 3 * a - 1e-12)
        allowed = {0.0, a} | {1 - c * a for c in range(4)}
        assert all(min(abs(x - y) for y in allowed) < 1e-12 for x in np.unique(W))
        Wsum += W
        for j in range(m):
            act[j] += (bits >> j) & 1
    assert np.all(np.abs(act / T - 0.5) < 4 * 0.5 / math.sqrt(T))
    assert np.abs(Wsum / T - (np.eye(K) - a * 0.5 * L)).max() < 0.02


# ------------------------------------------------------------------------------------------
# accumulate / normalise
# ------------------------------------------------------------------------------------------
def test_accumulate_is_a_prefix_sum_over_minibatches():
    G = _rand((3, 5, 7), 0)
    acc = O.accumulate(G, [0, 2, 5])
    assert np.all(acc[0] == 0)
    assert np.allclose(acc[1], G[1, 0] + G[1, 1], rtol=0, atol=1e-15)
    assert np.allclose(acc[2], G[2].sum(0), rtol=0, atol=1e-14)
    # abandoned mini-batches have no influence whatsoever
    G2 = G.copy(); G2[1, 2:] = 1e30
    assert np.array_equal(O.accumulate(G2, [0, 2, 5])[1], acc[1])


def test_least_squares_accumulated_gradient_is_the_joint_batch_gradient():
    # Eq. 23: the sum of the mini-batch gradients is the gradient on the joint data of the finished
    # mini-batches.  Learner data (A, b), B rows in M equal mini-batches, loss 1/(2 rows)|Ax-b|^2.
    rng = np.random.default_rng(5)
    Pdim, M, rows = 6, 4, 5
    B = M * rows
    A = rng.standard_normal((B, Pdim)); b = rng.standard_normal(B); x = rng.standard_normal(Pdim)
    G = np.zeros((1, M, Pdim))
    for m in range(M):
        Am, bm = A[m * rows:(m + 1) * rows], b[m * rows:(m + 1) * rows]
        G[0, m] = Am.T @ (Am @ x - bm) / rows                      # mean-convention mini-batch gradient
    for n in range(1, M + 1):
        An, bn = A[:n * rows], b[:n * rows]
        joint = An.T @ (An @ x - bn) / (n * rows)                    # gradient on the joint finished rows
        # "mean" normalisation: one plain SGD step from x with V=0, mom=0, W=I must move by -lr*joint
        Xn, Vn = O.step(x[None, :].copy(), np.zeros((1, Pdim)), G, [n], np.eye(1), 0.5, 0.0, norm="mean")
        assert np.allclose(Vn[0], joint, rtol=1e-12, atol=1e-14)
        assert np.allclose(Xn[0], x - 0.5 * joint, rtol=1e-12, atol=1e-14)
    # "paper" normalisation with sum-convention gradients g_m = A_m^T(A_m x - b_m)/B (Eq. 21-23):
    Gs = G * rows / B
    full = A.T @ (A @ x - b) / B
    Xn, Vn = O.step(x[None, :].copy(), np.zeros((1, Pdim)), Gs, [M], np.eye(1), 0.5, 0.0, norm="paper")
    assert np.allclose(Xn[0], x - 0.5 * full, rtol=1e-12, atol=1e-14)         # n = N: large-batch step
    n = 3
    Xn, _ = O.step(x[None, :].copy(), np.zeros((1, Pdim)), Gs, [n], np.eye(1), 0.5, 0.0, norm="paper")
    assert np.allclose(Xn[0], x - 0.5 * (n / M) * Gs[0, :n].sum(0), rtol=1e-12, atol=1e-14)   # Eq. 19


def test_scale_factors():
    assert O.scale_factors([0, 1, 2, 4], 4, "mean") == [0.0, 1.0, 0.5, 0.25]
    assert O.scale_factors([0, 1, 2, 4], 4, "paper") == [0.0, 0.25, 0.5, 1.0]


# ------------------------------------------------------------------------------------------
# whole step: reductions to textbook updates
# ------------------------------------------------------------------------------------------
def _sync_momentum_sgd(x0, gbar_per_step, lr, mom):
    """Synchronous mini-batch SGD with momentum (Eq. 2 with a velocity), written independently."""
    x = x0.copy(); v = np.zeros_like(x0); traj = []
    for g in gbar_per_step:
        v = mom * v + g
        x = x - lr * v
        traj.append(x.copy())
    return traj


@pytest.mark.parametrize("order", ["mix_then_update", "update_then_mix"])
@pytest.mark.parametrize("K", [3, 4, 5])
def test_all_finished_full_mixing_reduces_to_synchronous_sgd(order, K):
    M, Pdim, steps = 4, 33, 10
    lr, mom = 0.125, 0.5          # exact in fp32
    x0 = _rand(Pdim, 1, 0.01)
    orc = O.Oracle(K, Pdim, M, lr, mom, "allreduce", order=order)
    orc.set_params(x0)
    gbars = []
    for t in range(steps):
        G = _rand((K, M, Pdim), 100 + t)
        gbars.append(G.mean(axis=(0, 1)))                  # (1/K) sum_i (1/M) sum_m
        orc.step(G, [M] * K)
        ref = _sync_momentum_sgd(x0, gbars, lr, mom)[-1]
        assert np.allclose(O.mean_params(orc.X), ref, rtol=1e-12, atol=1e-15)
        if order == "update_then_mix":                     # Eq. 4-5: every learner holds the mean
            for i in range(K):
                assert np.allclose(orc.X[i], ref, rtol=1e-12, atol=1e-15)
    if order == "mix_then_update":                         # Alg. 2 order: learners differ, mean does not
        assert np.abs(orc.X[0] - orc.X[1]).max() > 1e-3


def test_identity_mixing_is_independent_local_sgd():
    K, M, Pdim, steps = 3, 4, 17, 6
    lr, mom = 0.1, 0.9
    x0 = _rand((K, Pdim), 2)
    n_seq = [[1, 4, 2], [3, 3, 1], [4, 4, 4], [2, 1, 3], [1, 1, 1], [4, 2, 3]]
    Gs = [_rand((K, M, Pdim), 200 + t) for t in range(steps)]
    orc = O.Oracle(K, Pdim, M, lr, mom, "dpsgd", W=O.identity_W(K))
    orc.set_params(x0)
    for t in range(steps):
        orc.step(Gs[t], n_seq[t])
    lr32, mom32 = float(np.float32(lr)), float(np.float32(mom))
    for i in range(K):                                     # single-learner momentum SGD, by hand
        x = x0[i].copy(); v = np.zeros(Pdim)
        for t in range(steps):
            g = Gs[t][i, :n_seq[t][i]].sum(0) / n_seq[t][i]
            v = mom32 * v + g
            x = x - lr32 * v
        assert np.allclose(orc.X[i], x, rtol=1e-12, atol=1e-15)


def test_doubly_stochastic_mixing_preserves_the_learner_mean():
    K, M, Pdim = 16, 4, 11
    X = _rand((K, Pdim), 3); V = _rand((K, Pdim), 4)
    Gz = np.zeros((K, M, Pdim))
    for W in (O.ring_W(K), O.full_W(K),
              O.matcha_W(O.greedy_matchings(O.random_regular_graph(3, K, 3)[0], K), 0b101, 0.2, K)):
        # zero gradients and zero velocity: mean is preserved up to the row-sum error of fp32 weights
        Xn, _ = O.step(X, np.zeros_like(V), Gz, [1] * K, W, 0.1, 0.9)
        assert np.allclose(Xn.mean(0), (W.sum(0)[:, None] * X).mean(0), rtol=0, atol=1e-15)
        assert np.allclose(Xn.mean(0), X.mean(0), rtol=0, atol=3e-7)
        # in general: mean(X') = mean(W X) - lr * mean(V')
        G = _rand((K, M, Pdim), 5)
        Xn, Vn = O.step(X, V, G, [2] * K, W, 0.1, 0.9)
        lr32 = float(np.float32(0.1))
        assert np.allclose(Xn.mean(0), (W @ X).mean(0) - lr32 * Vn.mean(0), rtol=0, atol=1e-14)


def test_ring_consensus_follows_the_circulant_spectrum():
    # zero gradients: X^t = W^t X^0; W circulant with eigenvalues w(1 + 2cos(2 pi k/K)) on the DFT basis
    K, Pdim, T = 16, 5, 7
    X0 = _rand((K, Pdim), 6)
    orc = O.Oracle(K, Pdim, 2, 0.1, 0.9, "dpsgd", W=O.ring_W(K))
    orc.set_params(X0)
    for _ in range(T):
        orc.step(np.zeros((K, 2, Pdim)), [1] * K)
    w = float(np.float32(1 / 3))
    lam = w * (1 + 2 * np.cos(2 * np.pi * np.arange(K) / K))
    want = np.fft.ifft((lam ** T)[:, None] * np.fft.fft(X0, axis=0), axis=0).real
    assert np.allclose(orc.X, want, rtol=0, atol=1e-13)


def test_update_then_mix_is_the_dpsgd_baseline_rule():
    # Eq. 6: x_i <- sum_j W_ij (x_j - lr g_j), here with mom = 0
    K, M, Pdim = 5, 2, 9
    X = _rand((K, Pdim), 7); G = _rand((K, M, Pdim), 8); W = O.ring_W(K)
    lr32 = float(np.float32(0.3))
    Xn, _ = O.step(X, np.zeros((K, Pdim)), G, [M] * K, W, 0.3, 0.0, order="update_then_mix")
    assert np.allclose(Xn, W @ (X - lr32 * G.mean(1)), rtol=1e-13, atol=1e-15)
    Xa, _ = O.step(X, np.zeros((K, Pdim)), G, [M] * K, W, 0.3, 0.0, order="mix_then_update")
    assert np.allclose(Xa, W @ X - lr32 * G.mean(1), rtol=1e-13, atol=1e-15)     # Alg. 2


def test_zero_finished_learner_only_mixes_and_decays():
    K, M, Pdim = 3, 2, 4
    X = _rand((K, Pdim), 9); V = _rand((K, Pdim), 10); G = _rand((K, M, Pdim), 11)
    Xn, Vn = O.step(X, V, G, [0, 1, 2], O.identity_W(K), 0.1, 0.5)
    assert np.allclose(Vn[0], 0.5 * V[0]) and np.allclose(Xn[0], X[0] - float(np.float32(0.1)) * Vn[0])


# ------------------------------------------------------------------------------------------
# brute force in exact rationals, tiny sizes
# ------------------------------------------------------------------------------------------
def _frac_matrix(a):
    return [[Fraction(float(v)) for v in row] for row in a]


@pytest.mark.parametrize("K,Pdim,M,norm,order", [
    (4, 8, 4, "mean", "mix_then_update"),
    (3, 5, 3, "paper", "mix_then_update"),
    (4, 6, 2, "mean", "update_then_mix"),
    (2, 64, 4, "paper", "update_then_mix"),
    (1, 3, 1, "mean", "mix_then_update"),
])
def test_step_against_exact_rational_matrix_form(K, Pdim, M, norm, order):
    """V' = mom V + diag(s) A,  X' = W X - lr V'  (or W (X - lr V')), with Python Fractions."""
    rng = np.random.default_rng(K * 100 + Pdim)
    # small dyadic values keep fp64 exact enough that the oracle must match to ~1e-15
    X = rng.integers(-8, 9, (K, Pdim)) / 8.0
    V = rng.integers(-8, 9, (K, Pdim)) / 16.0
    G = rng.integers(-16, 17, (K, M, Pdim)) / 4.0
    n = [int(v) for v in rng.integers(0, M + 1, K)]
    if K >= 3:
        W = O.ring_W(K)
    elif K == 2:
        W = np.array([[0.75, 0.25], [0.25, 0.75]])
    else:
        W = np.eye(1)
    lr, mom = 0.25, 0.5
    Xn, Vn = O.step(X, V, G, n, W, lr, mom, norm=norm, order=order)
    fX, fV, fW = _frac_matrix(X), _frac_matrix(V), _frac_matrix(W)
    flr, fmom = Fraction(lr), Fraction(mom)
    fVn = [[None] * Pdim for _ in range(K)]
    for i in range(K):
        s = (Fraction(0) if n[i] == 0 else Fraction(1, n[i])) if norm == "mean" else Fraction(n[i], M)
        for p in range(Pdim):
            a = sum((Fraction(float(G[i, m, p])) for m in range(n[i])), Fraction(0))
            fVn[i][p] = fmom * fV[i][p] + s * a
    for i in range(K):
        for p in range(Pdim):
            if order == "mix_then_update":
                want = sum(fW[i][j] * fX[j][p] for j in range(K)) - flr * fVn[i][p]
            else:
                want = sum(fW[i][j] * (fX[j][p] - flr * fVn[j][p]) for j in range(K))
            assert abs(Fraction(float(Xn[i, p])) - want) <= Fraction(1, 10 ** 14)
            assert abs(Fraction(float(Vn[i, p])) - fVn[i][p]) <= Fraction(1, 10 ** 14)


def test_step_against_dense_numpy_matrix_form():
    K, M, Pdim = 4, 4, 64
    X = _rand((K, Pdim), 20); V = _rand((K, Pdim), 21); G = _rand((K, M, Pdim), 22)
    n = [1, 4, 2, 3]
    W = O.matcha_W([[1, 0, 3, 2], [2, 3, 0, 1]], 0b01, 0.2, K)
    Xn, Vn = O.step(X, V, G, n, W, 0.05, 0.9)
    mask = (np.arange(M)[None, :] < np.array(n)[:, None]).astype(float)
    A = np.einsum("km,kmp->kp", mask, G)
    Vw = float(np.float32(0.9)) * V + np.diag(1.0 / np.array(n)) @ A
    assert np.allclose(Vn, Vw, rtol=1e-13, atol=1e-15)
    assert np.allclose(Xn, W @ X - float(np.float32(0.05)) * Vw, rtol=1e-13, atol=1e-15)


# ------------------------------------------------------------------------------------------
# centralized (parameter-server) variant
# ------------------------------------------------------------------------------------------
def test_centralized_step_equals_synchronous_sgd_and_the_allreduce_mean():
    K, M, Pdim, steps = 4, 4, 12, 5
    lr, mom = 0.25, 0.5
    x0 = _rand(Pdim, 30)
    x = x0.copy(); v = np.zeros(Pdim)
    orc = O.Oracle(K, Pdim, M, lr, mom, "allreduce")
    orc.set_params(x0)
    gbars = []
    for t in range(steps):
        G = _rand((K, M, Pdim), 300 + t)
        n = [M] * K if t % 2 == 0 else [1, 2, 3, 4]
        x, v = O.step_centralized(x, v, G, n, lr, mom)
        orc.step(G, n)
        gbars.append(np.mean([G[i, :n[i]].mean(0) for i in range(K)], axis=0))
        # Eq. 2 on the per-learner mean gradients
        assert np.allclose(x, _sync_momentum_sgd(x0, gbars, lr, mom)[-1], rtol=1e-12, atol=1e-15)
        # the decentralized all-reduce variant's output (mean model) follows the same trajectory
        assert np.allclose(O.mean_params(orc.X), x, rtol=1e-12, atol=1e-15)


def test_mean_params():
    X = np.arange(12.0).reshape(3, 4)
    assert O.mean_params(X).tolist() == [4.0, 5.0, 6.0, 7.0]


# ------------------------------------------------------------------------------------------
# MATCHA's design problem: activation probabilities under a budget, step size alpha
# ------------------------------------------------------------------------------------------
def _path_matchings():
    # path 0-1-2-3-4-5 split into two matchings; plus a chord matching {0-5}
    return [[1, 0, 3, 2, 5, 4], [-1, 2, 1, 4, 3, -1], [5, -1, -1, -1, -1, 0]]


def test_second_moment_closed_form_equals_enumeration_over_activation_patterns():
    K = 6
    partner = _path_matchings()
    Ls = O.matching_laplacians(partner, K)
    p, alpha = [0.7, 0.35, 0.9], 0.3
    want = np.zeros((K, K))
    for pattern in range(8):                                   # all 2^m activation patterns, exactly
        prob = 1.0
        for j in range(3):
            prob *= p[j] if (pattern >> j) & 1 else 1.0 - p[j]
        W = np.eye(K) - alpha * sum((Ls[j] for j in range(3) if (pattern >> j) & 1), np.zeros((K, K)))
        want += prob * (W.T @ W)
    assert np.allclose(O.matcha_second_moment(Ls, p, alpha), want, rtol=0, atol=1e-14)
    for L in Ls:                                                 # the identity the closed form rests on
        assert np.array_equal(L @ L, 2.0 * L)


def test_probability_projection():
    q = O.project_budget(np.array([0.9, 0.8, -0.2, 1.4]), 10.0)
    assert q.tolist() == [0.9, 0.8, 0.0, 1.0]
    q = O.project_budget(np.array([0.9, 0.8, 0.7]), 1.2)
    assert abs(q.sum() - 1.2) < 1e-9 and np.all(q >= 0) and np.all(q <= 1)
    assert np.allclose(q - q[0], np.array([0.0, -0.1, -0.2]), atol=1e-9)   # equal shift of the free coordinates
    # brute force: no feasible grid point is closer
    target = np.array([0.9, 0.8, 0.7])
    best = min(((np.array([a, b, c]) - target) @ (np.array([a, b, c]) - target))
               for a in np.linspace(0, 1, 41) for b in np.linspace(0, 1, 41) for c in np.linspace(0, 1, 41)
               if a + b + c <= 1.2 + 1e-12)
    assert (q - target) @ (q - target) <= best + 1e-9


def test_algebraic_connectivity_against_textbook_spectra():
    """matcha_lambda2 is the SECOND smallest Laplacian eigenvalue of sum_j p_j L_j.  Closed forms:
    path graph on K vertices 2 - 2 cos(pi/K) (its eigenvalues 2 - 2 cos(pi k/K) are all distinct, so
    taking a neighbouring index fails), cycle 2 - 2 cos(2 pi/K), complete graph K; it scales
    linearly in a common activation probability."""
    for K in (5, 6, 9):
        even = [[-1] * K for _ in range(2)]
        for u in range(K - 1):                               # edges (0,1),(2,3),... and (1,2),(3,4),...
            even[u % 2][u], even[u % 2][u + 1] = u + 1, u
        Ls = O.matching_laplacians(even, K)
        want = 2.0 - 2.0 * math.cos(math.pi / K)
        assert O.matcha_lambda2(Ls, [1.0, 1.0]) == pytest.approx(want, abs=1e-12)
        assert O.matcha_lambda2(Ls, [0.25, 0.25]) == pytest.approx(0.25 * want, abs=1e-12)
        third = 2.0 - 2.0 * math.cos(2.0 * math.pi / K)      # the next eigenvalue of the path is different
        assert abs(third - want) > 0.1
    for K in (6, 8, 10):                                     # even cycle = two perfect matchings
        cyc = [[-1] * K for _ in range(2)]
        for u in range(K):
            v = (u + 1) % K
            cyc[u % 2][u], cyc[u % 2][v] = v, u
        assert O.matcha_lambda2(O.matching_laplacians(cyc, K), [1.0, 1.0]) == \
            pytest.approx(2.0 - 2.0 * math.cos(2.0 * math.pi / K), abs=1e-12)
    for K in (4, 6, 8):                                      # complete graph: round-robin 1-factorisation
        fac = []
        for r in range(K - 1):
            row = [-1] * K
            row[K - 1], row[r] = r, K - 1
            for k in range(1, K // 2):
                u, v = (r + k) % (K - 1), (r - k) % (K - 1)
                row[u], row[v] = v, u
            fac.append(row)
        Ls = O.matching_laplacians(fac, K)
        assert np.allclose(sum(Ls), K * np.eye(K) - np.ones((K, K)))      # the union is the complete graph
        assert O.matcha_lambda2(Ls, [1.0] * (K - 1)) == pytest.approx(float(K), abs=1e-10)


def test_optimal_probabilities_against_grid_search():
    K = 6
    Ls = O.matching_laplacians(_path_matchings(), K)
    budget = 0.5
    p, lam = O.matcha_optimal_probs(Ls, budget, iters=1500)
    assert np.all(p >= -1e-12) and np.all(p <= 1 + 1e-12) and p.sum() <= budget * 3 + 1e-9
    grid = np.linspace(0, 1, 51)
    best = max(O.matcha_lambda2(Ls, (a, b, c)) for a in grid for b in grid for c in grid
               if a + b + c <= budget * 3 + 1e-12)
    assert lam >= best - 1e-4                                    # as good as any grid point (iteration accuracy)
    assert lam <= best + 0.02                                    # and the grid (step 0.02) nearly reaches it
    assert lam > O.matcha_lambda2(Ls, [budget] * 3) + 1e-3       # better than spending the budget uniformly
    # full budget: every matching always active
    p1, lam1 = O.matcha_optimal_probs(Ls, 1.0, iters=200)
    assert np.allclose(p1, 1.0) and lam1 == pytest.approx(O.matcha_lambda2(Ls, [1, 1, 1]))


def test_optimal_alpha_against_grid_and_contraction():
    K = 16
    edges, _ = O.random_regular_graph(221100893, K, 3)
    partner = O.greedy_matchings(edges, K)
    Ls = O.matching_laplacians(partner, K)
    p, lam = O.matcha_optimal_probs(Ls, 0.5, iters=800)
    assert lam > 0                                               # expected topology is connected
    a, rho = O.matcha_optimal_alpha(Ls, p)
    grid = np.linspace(0.0, 1.0, 2001)
    vals = [O.matcha_rho(Ls, p, x) for x in grid]
    assert rho <= min(vals) + 1e-9 and abs(a - grid[int(np.argmin(vals))]) < 2e-3
    assert 0.0 < rho < 1.0                                       # mixing contracts the disagreement
    assert O.matcha_rho(Ls, p, 0.0) == pytest.approx(1.0)        # alpha = 0: W = I, no mixing
    # rho is convex in alpha
    assert all(vals[i] <= 0.5 * (vals[i - 1] + vals[i + 1]) + 1e-12 for i in range(1, len(vals) - 1))


def test_activation_with_per_matching_probabilities():
    probs = [0.0, 1.0, 0.25, 0.75]
    freq = np.zeros(4)
    T = 8000
    for t in range(T):
        bits = O.matcha_activation_probs(5, t, probs)
        for j in range(4):
            freq[j] += (bits >> j) & 1
    assert freq[0] == 0 and freq[1] == T
    assert abs(freq[2] / T - 0.25) < 0.02 and abs(freq[3] / T - 0.75) < 0.02
    # equal probabilities reduce to the single-probability form
    assert all(O.matcha_activation_probs(9, t, [0.5] * 5) == O.matcha_activation(9, t, 5, 0.5) for t in range(200))
