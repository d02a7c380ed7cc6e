"""CPU oracle for the Non-blocking SGD aggregate-and-update step.

THIS FILE IS TEST INFRASTRUCTURE, NOT PRODUCT CODE.  It is a plain, slow, fp64
restatement of what the path computes, written from the paper's statement of the
method.  It shares no code with the CUDA library and imports nothing from it.
Only the tests, the smoke check and the benchmark's CPU-baseline leg may call it.

Notation (paper symbol -> name used here):
  number of learners           P        -> K
  parameter dimension          d        -> P
  mini-batches per batch       N        -> M
  finished mini-batches        n_{k,i}  -> n[i]
  learning rate                eta      -> lr
  mixing matrix                W (PxP)  -> W (KxK)

What follows the paper, and where:
  accumulate   sum_{j<=n_i} grad F_i(x_i; xi_{i,j})     Alg. 1 / Alg. 2 accumulate step, Eq. 19
  LR adjust    eta_i = eta * n_i / N                    Sec. 3.2 "Adjust learning rate", Eq. 19
  mix          x_{k+1/2,i} = sum_p W_{i,p} x_{k,p}      Alg. 2 averaging step
  update       x_{k+1,i} = x_{k+1/2,i} - eta * (...)    Alg. 2 update step
  all-reduce   local update then mean over learners     Eq. 4-5
  D-PSGD base  x_i <- sum_j W_ij (x_j - eta g_j)        Eq. 6  (order "update_then_mix")
  centralized  x_ps <- x_ps - sum_i eta_i (...)          Alg. 3 server update
  output       (1/K) sum_i x_i                          Alg. 1 / Alg. 2 "Output"
  stragglers   one delay per learner per iteration,     Sec. 4.1 (exponential delays),
               constant speed inside an iteration,      Sec. 4.3 (constant speed, Corollary 1),
               first finisher ends the iteration        Alg. 1 inner loop

Readings the paper leaves open (each is a documented choice of this repository):
  * momentum is not in the paper; v <- mom*v + ghat, x <- x_half - lr*v (mom = 0 is the paper's update);
  * norm "mean":  ghat_i = acc_i / n_i  (mean of the finished mini-batch gradients);
    norm "paper": ghat_i = (n_i / M) * acc_i  (literal Alg. 2 update step, sum-convention gradients);
  * the counter-based generator below is this repository's own (parity unpinned as a choice; its
    arithmetic is pinned to the published SplitMix64 finaliser outputs in the tests);
  * the random regular graph construction and the greedy matching decomposition are this
    repository's own (the paper only says links are disjoint and activated with a probability).

Scalars that cross the library boundary as fp32 (lr, mom, alpha, W entries, activation probability)
are taken here as those fp32 values widened to double, so both sides see the same numbers.
"""
import math

import numpy as np

MASK64 = (1 << 64) - 1
GOLDEN = 0x9E3779B97F4A7C15

STREAM_INIT = 0
STREAM_GRAD = 1
STREAM_STRAGGLER = 2
STREAM_MATCHA = 3
STREAM_GRAPH = 4
STREAM_SLOWSET = 5


# ----------------------------------------------------------------------------------------------
# Counter-based generator (repository's own specification; finaliser = SplitMix64's output mix)
# ----------------------------------------------------------------------------------------------
def mix64(z):
    z &= MASK64
    z = ((z ^ (z >> 30)) * 0xBF58476D1CE4E5B9) & MASK64
    z = ((z ^ (z >> 27)) * 0x94D049BB133111EB) & MASK64
    return (z ^ (z >> 31)) & MASK64


def rng(seed, stream, a, b):
    """64 random bits addressed by (seed, stream, a, b); no state."""
    h = mix64(seed + GOLDEN)
    h = mix64(h + stream + GOLDEN)
    h = mix64(h + a + GOLDEN)
    h = mix64(h + b + GOLDEN)
    return h


def uniform01(r):
    """Map 64 random bits to a double in (0, 1]: never 0, so its logarithm is finite (the top
    value rounds to exactly 1.0, a zero delay)."""
    return ((r >> 11) + 0.5) * (2.0 ** -53)


def f32(x):
    """The fp32 value nearest to x, widened back to a Python float."""
    return float(np.float32(x))


# ----------------------------------------------------------------------------------------------
# Straggler simulator: stands in for the terminal signal of Alg. 1 inner loop
# ----------------------------------------------------------------------------------------------
def counts_uniform(seed, t, K, M):
    """Finished counts drawn uniformly from {1..M}, one per learner (the tiny configuration)."""
    return [1 + (rng(seed, STREAM_STRAGGLER, t, i) % M) for i in range(K)]


def delays_shifted_exp(seed, t, K, delta):
    """Per-learner mini-batch time tau_i = 1 + Exp(mean delta_i): one delay per learner per
    iteration (Sec. 4.1: i.i.d. exponential mini-batch times; Appendix A Remark 1: mean 1/lambda)."""
    tau = []
    for i in range(K):
        u = uniform01(rng(seed, STREAM_STRAGGLER, t, i))
        tau.append(1.0 + (-(float(delta[i])) * math.log(u)))
    return tau


def counts_from_delays(tau, M):
    """The fastest learner finishes all M mini-batches at T = M * min(tau) and raises the terminal
    signal (Alg. 1, broadcast step); learner i, working at constant speed (Sec. 4.3), has finished the
    mini-batches j with j * tau_i <= T; the one in flight is abandoned (Alg. 1, break step).  At least
    one mini-batch is counted for every learner."""
    T = float(M) * min(tau)
    out = []
    for tau_i in tau:
        c = 0
        for j in range(1, M + 1):
            if float(j) * tau_i <= T:
                c += 1
        out.append(max(1, c))
    return out


def slow_set(seed, t, K, n_slow):
    """Indices of the learners that are slow in iteration t (re-drawn every iteration, Sec. 6.1
    "Machines/Clusters"): the first n_slow entries of a partial Fisher-Yates shuffle of 0..K-1."""
    idx = list(range(K))
    for q in range(n_slow):
        r = rng(seed, STREAM_SLOWSET, t, q) % (K - q)
        idx[q], idx[q + r] = idx[q + r], idx[q]
    return idx[:n_slow]


def straggler_counts(model, seed, t, K, M, params=()):
    """model: "uniform_count" | "shifted_exp" (params = [delta]) |
    "shifted_exp_slowset" (params = [slow_fraction, delta_slow, delta_fast])."""
    if model == "uniform_count":
        return counts_uniform(seed, t, K, M)
    if model == "shifted_exp":
        return counts_from_delays(delays_shifted_exp(seed, t, K, [params[0]] * K), M)
    if model == "shifted_exp_slowset":
        frac, d_slow, d_fast = params
        n_slow = int(math.floor(frac * K))
        slow = set(slow_set(seed, t, K, n_slow))
        delta = [d_slow if i in slow else d_fast for i in range(K)]
        return counts_from_delays(delays_shifted_exp(seed, t, K, delta), M)
    raise ValueError(model)


def runtime_report(model, seed, K, M, steps, params=(), step0=0):
    """Run-time figures of the straggler model averaged over `steps` iterations (Sec. 4.2-4.3):
    Non-blocking SGD waits for the fastest learner, M*min(tau) per iteration (Lemma 1); a blocking
    method waits for the slowest, M*max(tau); their ratio is Theorem 1's; the throughput ratio is
    Theorem 5's Y*X_{K:K}/K with Y = sum_i 1/tau_i; Corollary 1's data per iteration, as a fraction
    of K batches, is Y*X_{1:K}/K; the floor rule gives sum n_i/(K*M)."""
    t_nb = t_bl = thr = frac = fin = tmin_s = tmax_s = 0.0
    for t in range(step0, step0 + steps):
        if model == "shifted_exp":
            delta = [params[0]] * K
        elif model == "shifted_exp_slowset":
            slow = set(slow_set(seed, t, K, int(math.floor(params[0] * K))))
            delta = [params[1] if i in slow else params[2] for i in range(K)]
        else:
            raise ValueError(model)
        tau = delays_shifted_exp(seed, t, K, delta)
        n = counts_from_delays(tau, M)
        Y = 0.0
        for x in tau:
            Y += 1.0 / x
        t_nb += float(M) * min(tau)
        t_bl += float(M) * max(tau)
        thr += Y * max(tau) / float(K)
        frac += Y * min(tau) / float(K)
        fin += float(sum(n)) / (float(K) * float(M))
        tmin_s += min(tau)
        tmax_s += max(tau)
    inv = 1.0 / float(steps)
    return {"mean_t_nonblocking": t_nb * inv, "mean_t_blocking": t_bl * inv, "ratio": t_nb / t_bl,
            "mean_throughput_ratio": thr * inv, "mean_fractional_data": frac * inv,
            "mean_finished_fraction": fin * inv, "mean_min_tau": tmin_s * inv, "mean_max_tau": tmax_s * inv,
            "steps": steps}


def finished_mask(n, M):
    """mask[i][m] = 1 iff mini-batch m of learner i was finished; unfinished ones are a suffix
    because a learner leaves its loop at the terminal signal (Alg. 1 inner loop)."""
    return np.array([[1 if m < n_i else 0 for m in range(M)] for n_i in n], dtype=np.uint8)


# ----------------------------------------------------------------------------------------------
# Topologies and mixing matrices
# ----------------------------------------------------------------------------------------------
def full_W(K):
    """All-reduce variant: W = (1/K) 1 1^T (Eq. 5 written as a mixing matrix), with the exact 1/K."""
    return np.full((K, K), 1.0 / K, dtype=np.float64)


def ring_W(K):
    """Ring with W_ii = W_{i,i+-1} = 1/3 (indices mod K; coinciding neighbours add up)."""
    w = f32(1.0 / 3.0)
    W = np.zeros((K, K), dtype=np.float64)
    for i in range(K):
        W[i, i] += w
        W[i, (i + 1) % K] += w
        W[i, (i - 1) % K] += w
    return W


def identity_W(K):
    return np.eye(K, dtype=np.float64)


def random_regular_graph(seed, K, d):
    """Simple connected d-regular graph on K vertices by the configuration model with rejection.
    Attempt a shuffles the d*K stubs with draws rng(seed, GRAPH, a, s) and pairs neighbours.
    Returns (sorted edge list of (min, max), attempts used)."""
    if (K * d) % 2 != 0 or d >= K:
        raise ValueError("no simple d-regular graph with these K, d")
    for a in range(100000):
        stubs = [v for v in range(K) for _ in range(d)]
        for s in range(d * K - 1, 0, -1):
            r = rng(seed, STREAM_GRAPH, a, s) % (s + 1)
            stubs[s], stubs[r] = stubs[r], stubs[s]
        edges = set()
        ok = True
        for e in range(0, d * K, 2):
            u, v = stubs[e], stubs[e + 1]
            if u == v:
                ok = False
                break
            key = (min(u, v), max(u, v))
            if key in edges:
                ok = False
                break
            edges.add(key)
        if not ok:
            continue
        adj = [[] for _ in range(K)]
        for (u, v) in edges:
            adj[u].append(v)
            adj[v].append(u)
        seen = [False] * K
        seen[0] = True
        stack = [0]
        while stack:
            u = stack.pop()
            for v in adj[u]:
                if not seen[v]:
                    seen[v] = True
                    stack.append(v)
        if all(seen):
            return sorted(edges), a + 1
    raise RuntimeError("no graph found")


def greedy_matchings(edges, K):
    """Decompose a graph into matchings: edges in lexicographic (min, max) order, each takes the
    smallest colour unused at both endpoints.  Returns partner[c][v] (-1 = unmatched in colour c).
    Any proper edge colouring would be a valid decomposition; this is the deterministic one used."""
    used = [set() for _ in range(K)]
    partner = []
    for (u, v) in sorted(edges):
        c = 0
        while c in used[u] or c in used[v]:
            c += 1
        while len(partner) <= c:
            partner.append([-1] * K)
        partner[c][u] = v
        partner[c][v] = u
        used[u].add(c)
        used[v].add(c)
    return partner


def matcha_activation(seed, t, n_matchings, prob):
    """Bit j = 1 iff matching j is active in iteration t: an independent Bernoulli(prob) draw per
    matching per iteration (Sec. 6.1: links become active in some iterations with a probability;
    the budget c_b is the average activation frequency)."""
    thr = int(math.floor(f32(prob) * 4294967296.0))
    bits = 0
    for j in range(n_matchings):
        if (rng(seed, STREAM_MATCHA, t, j) >> 32) < thr:
            bits |= (1 << j)
    return bits


def matcha_W(partner, bits, alpha, K):
    """W = I - alpha * sum_{active j} L_j, L_j the Laplacian of matching j."""
    a = f32(alpha)
    W = np.eye(K, dtype=np.float64)
    for j, row in enumerate(partner):
        if not (bits >> j) & 1:
            continue
        for u in range(K):
            v = row[u]
            if v >= 0 and u < v:
                W[u, u] -= a
                W[v, v] -= a
                W[u, v] += a
                W[v, u] += a
    return W


# ----------------------------------------------------------------------------------------------
# MATCHA's design problem (Sec. 6.1 names it: a communication budget c_b = average activation
# frequency of the links, probabilities that favour the links that matter for connectivity; the
# optimisation itself is only referenced there, so it is stated here from first principles):
#   L_bar(p) = sum_j p_j L_j                          expected Laplacian of the activated topology
#   probabilities: maximise lambda_2(L_bar(p))  s.t.  0 <= p_j <= 1,  sum_j p_j <= c_b * m
#   step size:     minimise rho(alpha) = || E[W^T W] - (1/K) 1 1^T ||_2,  W = I - alpha * L(k),
#                  E[W^T W] = I - 2 alpha L_bar + alpha^2 (L_bar^2 + 2 sum_j p_j (1 - p_j) L_j)
#                  (independent Bernoulli activations; L_j^2 = 2 L_j for a matching)
# ----------------------------------------------------------------------------------------------
def matching_laplacians(partner, K):
    Ls = []
    for row in partner:
        L = np.zeros((K, K), dtype=np.float64)
        for u in range(K):
            v = row[u]
            if v >= 0 and u < v:
                L[u, u] += 1.0
                L[v, v] += 1.0
                L[u, v] -= 1.0
                L[v, u] -= 1.0
        Ls.append(L)
    return Ls


def matcha_lambda2(Ls, p):
    """Algebraic connectivity (second smallest eigenvalue) of the expected Laplacian."""
    Lbar = sum(float(pj) * L for pj, L in zip(p, Ls))
    return float(np.linalg.eigvalsh(Lbar)[1])


def project_budget(p, total):
    """Euclidean projection onto {0 <= p_j <= 1, sum_j p_j <= total}."""
    q = np.clip(p, 0.0, 1.0)
    if q.sum() <= total:
        return q
    lo, hi = 0.0, float(np.max(p))
    for _ in range(100):
        mid = 0.5 * (lo + hi)
        if np.clip(p - mid, 0.0, 1.0).sum() > total:
            lo = mid
        else:
            hi = mid
    return np.clip(p - hi, 0.0, 1.0)


def matcha_optimal_probs(Ls, budget, iters=2000):
    """Projected supergradient ascent on the concave function p -> lambda_2(L_bar(p)); a
    supergradient is g_j = v^T L_j v for a unit Fiedler vector v.  Returns (p, lambda_2)."""
    m = len(Ls)
    total = float(budget) * m
    p = project_budget(np.full(m, float(budget)), total)
    best_p, best = p.copy(), matcha_lambda2(Ls, p)
    for it in range(1, iters + 1):
        Lbar = sum(pj * L for pj, L in zip(p, Ls))
        w, V = np.linalg.eigh(Lbar)
        v = V[:, 1]
        g = np.array([float(v @ L @ v) for L in Ls])
        nrm = float(np.linalg.norm(g))
        if nrm == 0.0:
            break
        p = project_budget(p + (0.5 / math.sqrt(it)) * g / nrm, total)
        val = matcha_lambda2(Ls, p)
        if val > best:
            best, best_p = val, p.copy()
    return best_p, best


def matcha_second_moment(Ls, p, alpha):
    """E[W^T W] for W = I - alpha * sum_j B_j L_j with independent B_j ~ Bernoulli(p_j)."""
    K = Ls[0].shape[0]
    Lbar = sum(float(pj) * L for pj, L in zip(p, Ls))
    Ltil = sum(float(pj) * (1.0 - float(pj)) * L for pj, L in zip(p, Ls))
    return np.eye(K) - 2.0 * alpha * Lbar + alpha * alpha * (Lbar @ Lbar + 2.0 * Ltil)


def matcha_rho(Ls, p, alpha):
    """Spectral norm of E[W^T W] - J, J = (1/K) 1 1^T: the per-step contraction of the disagreement."""
    K = Ls[0].shape[0]
    A = matcha_second_moment(Ls, p, alpha) - np.full((K, K), 1.0 / K)
    return float(np.max(np.abs(np.linalg.eigvalsh(A))))


def matcha_optimal_alpha(Ls, p, iters=80):
    """rho(alpha) is a maximum of convex quadratics in alpha, hence convex: golden-section search."""
    lo, hi = 0.0, 1.0
    gr = (math.sqrt(5.0) - 1.0) / 2.0
    c, d = hi - gr * (hi - lo), lo + gr * (hi - lo)
    fc, fd = matcha_rho(Ls, p, c), matcha_rho(Ls, p, d)
    for _ in range(iters):
        if fc < fd:
            hi, d, fd = d, c, fc
            c = hi - gr * (hi - lo)
            fc = matcha_rho(Ls, p, c)
        else:
            lo, c, fc = c, d, fd
            d = lo + gr * (hi - lo)
            fd = matcha_rho(Ls, p, d)
    a = 0.5 * (lo + hi)
    return a, matcha_rho(Ls, p, a)


def matcha_activation_probs(seed, t, probs):
    """Activation word with one probability per matching (fp32 values widened, as the library
    receives them): bit j = 1 iff the top 32 random bits fall below floor(p_j * 2^32)."""
    bits = 0
    for j, pj in enumerate(probs):
        thr = int(math.floor(f32(pj) * 4294967296.0))
        if (rng(seed, STREAM_MATCHA, t, j) >> 32) < thr:
            bits |= (1 << j)
    return bits


# ----------------------------------------------------------------------------------------------
# The step
# ----------------------------------------------------------------------------------------------
def accumulate(G, n):
    """acc_i = sum_{m < n_i} G[i, m, :] in fp64, m ascending (Alg. 1 accumulate step; Eq. 19)."""
    K, M, P = G.shape
    acc = np.zeros((K, P), dtype=np.float64)
    for i in range(K):
        for m in range(int(n[i])):
            acc[i] += G[i, m].astype(np.float64)
    return acc


def scale_factors(n, M, norm):
    s = []
    for n_i in n:
        if norm == "mean":
            s.append(0.0 if n_i == 0 else 1.0 / float(n_i))
        elif norm == "paper":
            s.append(float(n_i) / float(M))
        else:
            raise ValueError(norm)
    return s


def step(X, V, G, n, W, lr, mom, norm="mean", order="mix_then_update"):
    """One iteration for all learners.  X, V: [K, P] float64 (not modified).  G: [K, M, P] any
    float dtype (the exact values the GPU receives).  n: finished counts.  W: [K, K] float64.
    Returns (X_next, V_next)."""
    K, M, P = G.shape
    lr = f32(lr)
    mom = f32(mom)
    acc = accumulate(G, n)
    s = scale_factors(n, M, norm)
    Vn = np.empty_like(V)
    for i in range(K):
        Vn[i] = mom * V[i] + s[i] * acc[i]
    Xn = np.zeros_like(X)
    if order == "mix_then_update":  # Alg. 2: average the old models, then step
        for i in range(K):
            for j in range(K):
                if W[i, j] != 0.0:
                    Xn[i] += W[i, j] * X[j]
            Xn[i] -= lr * Vn[i]
    elif order == "update_then_mix":  # Eq. 4-6: local step, then average
        Y = np.empty_like(X)
        for j in range(K):
            Y[j] = X[j] - lr * Vn[j]
        for i in range(K):
            for j in range(K):
                if W[i, j] != 0.0:
                    Xn[i] += W[i, j] * Y[j]
    else:
        raise ValueError(order)
    return Xn, Vn


def step_centralized(x_ps, v_ps, G, n, lr, mom, norm="mean"):
    """Non-blocking synchronous centralized step (Alg. 3, server update and broadcast): one shared model; the
    learners' scaled accumulated gradients are combined (as a mean over learners, matching Eq. 2)
    and the parameter-server model takes a momentum step.  x_ps, v_ps: [P] float64."""
    K, M, P = G.shape
    lr = f32(lr)
    mom = f32(mom)
    acc = accumulate(G, n)
    s = scale_factors(n, M, norm)
    g = np.zeros(P, dtype=np.float64)
    for i in range(K):
        g += s[i] * acc[i]
    g /= float(K)
    v_new = mom * v_ps + g
    return x_ps - lr * v_new, v_new


def mean_params(X):
    """Output of Alg. 1 / Alg. 2: the average of all workers' models."""
    K = X.shape[0]
    out = np.zeros(X.shape[1], dtype=np.float64)
    for i in range(K):
        out += X[i]
    return out / float(K)


class Oracle:
    """Holds X, V (fp64) and the step counter for one run; thin wrapper over step()."""

    def __init__(self, K, P, M, lr, mom, variant, W=None, partner=None, alpha=0.0, prob=0.0,
                 seed=0, norm="mean", order="mix_then_update"):
        self.K, self.P, self.M = K, P, M
        self.lr, self.mom = lr, mom
        self.variant = variant  # "allreduce" | "dpsgd" | "matcha"
        self.W = W
        self.partner, self.alpha, self.prob, self.seed = partner, alpha, prob, seed
        self.norm, self.order = norm, order
        self.t = 0
        self.X = np.zeros((K, P), dtype=np.float64)
        self.V = np.zeros((K, P), dtype=np.float64)

    def set_params(self, x0):
        x0 = np.asarray(x0, dtype=np.float64)
        if x0.ndim == 1:  # identical initialisation of all learners (Alg. 1 initialisation)
            for i in range(self.K):
                self.X[i] = x0
        else:
            self.X[:] = x0
        self.V[:] = 0.0

    def mixing_matrix(self, t):
        if self.variant == "allreduce":
            return full_W(self.K)
        if self.variant == "dpsgd":
            return self.W
        if self.variant == "matcha":
            if isinstance(self.prob, (list, tuple, np.ndarray)):
                bits = matcha_activation_probs(self.seed, t, self.prob)
            else:
                bits = matcha_activation(self.seed, t, len(self.partner), self.prob)
            return matcha_W(self.partner, bits, self.alpha, self.K)
        raise ValueError(self.variant)

    def step(self, G, n):
        W = self.mixing_matrix(self.t)
        self.X, self.V = step(self.X, self.V, G, n, W, self.lr, self.mom, self.norm, self.order)
        self.t += 1
