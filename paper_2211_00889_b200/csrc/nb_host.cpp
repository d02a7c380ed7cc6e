// Host-only parts of the library: the straggler simulator that stands in for the terminal signal
// of Alg. 1, and the topology / mixing-matrix builders (ring, full, explicit CSR, explicit
// matchings, seeded random regular graph with a greedy matching decomposition).  No CUDA here.
#include <algorithm>
#include <cmath>
#include <cstring>
#include <set>
#include <utility>

#include "nb_internal.h"

namespace nb {

namespace {

// 64 random bits -> double in (0, 1]; never 0, so log() is finite.
inline double uniform01(uint64_t r) { return ((double)(r >> 11) + 0.5) * 0x1.0p-53; }

bool check_doubly_stochastic(const Mixing &mx, std::string *err) {
  const int K = mx.K;
  std::vector<double> rs(K, 0.0), cs(K, 0.0);
  for (int i = 0; i < K; ++i)
    for (int e = mx.row_ptr[i]; e < mx.row_ptr[i + 1]; ++e) {
      rs[i] += mx.val[e];
      cs[mx.col[e]] += mx.val[e];
    }
  for (int i = 0; i < K; ++i)
    if (std::fabs(rs[i] - 1.0) > 1e-5 || std::fabs(cs[i] - 1.0) > 1e-5) {
      *err = "mixing matrix is not doubly stochastic: row/column " + std::to_string(i) +
             " sums to " + std::to_string(rs[i]) + " / " + std::to_string(cs[i]);
      return false;
    }
  return true;
}

// Simple connected d-regular graph by the configuration model with rejection; attempt a shuffles
// the stubs with rng(seed, kGraph, a, s).  Edges come back sorted by (min, max).
bool random_regular(uint64_t seed, int K, int d, std::vector<std::pair<int, int>> *edges, int *attempts) {
  const int S = K * d;
  std::vector<int> stubs(S);
  for (int a = 0; a < 100000; ++a) {
    for (int v = 0, s = 0; v < K; ++v)
      for (int r = 0; r < d; ++r) stubs[s++] = v;
    for (int s = S - 1; s >= 1; --s) {
      int r = (int)(rng(seed, kGraph, (uint64_t)a, (uint64_t)s) % (uint64_t)(s + 1));
      std::swap(stubs[s], stubs[r]);
    }
    std::set<std::pair<int, int>> es;
    bool ok = true;
    for (int e = 0; e < S && ok; e += 2) {
      int u = stubs[e], v = stubs[e + 1];
      if (u == v) { ok = false; break; }
      std::pair<int, int> key(std::min(u, v), std::max(u, v));
      if (!es.insert(key).second) ok = false;
    }
    if (!ok) continue;
    std::vector<std::vector<int>> adj(K);
    for (auto &e : es) { adj[e.first].push_back(e.second); adj[e.second].push_back(e.first); }
    std::vector<char> seen(K, 0);
    std::vector<int> stack(1, 0);
    seen[0] = 1;
    int n_seen = 1;
    while (!stack.empty()) {
      int u = stack.back();
      stack.pop_back();
      for (int v : adj[u])
        if (!seen[v]) { seen[v] = 1; ++n_seen; stack.push_back(v); }
    }
    if (n_seen != K) continue;
    edges->assign(es.begin(), es.end());
    *attempts = a + 1;
    return true;
  }
  return false;
}

// Edges in (min, max) order; each takes the smallest colour free at both endpoints.
int greedy_matchings(const std::vector<std::pair<int, int>> &edges, int K, std::vector<int32_t> *partner) {
  std::vector<uint64_t> used(K, 0);
  int n_col = 0;
  partner->clear();
  for (auto &e : edges) {
    int c = 0;
    while (((used[e.first] | used[e.second]) >> c) & 1ull) ++c;
    if (c >= 63) return -1;
    if (c >= n_col) { n_col = c + 1; partner->resize((size_t)n_col * K, -1); }
    (*partner)[(size_t)c * K + e.first] = e.second;
    (*partner)[(size_t)c * K + e.second] = e.first;
    used[e.first] |= 1ull << c;
    used[e.second] |= 1ull << c;
  }
  return n_col;
}

bool check_partner_table(const int32_t *partner, int n, int K, std::string *err) {
  std::set<std::pair<int, int>> seen;
  for (int c = 0; c < n; ++c)
    for (int u = 0; u < K; ++u) {
      int v = partner[(size_t)c * K + u];
      if (v == -1) continue;
      if (v < 0 || v >= K || v == u || partner[(size_t)c * K + v] != u) {
        *err = "matching " + std::to_string(c) + " is not an involution at vertex " + std::to_string(u);
        return false;
      }
      if (u < v && !seen.insert({u, v}).second) {
        *err = "edge (" + std::to_string(u) + "," + std::to_string(v) + ") appears in two matchings";
        return false;
      }
    }
  return true;
}

}  // namespace

int build_mixing(const nb_topology *topo, int variant, int K, Mixing *out, std::string *err) {
  if (K < 1) { *err = "K must be >= 1"; return NB_ERR_ARG; }
  if (K > NB_MAX_K) { *err = "K exceeds NB_MAX_K"; return NB_ERR_UNSUPPORTED; }
  Mixing mx;
  mx.variant = variant;
  mx.K = K;
  if (variant == NB_ALLREDUCE || variant == NB_CENTRALIZED) {
    if (topo && topo->kind != NB_TOPO_FULL) { *err = "this variant takes the FULL topology (or none)"; return NB_ERR_ARG; }
    *out = mx;
    return NB_OK;
  }
  if (!topo) { *err = "topology required for this variant"; return NB_ERR_ARG; }
  if (variant == NB_DPSGD) {
    mx.row_ptr.assign(K + 1, 0);
    if (topo->kind == NB_TOPO_RING || topo->kind == NB_TOPO_FULL) {
      std::vector<float> W((size_t)K * K, 0.f);
      if (topo->kind == NB_TOPO_RING) {
        const float w = 1.0f / 3.0f;
        for (int i = 0; i < K; ++i) {
          W[(size_t)i * K + i] += w;
          W[(size_t)i * K + (i + 1) % K] += w;
          W[(size_t)i * K + (i + K - 1) % K] += w;
        }
      } else {
        for (auto &w : W) w = 1.0f / (float)K;
      }
      for (int i = 0; i < K; ++i) {
        for (int j = 0; j < K; ++j)
          if (W[(size_t)i * K + j] != 0.f) { mx.col.push_back(j); mx.val.push_back(W[(size_t)i * K + j]); }
        mx.row_ptr[i + 1] = (int32_t)mx.col.size();
      }
    } else if (topo->kind == NB_TOPO_CSR) {
      if (!topo->row_ptr || !topo->col_idx || !topo->val) { *err = "CSR arrays missing"; return NB_ERR_ARG; }
      if (topo->row_ptr[0] != 0) { *err = "row_ptr[0] must be 0"; return NB_ERR_ARG; }
      for (int i = 0; i < K; ++i) {
        if (topo->row_ptr[i + 1] < topo->row_ptr[i]) { *err = "row_ptr must be non-decreasing"; return NB_ERR_ARG; }
        // sort each row by column so the summation order is ascending j
        std::vector<std::pair<int32_t, float>> row;
        for (int e = topo->row_ptr[i]; e < topo->row_ptr[i + 1]; ++e) {
          int32_t j = topo->col_idx[e];
          if (j < 0 || j >= K) { *err = "col_idx out of range"; return NB_ERR_ARG; }
          row.push_back({j, topo->val[e]});
        }
        std::sort(row.begin(), row.end(), [](auto &a, auto &b) { return a.first < b.first; });
        for (size_t e = 0; e < row.size(); ++e) {
          if (e && row[e].first == row[e - 1].first) { *err = "duplicate column in a CSR row"; return NB_ERR_ARG; }
          mx.col.push_back(row[e].first);
          mx.val.push_back(row[e].second);
        }
        mx.row_ptr[i + 1] = (int32_t)mx.col.size();
      }
    } else {
      *err = "NB_DPSGD takes the RING, FULL or CSR topology";
      return NB_ERR_ARG;
    }
    if (mx.col.size() > NB_MAX_NNZ) { *err = "mixing matrix has more than NB_MAX_NNZ non-zeros"; return NB_ERR_UNSUPPORTED; }
    if (!check_doubly_stochastic(mx, err)) return NB_ERR_ARG;
    *out = mx;
    return NB_OK;
  }
  if (variant == NB_MATCHA) {
    if (topo->kind == NB_TOPO_MATCHINGS) {
      if (topo->n_matchings < 0 || (topo->n_matchings > 0 && !topo->partner)) { *err = "partner table missing"; return NB_ERR_ARG; }
      if (topo->n_matchings > NB_MAX_MATCHINGS) { *err = "more than NB_MAX_MATCHINGS matchings"; return NB_ERR_UNSUPPORTED; }
      if (!check_partner_table(topo->partner, topo->n_matchings, K, err)) return NB_ERR_ARG;
      mx.n_matchings = topo->n_matchings;
      mx.partner.assign(topo->partner, topo->partner + (size_t)topo->n_matchings * K);
      mx.attempts = 0;
    } else if (topo->kind == NB_TOPO_RANDOM_REGULAR) {
      const int d = topo->degree;
      if (d < 1 || d >= K || ((K * d) & 1)) { *err = "no simple regular graph with this K and degree"; return NB_ERR_ARG; }
      std::vector<std::pair<int, int>> edges;
      if (!random_regular(topo->seed, K, d, &edges, &mx.attempts)) { *err = "random regular graph: no draw accepted"; return NB_ERR_ARG; }
      int n = greedy_matchings(edges, K, &mx.partner);
      if (n < 0 || n > NB_MAX_MATCHINGS) { *err = "more than NB_MAX_MATCHINGS matchings"; return NB_ERR_UNSUPPORTED; }
      mx.n_matchings = n;
    } else {
      *err = "NB_MATCHA takes the MATCHINGS or RANDOM_REGULAR topology";
      return NB_ERR_ARG;
    }
    mx.probs.assign(mx.n_matchings, topo->act_prob);
    if (topo->act_probs)
      for (int c = 0; c < mx.n_matchings; ++c) mx.probs[c] = topo->act_probs[c];
    else if (!(topo->act_prob >= 0.f && topo->act_prob <= 1.f)) { *err = "act_prob must be in [0,1]"; return NB_ERR_ARG; }
    mx.thr.resize(mx.n_matchings);
    for (int c = 0; c < mx.n_matchings; ++c) {
      if (!(mx.probs[c] >= 0.f && mx.probs[c] <= 1.f)) { *err = "activation probabilities must be in [0,1]"; return NB_ERR_ARG; }
      mx.thr[c] = activation_threshold(mx.probs[c]);
    }
    // rows and columns of W = I - alpha * sum_active L_j sum to one for every alpha; alpha <= 1 keeps
    // every I - alpha * L_j a contraction (a vertex whose active degree exceeds 1/alpha gets a
    // negative diagonal weight, which MATCHA's optimal step sizes do produce)
    if (!(topo->alpha >= 0.f && topo->alpha <= 1.0f)) { *err = "alpha must be in [0, 1]"; return NB_ERR_ARG; }
    if ((size_t)K * (size_t)(1 + mx.n_matchings) > NB_MAX_NNZ) { *err = "K*(1+matchings) exceeds NB_MAX_NNZ"; return NB_ERR_UNSUPPORTED; }
    mx.alpha = topo->alpha;
    mx.seed = topo->seed;
    *out = mx;
    return NB_OK;
  }
  *err = "unknown variant";
  return NB_ERR_ARG;
}

void dense_W(const Mixing &mx, int64_t step, float *W, uint32_t *bits) {
  const int K = mx.K;
  std::fill(W, W + (size_t)K * K, 0.f);
  uint32_t b = 0;
  if (mx.variant == NB_ALLREDUCE || mx.variant == NB_CENTRALIZED) {
    for (size_t e = 0; e < (size_t)K * K; ++e) W[e] = 1.0f / (float)K;
  } else if (mx.variant == NB_DPSGD) {
    for (int i = 0; i < K; ++i)
      for (int e = mx.row_ptr[i]; e < mx.row_ptr[i + 1]; ++e) W[(size_t)i * K + mx.col[e]] = mx.val[e];
  } else {
    b = matcha_bits(mx.seed, step, mx.n_matchings, mx.thr.data());
    for (int i = 0; i < K; ++i) {
      int cnt = 0;
      for (int c = 0; c < mx.n_matchings; ++c) {
        int v = mx.partner[(size_t)c * K + i];
        if (((b >> c) & 1u) && v >= 0) { W[(size_t)i * K + v] = mx.alpha; ++cnt; }
      }
      W[(size_t)i * K + i] = 1.0f - mx.alpha * (float)cnt;
    }
  }
  if (bits) *bits = b;
}

}  // namespace nb

namespace nb {
namespace {

// Cyclic Jacobi eigenvalue iteration for a symmetric n x n matrix (row-major, destroyed).
// Eigenvalues ascending in w, matching unit eigenvectors in the columns of V.
void jacobi_eigh(std::vector<double> &A, int n, std::vector<double> &w, std::vector<double> &V) {
  V.assign((size_t)n * n, 0.0);
  for (int i = 0; i < n; ++i) V[(size_t)i * n + i] = 1.0;
  for (int sweep = 0; sweep < 60; ++sweep) {
    double off = 0.0;
    for (int p = 0; p < n; ++p)
      for (int q = p + 1; q < n; ++q) off += A[(size_t)p * n + q] * A[(size_t)p * n + q];
    if (off < 1e-26) break;
    for (int p = 0; p < n; ++p)
      for (int q = p + 1; q < n; ++q) {
        const double apq = A[(size_t)p * n + q];
        if (std::fabs(apq) < 1e-300) continue;
        const double theta = (A[(size_t)q * n + q] - A[(size_t)p * n + p]) / (2.0 * apq);
        const double t = (theta >= 0 ? 1.0 : -1.0) / (std::fabs(theta) + std::sqrt(theta * theta + 1.0));
        const double c = 1.0 / std::sqrt(t * t + 1.0), sn = t * c;
        for (int k = 0; k < n; ++k) {  // columns p, q
          const double akp = A[(size_t)k * n + p], akq = A[(size_t)k * n + q];
          A[(size_t)k * n + p] = c * akp - sn * akq;
          A[(size_t)k * n + q] = sn * akp + c * akq;
        }
        for (int k = 0; k < n; ++k) {  // rows p, q
          const double apk = A[(size_t)p * n + k], aqk = A[(size_t)q * n + k];
          A[(size_t)p * n + k] = c * apk - sn * aqk;
          A[(size_t)q * n + k] = sn * apk + c * aqk;
        }
        for (int k = 0; k < n; ++k) {
          const double vkp = V[(size_t)k * n + p], vkq = V[(size_t)k * n + q];
          V[(size_t)k * n + p] = c * vkp - sn * vkq;
          V[(size_t)k * n + q] = sn * vkp + c * vkq;
        }
      }
  }
  std::vector<int> idx(n);
  for (int i = 0; i < n; ++i) idx[i] = i;
  std::sort(idx.begin(), idx.end(), [&](int a, int b) { return A[(size_t)a * n + a] < A[(size_t)b * n + b]; });
  w.resize(n);
  std::vector<double> Vs((size_t)n * n);
  for (int j = 0; j < n; ++j) {
    w[j] = A[(size_t)idx[j] * n + idx[j]];
    for (int k = 0; k < n; ++k) Vs[(size_t)k * n + j] = V[(size_t)k * n + idx[j]];
  }
  V.swap(Vs);
}

// sum_j p_j L_j for the matchings in `partner`
void expected_laplacian(const std::vector<int32_t> &partner, int m, int K, const std::vector<double> &p,
                        std::vector<double> &L) {
  L.assign((size_t)K * K, 0.0);
  for (int c = 0; c < m; ++c)
    for (int u = 0; u < K; ++u) {
      const int v = partner[(size_t)c * K + u];
      if (v > u) {
        L[(size_t)u * K + u] += p[c];
        L[(size_t)v * K + v] += p[c];
        L[(size_t)u * K + v] -= p[c];
        L[(size_t)v * K + u] -= p[c];
      }
    }
}

// Euclidean projection onto {0 <= p_j <= 1, sum p_j <= total}
void project_budget(std::vector<double> &p, double total) {
  std::vector<double> raw = p;
  double sum = 0.0, pmax = 0.0;
  for (auto &x : p) { x = std::min(1.0, std::max(0.0, x)); sum += x; }
  if (sum <= total) return;
  for (double x : raw) pmax = std::max(pmax, x);
  double lo = 0.0, hi = pmax;
  for (int it = 0; it < 100; ++it) {
    const double mid = 0.5 * (lo + hi);
    double sm = 0.0;
    for (double x : raw) sm += std::min(1.0, std::max(0.0, x - mid));
    if (sm > total) lo = mid; else hi = mid;
  }
  for (size_t j = 0; j < p.size(); ++j) p[j] = std::min(1.0, std::max(0.0, raw[j] - hi));
}

double lambda2_of(const std::vector<int32_t> &partner, int m, int K, const std::vector<double> &p,
                  std::vector<double> *fiedler) {
  std::vector<double> L, w, V;
  expected_laplacian(partner, m, K, p, L);
  jacobi_eigh(L, K, w, V);
  if (K < 2) return 0.0;
  if (fiedler) {
    fiedler->resize(K);
    for (int k = 0; k < K; ++k) (*fiedler)[k] = V[(size_t)k * K + 1];
  }
  return w[1];
}

// || E[W^T W] - J ||_2 with E[W^T W] = I - 2a L_bar + a^2 (L_bar^2 + 2 sum_j p_j (1 - p_j) L_j)
double rho_of(const std::vector<int32_t> &partner, int m, int K, const std::vector<double> &p, double a) {
  std::vector<double> Lb, Lt, pt(m);
  for (int c = 0; c < m; ++c) pt[c] = p[c] * (1.0 - p[c]);
  expected_laplacian(partner, m, K, p, Lb);
  expected_laplacian(partner, m, K, pt, Lt);
  std::vector<double> A((size_t)K * K);
  for (int i = 0; i < K; ++i)
    for (int j = 0; j < K; ++j) {
      double l2 = 0.0;
      for (int k = 0; k < K; ++k) l2 += Lb[(size_t)i * K + k] * Lb[(size_t)k * K + j];
      A[(size_t)i * K + j] = (i == j ? 1.0 : 0.0) - 2.0 * a * Lb[(size_t)i * K + j] +
                             a * a * (l2 + 2.0 * Lt[(size_t)i * K + j]) - 1.0 / (double)K;
    }
  std::vector<double> w, V;
  jacobi_eigh(A, K, w, V);
  return std::max(std::fabs(w[0]), std::fabs(w[K - 1]));
}

}  // namespace
}  // namespace nb

extern "C" int nb_matcha_optimize(const nb_topology *topo, int K, float budget, int iters, float *probs, float *alpha,
                                  float *lambda2, float *rho) {
  using namespace nb;
  if (!topo || !(budget > 0.f && budget <= 1.f) || iters < 0) return NB_ERR_ARG;
  Mixing mx;
  std::string err;
  nb_topology t = *topo;
  t.alpha = 0.f;
  t.act_prob = 0.f;
  t.act_probs = nullptr;
  int st = build_mixing(&t, NB_MATCHA, K, &mx, &err);
  if (st != NB_OK) return st;
  const int m = mx.n_matchings;
  if (m < 1 || K < 2) return NB_ERR_ARG;
  if (iters == 0) iters = 1000;
  const double total = (double)budget * m;
  std::vector<double> p(m, (double)budget), best_p, fied, g(m);
  project_budget(p, total);
  best_p = p;
  double best = lambda2_of(mx.partner, m, K, p, &fied);
  for (int it = 1; it <= iters; ++it) {
    double nrm = 0.0;
    for (int c = 0; c < m; ++c) {  // supergradient g_c = v^T L_c v = sum over the matching's edges of (v_u - v_w)^2
      double s = 0.0;
      for (int u = 0; u < K; ++u) {
        const int v = mx.partner[(size_t)c * K + u];
        if (v > u) s += (fied[u] - fied[v]) * (fied[u] - fied[v]);
      }
      g[c] = s;
      nrm += s * s;
    }
    nrm = std::sqrt(nrm);
    if (nrm == 0.0) break;
    const double step = 0.5 / std::sqrt((double)it);
    for (int c = 0; c < m; ++c) p[c] += step * g[c] / nrm;
    project_budget(p, total);
    const double val = lambda2_of(mx.partner, m, K, p, &fied);
    if (val > best) { best = val; best_p = p; }
  }
  // the library consumes fp32 probabilities: evaluate alpha and rho at the rounded values
  std::vector<double> pf(m);
  for (int c = 0; c < m; ++c) pf[c] = (double)(float)best_p[c];
  double lo = 0.0, hi = 1.0;
  const double gr = (std::sqrt(5.0) - 1.0) / 2.0;
  double c1 = hi - gr * (hi - lo), d1 = lo + gr * (hi - lo);
  double fc = rho_of(mx.partner, m, K, pf, c1), fd = rho_of(mx.partner, m, K, pf, d1);
  for (int it = 0; it < 80; ++it) {
    if (fc < fd) { hi = d1; d1 = c1; fd = fc; c1 = hi - gr * (hi - lo); fc = rho_of(mx.partner, m, K, pf, c1); }
    else { lo = c1; c1 = d1; fc = fd; d1 = lo + gr * (hi - lo); fd = rho_of(mx.partner, m, K, pf, d1); }
  }
  const float a = (float)(0.5 * (lo + hi));
  if (probs) for (int c = 0; c < m; ++c) probs[c] = (float)best_p[c];
  if (alpha) *alpha = a;
  if (lambda2) *lambda2 = (float)lambda2_of(mx.partner, m, K, pf, nullptr);
  if (rho) *rho = (float)rho_of(mx.partner, m, K, pf, (double)a);
  return NB_OK;
}

// -------------------------------------------------------------------------------------------------
// C ABI: host-only entry points
// -------------------------------------------------------------------------------------------------
extern "C" int nb_straggler_sample(const nb_straggler *cfg, int K, int M, int64_t step, int32_t *finished,
                                   uint8_t *mask, double *tau_out) {
  using namespace nb;
  if (!cfg || !finished || K < 1 || K > NB_MAX_K || M < 1 || step < 0) return NB_ERR_ARG;
  double tau[NB_MAX_K];
  if (cfg->model == NB_STRAG_UNIFORM_COUNT) {
    for (int i = 0; i < K; ++i) {
      finished[i] = 1 + (int32_t)(rng(cfg->seed, kStraggler, (uint64_t)step, (uint64_t)i) % (uint64_t)M);
      tau[i] = 0.0;
    }
  } else if (cfg->model == NB_STRAG_SHIFTED_EXP || cfg->model == NB_STRAG_SHIFTED_EXP_SLOWSET) {
    double delta[NB_MAX_K];
    if (cfg->model == NB_STRAG_SHIFTED_EXP) {
      if (!(cfg->params[0] >= 0.0)) return NB_ERR_ARG;
      for (int i = 0; i < K; ++i) delta[i] = cfg->params[0];
    } else {
      const double frac = cfg->params[0];
      if (!(frac >= 0.0 && frac <= 1.0) || !(cfg->params[1] >= 0.0) || !(cfg->params[2] >= 0.0)) return NB_ERR_ARG;
      const int n_slow = (int)std::floor(frac * (double)K);
      int idx[NB_MAX_K];
      for (int i = 0; i < K; ++i) { idx[i] = i; delta[i] = cfg->params[2]; }
      for (int q = 0; q < n_slow; ++q) {  // partial Fisher-Yates: the slow set is re-drawn every step
        int r = (int)(rng(cfg->seed, kSlowSet, (uint64_t)step, (uint64_t)q) % (uint64_t)(K - q));
        std::swap(idx[q], idx[q + r]);
        delta[idx[q]] = cfg->params[1];
      }
    }
    double tmin = 0.0;
    for (int i = 0; i < K; ++i) {
      const double u = uniform01(rng(cfg->seed, kStraggler, (uint64_t)step, (uint64_t)i));
      tau[i] = 1.0 + (-(delta[i]) * std::log(u));
      if (i == 0 || tau[i] < tmin) tmin = tau[i];
    }
    const double T = (double)M * tmin;  // the fastest learner finishes its batch and ends the iteration
    for (int i = 0; i < K; ++i) {
      int c = 0;
      for (int j = 1; j <= M; ++j)
        if ((double)j * tau[i] <= T) ++c;
      finished[i] = c < 1 ? 1 : c;
    }
  } else {
    return NB_ERR_ARG;
  }
  if (mask)
    for (int i = 0; i < K; ++i)
      for (int m = 0; m < M; ++m) mask[(size_t)i * M + m] = (uint8_t)(m < finished[i]);
  if (tau_out) std::memcpy(tau_out, tau, sizeof(double) * K);
  return NB_OK;
}

extern "C" int nb_topology_matchings(const nb_topology *topo, int K, int32_t *partner, int32_t *n_matchings,
                                     int32_t *attempts) {
  if (!topo || !partner || !n_matchings) return NB_ERR_ARG;
  nb::Mixing mx;
  std::string err;
  nb_topology t = *topo;
  if (t.kind == NB_TOPO_RANDOM_REGULAR || t.kind == NB_TOPO_MATCHINGS) {
    // alpha / activation probabilities do not matter for the decomposition itself
    t.alpha = 0.f;
    t.act_prob = 0.f;
    t.act_probs = nullptr;
  }
  int st = nb::build_mixing(&t, NB_MATCHA, K, &mx, &err);
  if (st != NB_OK) return st;
  *n_matchings = mx.n_matchings;
  std::copy(mx.partner.begin(), mx.partner.end(), partner);
  if (attempts) *attempts = mx.attempts;
  return NB_OK;
}

extern "C" int nb_mixing_matrix(const nb_topology *topo, int variant, int K, int64_t step, float *W_dense,
                                uint32_t *bits) {
  if (!W_dense || step < 0) return NB_ERR_ARG;
  nb::Mixing mx;
  std::string err;
  int st = nb::build_mixing(topo, variant, K, &mx, &err);
  if (st != NB_OK) return st;
  nb::dense_W(mx, step, W_dense, bits);
  return NB_OK;
}

extern "C" int nb_runtime_report_compute(const nb_straggler *cfg, int K, int M, int64_t step0, int64_t steps,
                                         nb_runtime_report *out) {
  if (!cfg || !out || K < 1 || K > NB_MAX_K || M < 1 || step0 < 0 || steps < 1) return NB_ERR_ARG;
  if (cfg->model == NB_STRAG_UNIFORM_COUNT) return NB_ERR_UNSUPPORTED;
  double tau[NB_MAX_K];
  int32_t n[NB_MAX_K];
  double s_nb = 0, s_bl = 0, s_thr = 0, s_frac = 0, s_fin = 0, s_min = 0, s_max = 0;
  for (int64_t t = step0; t < step0 + steps; ++t) {
    int rc = nb_straggler_sample(cfg, K, M, t, n, nullptr, tau);
    if (rc != NB_OK) return rc;
    double tmin = tau[0], tmax = tau[0], Y = 0.0;
    int64_t fin = 0;
    for (int i = 0; i < K; ++i) {
      if (tau[i] < tmin) tmin = tau[i];
      if (tau[i] > tmax) tmax = tau[i];
      Y += 1.0 / tau[i];
      fin += n[i];
    }
    s_min += tmin;
    s_max += tmax;
    s_nb += (double)M * tmin;
    s_bl += (double)M * tmax;
    s_thr += Y * tmax / (double)K;
    s_frac += Y * tmin / (double)K;
    s_fin += (double)fin / ((double)K * (double)M);
  }
  const double inv = 1.0 / (double)steps;
  out->mean_t_nonblocking = s_nb * inv;
  out->mean_t_blocking = s_bl * inv;
  out->ratio = s_nb / s_bl;
  out->mean_throughput_ratio = s_thr * inv;
  out->mean_fractional_data = s_frac * inv;
  out->mean_finished_fraction = s_fin * inv;
  out->mean_min_tau = s_min * inv;
  out->mean_max_tau = s_max * inv;
  out->steps = steps;
  return NB_OK;
}
