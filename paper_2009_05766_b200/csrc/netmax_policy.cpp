// Host control plane of the NetMax simulator: the iteration-time model (Section II-B) and
// the communication-policy generator (Algorithm 3 with Eq. 8-14 and Eq. 22).
//
// Readings where the paper is silent or garbled:
//   * the grids are rho_k = k U_rho / K and t_bar_r = U - (R - r)(U - L)/R;
//   * U_rho = min(0.5/alpha, (1 - 1e-6) / (alpha max_i sum_{m != i}(d_im + d_mi))), because
//     beyond it the floors of Eq. 11 alone exceed a row sum of one;
//   * L = max_i (alpha rho / M) sum_{m != i} t_im (d_im + d_mi)   (Eq. 25-26);
//   * d_ii = 1 for selectability and t_ii = C_i; Eq. 11 is taken closed;
//   * the LP (Eq. 14) decouples by row and its optimum is not unique: when p_ii = 0 is
//     feasible the row is floor + (1 - sum floors) * q with q_m ~ exp(-eta t_im) matched to
//     the required mean time (the maximum-entropy optimum); otherwise p_ii is the least
//     value that meets the time constraint and the remainder goes to the fastest peer(s);
//   * with every row meeting Eq. 10, p_i = 1/M (Lemma 1), which Y_P uses directly;
//   * eps = 1e-3; infeasible grid points are skipped; ties keep the earlier grid point.
//
// The same search for pull rules with a constant weight w (the section on extending existing
// decentralised PSGD approaches), netmax_policy_generate_fixed_weight:
//   * E[D^T D] for D = I + w e_i (e_m - e_i)^T has y_im = (w - w^2)(p_i p_im + p_m p_mi), so the
//     replacement of Eq. 11 ("every y_im on a link is positive") reads p_im + p_mi > 0; it is taken
//     closed with a floor phi on both directions of every link, and phi takes rho's place in the
//     outer loop (phi_k = k U_phi / K, U_phi where the floors alone fill a row);
//   * Y_P is doubly stochastic only if, besides Eq. 10 (p_i = 1/M), the columns of P sum to 1
//     (row sums of Y_P are 1 + w (sum_m p_m p_mi - p_i sum_m p_im)): an added constraint that couples
//     the rows of the LP;
//   * the optimum is again not unique; the reading is p_ii = 0 and the maximum-entropy P above the
//     floors, p_im = phi + A_i B_m exp(-eta_i t_im), found by alternating scalings: rows (A_i and
//     eta_i from the row's sum and mean time), then columns (B_m from the column sums); the inner
//     grid takes the midpoints of R cells of [L, U].
#include "../../include/netmax.h"

#include <algorithm>
#include <cmath>
#include <cstdio>
#include <functional>
#include <thread>
#include <vector>

#include "netmax_policy.h"

namespace {

constexpr double kEtaCap = 600.0;
constexpr double kTie = 1e-12;
constexpr double kEps = 1e-3;

int fail(int code, const std::string& msg) {
  netmax::set_global_error(msg);
  return code;
}

void parallel_for(int n, int min_parallel, const std::function<void(int, int)>& body) {
  unsigned hw = std::thread::hardware_concurrency();
  int threads = (n >= min_parallel && hw > 1) ? (int)std::min<unsigned>(hw, 16) : 1;
  if (threads <= 1) { body(0, n); return; }
  std::vector<std::thread> pool;
  const int per = (n + threads - 1) / threads;
  for (int t = 0; t < threads; ++t) {
    const int a = std::min(n, t * per), b = std::min(n, a + per);
    if (a < b) pool.emplace_back(body, a, b);
  }
  for (auto& th : pool) th.join();
}

struct Row {
  std::vector<int> nb;        // neighbours m != i
  std::vector<double> t, f1;  // their iteration times and d_im + d_mi
  double C = 0, tmin = 0, tmax = 0, sum_f1 = 0, sum_f1t = 0;
};

// Exponential tilt: q_m ~ exp(-eta s_m), s in [0,1], with mean s equal to sig.  The mean is
// decreasing in eta; Newton steps are kept inside a shrinking bracket.
bool tilt(const std::vector<double>& s, double sig, std::vector<double>& q) {
  const size_t n = s.size();
  q.resize(n);
  auto stats = [&](double eta, double& mean, double& var) {
    double z = 0, a = 0, b = 0;
    for (size_t j = 0; j < n; ++j) {
      const double w = std::exp(-eta * s[j]);
      q[j] = w;
      z += w;
      a += w * s[j];
      b += w * s[j] * s[j];
    }
    mean = a / z;
    var = b / z - mean * mean;
    for (size_t j = 0; j < n; ++j) q[j] /= z;
  };
  double mean, var;
  double lo = -kEtaCap, hi = kEtaCap, eta = 0.0;
  stats(lo, mean, var);
  if (sig >= mean) {
    eta = lo;
  } else {
    stats(hi, mean, var);
    if (sig <= mean) {
      eta = hi;
    } else {
      stats(eta, mean, var);
      for (int it = 0; it < 200; ++it) {
        const double gap = mean - sig;
        if (std::fabs(gap) <= 1e-15) break;
        if (gap > 0) lo = eta; else hi = eta;
        double next = (var > 1e-300) ? eta + gap / var : 0.5 * (lo + hi);
        if (!(next > lo && next < hi)) next = 0.5 * (lo + hi);
        if (next == eta || hi - lo <= 1e-15 * (1.0 + std::fabs(eta))) break;
        eta = next;
        stats(eta, mean, var);
      }
    }
  }
  stats(eta, mean, var);
  return std::fabs(mean - sig) <= 1e-9;
}

// One row of the LP at (rho, T = M t_bar).  Returns false when the row is infeasible.
bool solve_row(const Row& row, int i, int M, double ar /* alpha rho */, double T, double* out) {
  const size_t n = row.nb.size();
  const double F = ar * row.sum_f1;
  if (F > 1.0) return false;
  const double free_mass = 1.0 - F;
  const double A = ar * row.sum_f1t;
  const double lo = A + free_mass * row.tmin, hi = A + free_mass * row.tmax;
  std::fill(out, out + M, 0.0);
  if (T > hi * (1.0 + kTie)) return false;
  if (T >= lo * (1.0 - kTie)) {
    if (free_mass <= 0.0) {
      for (size_t j = 0; j < n; ++j) out[row.nb[j]] = ar * row.f1[j];
      return true;
    }
    const double target = std::min(std::max((T - A) / free_mass, row.tmin), row.tmax);
    const double scale = row.tmax - row.tmin;
    std::vector<double> q(n, 1.0 / (double)n);
    if (scale > kTie * row.tmax) {
      std::vector<double> s(n);
      for (size_t j = 0; j < n; ++j) s[j] = (row.t[j] - row.tmin) / scale;
      if (!tilt(s, (target - row.tmin) / scale, q)) return false;
    }
    for (size_t j = 0; j < n; ++j) out[row.nb[j]] = ar * row.f1[j] + free_mass * q[j];
    return true;
  }
  double pii = (lo - T) / (row.tmin - row.C);
  if (pii > free_mass * (1.0 + kTie)) return false;
  pii = std::min(pii, free_mass);
  int fastest = 0;
  for (size_t j = 0; j < n; ++j) fastest += (row.t[j] <= row.tmin * (1.0 + kTie));
  for (size_t j = 0; j < n; ++j) {
    const bool fast = row.t[j] <= row.tmin * (1.0 + kTie);
    out[row.nb[j]] = ar * row.f1[j] + (fast ? (free_mass - pii) / fastest : 0.0);
  }
  out[i] = pii;
  return true;
}

// Eigenvalues of a small dense symmetric matrix by cyclic Jacobi rotations (in place).
void jacobi_eigenvalues(std::vector<double>& a, int n, std::vector<double>& eig) {
  for (int sweep = 0; sweep < 60; ++sweep) {
    double off = 0.0, diag = 0.0;
    for (int p = 0; p < n; ++p) {
      diag += a[(size_t)p * n + p] * a[(size_t)p * n + p];
      for (int q = p + 1; q < n; ++q) off += a[(size_t)p * n + q] * a[(size_t)p * n + q];
    }
    if (off <= 1e-30 * (diag + 1e-300)) break;
    for (int p = 0; p < n - 1; ++p)
      for (int q = p + 1; q < n; ++q) {
        const double apq = a[(size_t)p * n + q];
        if (apq == 0.0) continue;
        const double theta = (a[(size_t)q * n + q] - a[(size_t)p * n + p]) / (2.0 * apq);
        const double t = (theta >= 0 ? 1.0 : -1.0) / (std::fabs(theta) + std::sqrt(theta * theta + 1.0));
        const double c = 1.0 / std::sqrt(t * t + 1.0), s = t * c;
        for (int k = 0; k < n; ++k) {  // columns p, q
          const double akp = a[(size_t)k * n + p], akq = a[(size_t)k * n + q];
          a[(size_t)k * n + p] = c * akp - s * akq;
          a[(size_t)k * n + q] = s * akp + c * akq;
        }
        for (int k = 0; k < n; ++k) {  // rows p, q
          const double apk = a[(size_t)p * n + k], aqk = a[(size_t)q * n + k];
          a[(size_t)p * n + k] = c * apk - s * aqk;
          a[(size_t)q * n + k] = s * apk + c * aqk;
        }
      }
  }
  eig.resize(n);
  for (int p = 0; p < n; ++p) eig[p] = a[(size_t)p * n + p];
  std::sort(eig.begin(), eig.end());
}

// Second largest eigenvalue of the symmetric doubly stochastic Y: the largest eigenvalue of
// Y restricted to the complement of the all-ones vector.  Dense Jacobi for small M; Lanczos
// with full reorthogonalisation (Ritz values by Jacobi) otherwise.
double second_eigenvalue(const std::vector<double>& Y, int M) {
  if (M <= 96) {
    std::vector<double> a(Y), eig;
    jacobi_eigenvalues(a, M, eig);
    return eig[M - 2];
  }
  auto matvec = [&](const std::vector<double>& v, std::vector<double>& out) {
    double mean = 0.0;
    for (int j = 0; j < M; ++j) mean += v[j];
    mean /= M;
    parallel_for(M, 512, [&](int a, int b) {
      for (int i = a; i < b; ++i) {
        const double* row = Y.data() + (size_t)i * M;
        double acc = 0.0;
        for (int j = 0; j < M; ++j) acc += row[j] * v[j];
        out[i] = acc - mean;  // (Y - 11^T/M) v
      }
    });
  };
  const int max_steps = std::min(M - 1, 300);
  std::vector<std::vector<double>> V;
  std::vector<double> alpha, beta, v(M), wv(M);
  uint64_t lcg = 0x9E3779B97F4A7C15ull;
  double mean = 0.0;
  for (int j = 0; j < M; ++j) {
    lcg = lcg * 6364136223846793005ull + 1442695040888963407ull;
    v[j] = (double)(lcg >> 11) / 9007199254740992.0 - 0.5;
    mean += v[j];
  }
  mean /= M;
  double nrm = 0.0;
  for (int j = 0; j < M; ++j) { v[j] -= mean; nrm += v[j] * v[j]; }
  nrm = std::sqrt(nrm);
  for (int j = 0; j < M; ++j) v[j] /= nrm;
  double best = 0.0;
  for (int step = 0; step < max_steps; ++step) {
    V.push_back(v);
    matvec(v, wv);
    double a = 0.0;
    for (int j = 0; j < M; ++j) a += wv[j] * v[j];
    alpha.push_back(a);
    for (int pass = 0; pass < 2; ++pass)  // full reorthogonalisation, twice
      for (const auto& u : V) {
        double dot = 0.0;
        for (int j = 0; j < M; ++j) dot += wv[j] * u[j];
        for (int j = 0; j < M; ++j) wv[j] -= dot * u[j];
      }
    double b = 0.0;
    for (int j = 0; j < M; ++j) b += wv[j] * wv[j];
    b = std::sqrt(b);
    const int m = (int)alpha.size();
    if ((m % 10 == 0) || b < 1e-13 || step == max_steps - 1) {
      std::vector<double> Tm((size_t)m * m, 0.0), eig;
      for (int k = 0; k < m; ++k) {
        Tm[(size_t)k * m + k] = alpha[k];
        if (k + 1 < m) Tm[(size_t)k * m + k + 1] = Tm[(size_t)(k + 1) * m + k] = beta[k];
      }
      jacobi_eigenvalues(Tm, m, eig);
      const double top = eig[m - 1];
      const bool settled = std::fabs(top - best) <= 1e-13 * std::max(1.0, std::fabs(top));
      best = top;
      if (b < 1e-13 || (settled && m >= 20)) break;
    }
    beta.push_back(b);
    for (int j = 0; j < M; ++j) v[j] = wv[j] / b;
  }
  return best;
}

}  // namespace

namespace netmax {
// Largest eigenvalue of the symmetric tridiagonal matrix with diagonal alpha[0..m) and
// off-diagonal beta[0..m-1) (the Ritz values of a Lanczos run).
double tridiagonal_top_eigenvalue(const std::vector<double>& alpha, const std::vector<double>& beta) {
  const int m = (int)alpha.size();
  std::vector<double> Tm((size_t)m * m, 0.0), eig;
  for (int k = 0; k < m; ++k) {
    Tm[(size_t)k * m + k] = alpha[k];
    if (k + 1 < m) Tm[(size_t)k * m + k + 1] = Tm[(size_t)(k + 1) * m + k] = beta[k];
  }
  jacobi_eigenvalues(Tm, m, eig);
  return eig[m - 1];
}
}  // namespace netmax

extern "C" {

int netmax_iteration_times(int32_t M, int64_t d, const double* speed, double* t_out, uint8_t* adj_out) {
  if (M < 2 || d < 1 || !speed || !t_out || !adj_out) return fail(NETMAX_INVALID_ARG, "iteration_times: bad argument");
  double nmin = INFINITY;
  for (int i = 0; i < M; ++i)
    for (int m = 0; m < M; ++m) {
      const size_t at = (size_t)i * M + m;
      const double a = speed[at], b = speed[(size_t)m * M + i];
      if (!std::isfinite(a)) return fail(NETMAX_INVALID_ARG, "iteration_times: link speed is not finite");
      const bool link = (i != m) && a > 0.0 && b > 0.0;
      adj_out[at] = link ? 1 : 0;
      t_out[at] = link ? 32.0 * (double)d / (a * 1e9) : 0.0;   // N_im: a full fp32 replica over the link
      if (link) nmin = std::min(nmin, t_out[at]);
    }
  if (!std::isfinite(nmin)) return fail(NETMAX_NOT_CONNECTED, "iteration_times: no link has a positive speed");
  const double C = 0.25 * nmin;   // C_i: computation is the short part of an iteration
  for (int i = 0; i < M; ++i)
    for (int m = 0; m < M; ++m) {
      const size_t at = (size_t)i * M + m;
      if (i == m) t_out[at] = C;
      else if (adj_out[at]) t_out[at] = std::max(C, t_out[at]);   // t_im = max{C_i, N_im}
    }
  return NETMAX_OK;
}

int netmax_policy_generate(int32_t M, const double* t, const uint8_t* adj, double lr, int32_t K, int32_t R,
                           double* prob_out, double* rho_out, double* info_out) {
  return netmax_policy_generate_ex(M, t, adj, lr, K, R, 0.0, prob_out, rho_out, info_out);
}

int netmax_policy_generate_ex(int32_t M, const double* t, const uint8_t* adj, double lr, int32_t K, int32_t R,
                              double rho_upper, double* prob_out, double* rho_out, double* info_out) {
  if (M < 2 || !t || !adj || !prob_out || !rho_out || !(lr > 0.0) || K < 1 || R < 1)
    return fail(NETMAX_INVALID_ARG, "policy_generate: bad argument");
  std::vector<Row> rows(M);
  double max_f1 = 0.0, U_time = INFINITY;
  for (int i = 0; i < M; ++i) {
    Row& r = rows[i];
    r.C = t[(size_t)i * M + i];
    r.tmin = INFINITY;
    r.tmax = 0.0;
    for (int m = 0; m < M; ++m) {
      if (m == i || !adj[(size_t)i * M + m]) continue;
      const double tm = t[(size_t)i * M + m];
      if (!(tm > 0.0) || !std::isfinite(tm)) return fail(NETMAX_INVALID_ARG, "policy_generate: iteration time on a link is not positive");
      const double f1 = (double)adj[(size_t)i * M + m] + (double)adj[(size_t)m * M + i];
      r.nb.push_back(m);
      r.t.push_back(tm);
      r.f1.push_back(f1);
      r.sum_f1 += f1;
      r.sum_f1t += f1 * tm;
      r.tmin = std::min(r.tmin, tm);
      r.tmax = std::max(r.tmax, tm);
    }
    if (r.nb.empty()) return fail(NETMAX_NOT_CONNECTED, "policy_generate: a worker has no neighbour");
    if (!(r.C < r.tmin)) return fail(NETMAX_INVALID_ARG, "policy_generate: t_ii must be below every t_im");
    max_f1 = std::max(max_f1, r.sum_f1);
    U_time = std::min(U_time, r.tmax / M);
  }
  const double U_rho = rho_upper > 0.0 ? rho_upper : std::min(0.5 / lr, (1.0 - 1e-6) / (lr * max_f1));

  std::vector<double> P((size_t)M * M), Y((size_t)M * M), bestP;
  double best_tconv = INFINITY, best_rho = 0, best_lam = 0, best_tbar = 0;
  int best_k = 0, best_r = 0;
  for (int k = 1; k <= K; ++k) {
    const double rho = k * U_rho / K, ar = lr * rho;
    double L = 0.0;
    for (int i = 0; i < M; ++i) L = std::max(L, ar / M * rows[i].sum_f1t);
    if (!(U_time > L)) continue;
    const double delta = (U_time - L) / R;
    for (int r = 1; r <= R; ++r) {
      const double tbar = U_time - (R - r) * delta, T = M * tbar;
      std::vector<uint8_t> ok(M, 1);
      parallel_for(M, 256, [&](int a, int b) {
        for (int i = a; i < b; ++i) ok[i] = solve_row(rows[i], i, M, ar, T, P.data() + (size_t)i * M) ? 1 : 0;
      });
      if (std::find(ok.begin(), ok.end(), (uint8_t)0) != ok.end()) continue;
      // Y_P (Eq. 22) with p_i = 1/M: p_im gamma_im = (d_im+d_mi)/2, p_im gamma_im^2 = (d_im+d_mi)^2/(4 p_im)
      parallel_for(M, 256, [&](int a, int b) {
        for (int i = a; i < b; ++i) {
          double rowsum = 0.0;
          for (int m = 0; m < M; ++m) {
            if (m == i) continue;
            const double pim = P[(size_t)i * M + m], pmi = P[(size_t)m * M + i];
            const double ds = (double)adj[(size_t)i * M + m] + (double)adj[(size_t)m * M + i];
            double lin = 0.0, quad = 0.0;
            if (pim > 0.0) { lin += 0.5 * ds; quad += ds * ds / (4.0 * pim); }
            if (pmi > 0.0) { lin += 0.5 * ds; quad += ds * ds / (4.0 * pmi); }
            const double y = (ar * lin - ar * ar * quad) / M;
            Y[(size_t)i * M + m] = y;
            rowsum += y;
          }
          Y[(size_t)i * M + i] = 1.0 - rowsum;
        }
      });
      const double lam2 = second_eigenvalue(Y, M);
      if (!(lam2 > 0.0 && lam2 < 1.0)) continue;
      const double tconv = tbar * std::log(kEps) / std::log(lam2);
      if (bestP.empty() || tconv < best_tconv * (1.0 - 1e-12)) {
        bestP = P;
        best_tconv = tconv;
        best_rho = rho;
        best_lam = lam2;
        best_tbar = tbar;
        best_k = k;
        best_r = r;
      }
    }
  }
  if (bestP.empty()) return fail(NETMAX_INFEASIBLE, "policy_generate: no feasible (rho, t_bar) grid point");
  std::copy(bestP.begin(), bestP.end(), prob_out);
  *rho_out = best_rho;
  if (info_out) {
    info_out[0] = best_lam;
    info_out[1] = best_tbar;
    info_out[2] = best_tconv;
    info_out[3] = best_k;
    info_out[4] = best_r;
  }
  return NETMAX_OK;
}

}  // extern "C"


// ---- constant pull weight -----------------------------------------------------------------------
namespace {

// The maximum-entropy P above the floor phi with zero diagonal, rows and columns summing to 1 and
// sum_m t_im p_im = T in every row.  Residual r = p - phi on links: r_im = A_i B_m exp(-eta_i s_im)
// with s the iteration times mapped to [0, 1].  Rows first (eta_i by a bracketed Newton iteration
// on the row's mean time, then A_i from its sum), then columns (B_m); repeated until every
// constraint holds to 1e-12.  Returns false when the constraints cannot be met.
bool solve_fixed_weight(int M, const double* t, const uint8_t* adj, double phi, double T, std::vector<double>& P) {
  std::vector<std::vector<int>> nb(M);
  std::vector<double> rows(M), cols(M, 1.0), tau(M);
  double tmin = INFINITY, tmax = 0.0;
  for (int i = 0; i < M; ++i)
    for (int m = 0; m < M; ++m)
      if (m != i && adj[(size_t)i * M + m]) {
        nb[i].push_back(m);
        tmin = std::min(tmin, t[(size_t)i * M + m]);
        tmax = std::max(tmax, t[(size_t)i * M + m]);
        cols[m] -= phi;
      }
  const bool homogeneous = tmax - tmin <= kTie * tmax;  // all links equally fast: the time constraint only says T = t
  if (homogeneous && std::fabs(T - tmin) > 1e-9 * tmax) return false;
  const double scale = homogeneous ? INFINITY : tmax - tmin;  // (t - tmin) / scale = 0 on every link then
  bool floors_fill = true;
  for (int i = 0; i < M; ++i) {
    rows[i] = 1.0 - phi * (double)nb[i].size();
    if (rows[i] < -1e-15) return false;
    double floor_time = 0.0;
    for (int m : nb[i]) floor_time += t[(size_t)i * M + m];
    tau[i] = homogeneous ? 0.0 : (T - phi * floor_time - tmin * rows[i]) / scale;  // target of sum_m s_im r_im
    if (rows[i] > 1e-15) floors_fill = false;
  }
  P.assign((size_t)M * M, 0.0);
  auto finish = [&](const std::vector<double>& r) {
    double worst = 0.0;
    std::vector<double> colsum(M, 0.0);
    for (int i = 0; i < M; ++i) {
      double sum = 0.0, time = 0.0;
      for (int m : nb[i]) {
        const double p = phi + r[(size_t)i * M + m];
        P[(size_t)i * M + m] = p;
        sum += p;
        time += p * t[(size_t)i * M + m];
        colsum[m] += p;
      }
      worst = std::max(worst, std::max(std::fabs(sum - 1.0), std::fabs(time - T) / tmax));
    }
    for (int m = 0; m < M; ++m) worst = std::max(worst, std::fabs(colsum[m] - 1.0));
    return worst <= 1e-9;
  };
  std::vector<double> r((size_t)M * M, 0.0);
  if (floors_fill) return finish(r);
  for (int i = 0; i < M; ++i)
    if (tau[i] < -1e-12 || tau[i] > rows[i] * (1.0 + 1e-12)) return false;

  std::vector<double> A(M, 1.0), B(M, 1.0), eta(M, 0.0), wgt(M);
  double err_mark = INFINITY;
  for (int sweep = 0; sweep < 20000; ++sweep) {
    // rows: weights B_m exp(-eta s_im); their mean s must equal tau_i / rows_i
    double row_change = 0.0;
    for (int i = 0; i < M; ++i) {
      if (!(rows[i] > 1e-15)) { A[i] = 0.0; continue; }
      const double sig = std::min(std::max(tau[i] / rows[i], 0.0), 1.0);
      auto stats = [&](double e, double& z, double& mean, double& var) {
        double a = 0.0, b = 0.0;
        z = 0.0;
        for (int m : nb[i]) {
          const double sv = (t[(size_t)i * M + m] - tmin) / scale;
          const double w = B[m] * std::exp(-e * sv);
          z += w;
          a += w * sv;
          b += w * sv * sv;
        }
        mean = a / z;
        var = b / z - mean * mean;
      };
      double lo = -kEtaCap, hi = kEtaCap, e = eta[i], z, mean, var;
      stats(lo, z, mean, var);
      if (sig >= mean) {
        e = lo;
      } else {
        stats(hi, z, mean, var);
        if (sig <= mean) {
          e = hi;
        } else {
          stats(e, z, mean, var);
          for (int it = 0; it < 200; ++it) {
            const double gap = mean - sig;
            if (std::fabs(gap) <= 1e-15) break;
            if (gap > 0) lo = e; else hi = e;
            double next = (var > 1e-300) ? e + gap / var : 0.5 * (lo + hi);
            if (!(next > lo && next < hi)) next = 0.5 * (lo + hi);
            if (next == e || hi - lo <= 1e-15 * (1.0 + std::fabs(e))) break;
            e = next;
            stats(e, z, mean, var);
          }
        }
      }
      stats(e, z, mean, var);
      row_change = std::max(row_change, std::fabs(e - eta[i]));
      eta[i] = e;
      A[i] = rows[i] / z;
    }
    // columns: B_m from the column sums
    double col_err = 0.0;
    std::fill(wgt.begin(), wgt.end(), 0.0);
    for (int i = 0; i < M; ++i)
      for (int m : nb[i]) wgt[m] += A[i] * std::exp(-eta[i] * (t[(size_t)i * M + m] - tmin) / scale);
    for (int m = 0; m < M; ++m) {
      if (!(wgt[m] > 0.0)) continue;
      const double next = std::max(cols[m], 0.0) / wgt[m];
      col_err = std::max(col_err, std::fabs(next - B[m]) * wgt[m]);   // column sum before the rescaling, off by this much
      B[m] = next;
    }
    if (col_err <= 1e-13 && row_change <= 1e-12) break;
    // a target outside the reachable set never settles: give up when 500 sweeps did not halve the misfit
    // (a grid point that converges more slowly than that counts as infeasible)
    if (sweep % 500 == 0) {
      if (sweep > 0 && col_err > 0.5 * err_mark) break;
      err_mark = col_err;
    }
  }
  for (int i = 0; i < M; ++i)
    for (int m : nb[i]) r[(size_t)i * M + m] = A[i] * B[m] * std::exp(-eta[i] * (t[(size_t)i * M + m] - tmin) / scale);
  return finish(r);
}

}  // namespace

extern "C" {

int netmax_policy_fixed_weight_at(int32_t M, const double* t, const uint8_t* adj, double floor, double t_bar, double* prob_out) {
  if (M < 2 || !t || !adj || !prob_out || !(floor >= 0.0) || !(t_bar > 0.0) || !std::isfinite(floor) || !std::isfinite(t_bar))
    return fail(NETMAX_INVALID_ARG, "policy_fixed_weight_at: bad argument");
  std::vector<double> P;
  if (!solve_fixed_weight(M, t, adj, floor, M * t_bar, P))
    return fail(NETMAX_INFEASIBLE, "policy_fixed_weight_at: no P meets the floors, the row and column sums and the mean iteration time");
  std::copy(P.begin(), P.end(), prob_out);
  return NETMAX_OK;
}

int netmax_policy_generate_fixed_weight(int32_t M, const double* t, const uint8_t* adj, double pull_weight, int32_t K,
                                        int32_t R, double floor_upper, double* prob_out, double* floor_out, double* info_out) {
  if (M < 2 || !t || !adj || !prob_out || !floor_out || !(pull_weight > 0.0 && pull_weight < 1.0) || K < 1 || R < 1)
    return fail(NETMAX_INVALID_ARG, "policy_generate_fixed_weight: bad argument");
  int max_deg = 0;
  for (int i = 0; i < M; ++i) {
    int deg = 0;
    for (int m = 0; m < M; ++m) {
      if (m == i || !adj[(size_t)i * M + m]) continue;
      if (!adj[(size_t)m * M + i]) return fail(NETMAX_INVALID_ARG, "policy_generate_fixed_weight: the link graph must be symmetric");
      const double tm = t[(size_t)i * M + m];
      if (!(tm > 0.0) || !std::isfinite(tm)) return fail(NETMAX_INVALID_ARG, "policy_generate_fixed_weight: iteration time on a link is not positive");
      ++deg;
    }
    if (deg == 0) return fail(NETMAX_NOT_CONNECTED, "policy_generate_fixed_weight: a worker has no neighbour");
    max_deg = std::max(max_deg, deg);
  }
  const double U_phi = floor_upper > 0.0 ? floor_upper : (1.0 - 1e-6) / max_deg;
  const double w = pull_weight;
  std::vector<double> P, Y((size_t)M * M), bestP;
  double best_tconv = INFINITY, best_phi = 0, best_lam = 0, best_tbar = 0;
  int best_k = 0, best_r = 0;
  for (int k = 1; k <= K; ++k) {
    const double phi = k * U_phi / K;
    // range of the rows' mean time: floors plus all of the remainder on the fastest / slowest link
    double L = 0.0, U = INFINITY;
    bool rows_ok = true;
    for (int i = 0; i < M; ++i) {
      double sum_t = 0.0, tmin = INFINITY, tmax = 0.0;
      int deg = 0;
      for (int m = 0; m < M; ++m) {
        if (m == i || !adj[(size_t)i * M + m]) continue;
        const double tm = t[(size_t)i * M + m];
        sum_t += tm;
        tmin = std::min(tmin, tm);
        tmax = std::max(tmax, tm);
        ++deg;
      }
      const double rest = 1.0 - phi * deg;
      if (rest < -1e-15) rows_ok = false;
      L = std::max(L, (phi * sum_t + rest * tmin) / M);
      U = std::min(U, (phi * sum_t + rest * tmax) / M);
    }
    if (!rows_ok || !(U >= L)) continue;
    for (int r = 1; r <= R; ++r) {
      const double tbar = L + (r - 0.5) * (U - L) / R;  // cell midpoints: the end points are degenerate vertices
      if (!solve_fixed_weight(M, t, adj, phi, M * tbar, P)) continue;
      // E[D^T D] with p_i = 1/M (Eq. 10 holds by construction)
      for (int i = 0; i < M; ++i) {
        double pulls = 0.0, pulled = 0.0;
        for (int m = 0; m < M; ++m) {
          if (m == i) continue;
          const double pim = P[(size_t)i * M + m], pmi = P[(size_t)m * M + i];
          Y[(size_t)i * M + m] = (w - w * w) * (pim + pmi) / M;
          pulls += pim;
          pulled += pmi;
        }
        Y[(size_t)i * M + i] = 1.0 - (2.0 * w - w * w) * pulls / M + w * w * pulled / M;
      }
      const double lam2 = second_eigenvalue(Y, M);
      if (!(lam2 > 0.0 && lam2 < 1.0)) continue;
      const double tconv = tbar * std::log(kEps) / std::log(lam2);
      if (bestP.empty() || tconv < best_tconv * (1.0 - 1e-12)) {
        bestP = P;
        best_tconv = tconv;
        best_phi = phi;
        best_lam = lam2;
        best_tbar = tbar;
        best_k = k;
        best_r = r;
      }
    }
  }
  if (bestP.empty()) return fail(NETMAX_INFEASIBLE, "policy_generate_fixed_weight: no feasible (floor, t_bar) grid point");
  std::copy(bestP.begin(), bestP.end(), prob_out);
  *floor_out = best_phi;
  if (info_out) {
    info_out[0] = best_lam;
    info_out[1] = best_tbar;
    info_out[2] = best_tconv;
    info_out[3] = best_k;
    info_out[4] = best_r;
  }
  return NETMAX_OK;
}

}  // extern "C"
