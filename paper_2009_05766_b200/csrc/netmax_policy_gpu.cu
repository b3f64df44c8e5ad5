// Communication-policy generation (Algorithm 3) on the GPU, for large M.
//
// Same readings and the same per-row solution as the host generator (netmax_policy.cpp): the
// grids rho_k = k U_rho / K and t_bar_r = U - (R - r)(U - L)/R; per grid point the row-wise LP
// optimum (Eq. 14 under Eq. 10-13: floor + exponential tilt, or least p_ii + fastest peers),
// Y_P (Eq. 22 with p_i = 1/M), its second largest eigenvalue by Lanczos on the complement of
// the all-ones vector, and the arg-min of t_bar ln(eps) / ln(lambda_2).  One CTA solves one row;
// the M x M matrices t, P and Y stay in device memory in fp64.
#include "../../include/netmax.h"

#include <algorithm>
#include <cmath>
#include <cstdio>
#include <vector>

#include <cuda_runtime.h>

#include "netmax_policy.h"

namespace {

constexpr int kRowThreads = 256;
constexpr double kEtaCap = 600.0;
constexpr double kTie = 1e-12;
constexpr double kEps = 1e-3;

struct RowInfo {  // per row, independent of the grid point
  double C, tmin, tmax, sum_f1, sum_f1t;
  int n_nb, n_fast;
};

__device__ __forceinline__ double warp_sum(double v) {
  for (int off = 16; off > 0; off >>= 1) v += __shfl_down_sync(0xffffffffu, v, off);
  return v;
}

// Sum of v over the CTA, returned to every thread.  s_buf: 33 doubles.
__device__ double block_sum(double v, double* s_buf) {
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, nw = blockDim.x >> 5;
  v = warp_sum(v);
  __syncthreads();
  if (lane == 0) s_buf[warp] = v;
  __syncthreads();
  if (warp == 0) {
    double t = lane < nw ? s_buf[lane] : 0.0;
    t = warp_sum(t);
    if (lane == 0) s_buf[32] = t;
  }
  __syncthreads();
  return s_buf[32];
}

__device__ double block_min(double v, double* s_buf) {
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, nw = blockDim.x >> 5;
  for (int off = 16; off > 0; off >>= 1) v = fmin(v, __shfl_down_sync(0xffffffffu, v, off));
  __syncthreads();
  if (lane == 0) s_buf[warp] = v;
  __syncthreads();
  if (warp == 0) {
    double t = lane < nw ? s_buf[lane] : INFINITY;
    for (int off = 16; off > 0; off >>= 1) t = fmin(t, __shfl_down_sync(0xffffffffu, t, off));
    if (lane == 0) s_buf[32] = t;
  }
  __syncthreads();
  return s_buf[32];
}

__global__ void __launch_bounds__(kRowThreads) row_info_kernel(int M, const double* t, const uint8_t* adj, RowInfo* info) {
  __shared__ double s_buf[33];
  const int i = blockIdx.x;
  double f1s = 0, f1t = 0, mn = INFINITY, mx = -INFINITY, nb = 0;
  for (int m = threadIdx.x; m < M; m += blockDim.x) {
    if (m == i || !adj[(size_t)i * M + m]) continue;
    const double tm = t[(size_t)i * M + m];
    const double f1 = (double)adj[(size_t)i * M + m] + (double)adj[(size_t)m * M + i];
    f1s += f1;
    f1t += f1 * tm;
    mn = fmin(mn, tm);
    mx = fmax(mx, tm);
    nb += 1;
  }
  f1s = block_sum(f1s, s_buf);
  f1t = block_sum(f1t, s_buf);
  nb = block_sum(nb, s_buf);
  mn = block_min(mn, s_buf);
  mx = -block_min(-mx, s_buf);
  double fast = 0;
  for (int m = threadIdx.x; m < M; m += blockDim.x)
    if (m != i && adj[(size_t)i * M + m] && t[(size_t)i * M + m] <= mn * (1.0 + kTie)) fast += 1;
  fast = block_sum(fast, s_buf);
  if (threadIdx.x == 0) {
    RowInfo r;
    r.C = t[(size_t)i * M + i];
    r.tmin = mn;
    r.tmax = mx;
    r.sum_f1 = f1s;
    r.sum_f1t = f1t;
    r.n_nb = (int)nb;
    r.n_fast = (int)fast;
    info[i] = r;
  }
}

// One row of the LP at (alpha rho, T = M t_bar); ok[i] = 0 marks an infeasible row.
__global__ void __launch_bounds__(kRowThreads) row_solve_kernel(int M, const double* t, const uint8_t* adj, const RowInfo* info,
                                                                double ar, double T, double* P, int* ok) {
  __shared__ double s_buf[33];
  const int i = blockIdx.x;
  const RowInfo r = info[i];
  const double* ti = t + (size_t)i * M;
  const uint8_t* ai = adj + (size_t)i * M;
  double* pi = P + (size_t)i * M;
  const double F = ar * r.sum_f1;
  const double free_mass = 1.0 - F, A = ar * r.sum_f1t;
  const double lo = A + free_mass * r.tmin, hi = A + free_mass * r.tmax;
  if (F > 1.0 || T > hi * (1.0 + kTie)) {
    if (threadIdx.x == 0) ok[i] = 0;
    return;
  }
  auto f1_of = [&](int m) { return (double)ai[m] + (double)adj[(size_t)m * M + i]; };
  if (T >= lo * (1.0 - kTie)) {
    const double scale = r.tmax - r.tmin;
    const bool flat = !(scale > kTie * r.tmax) || free_mass <= 0.0;
    double eta = 0.0, z = (double)r.n_nb;
    bool good = true;
    if (!flat) {
      const double target = fmin(fmax((T - A) / free_mass, r.tmin), r.tmax);
      const double sig = (target - r.tmin) / scale;
      // mean and variance of s under q ~ exp(-eta s), s = (t - tmin) / scale
      auto stats = [&](double e, double& mean, double& var, double& zz) {
        double a0 = 0, a1 = 0, a2 = 0;
        for (int m = threadIdx.x; m < M; m += blockDim.x) {
          if (m == i || !ai[m]) continue;
          const double s = (ti[m] - r.tmin) / scale, w = exp(-e * s);
          a0 += w;
          a1 += w * s;
          a2 += w * s * s;
        }
        a0 = block_sum(a0, s_buf);
        a1 = block_sum(a1, s_buf);
        a2 = block_sum(a2, s_buf);
        zz = a0;
        mean = a1 / a0;
        var = a2 / a0 - mean * mean;
      };
      double mean, var, elo = -kEtaCap, ehi = kEtaCap;
      stats(elo, mean, var, z);
      if (sig >= mean) {
        eta = elo;
      } else {
        stats(ehi, mean, var, z);
        if (sig <= mean) {
          eta = ehi;
        } else {
          stats(eta, mean, var, z);
          for (int it = 0; it < 200; ++it) {  // Newton steps kept inside a shrinking bracket
            const double gap = mean - sig;
            if (fabs(gap) <= 1e-15) break;
            if (gap > 0) elo = eta; else ehi = eta;
            double next = (var > 1e-300) ? eta + gap / var : 0.5 * (elo + ehi);
            if (!(next > elo && next < ehi)) next = 0.5 * (elo + ehi);
            if (next == eta || ehi - elo <= 1e-15 * (1.0 + fabs(eta))) break;
            eta = next;
            stats(eta, mean, var, z);
          }
        }
      }
      stats(eta, mean, var, z);
      good = fabs(mean - sig) <= 1e-9;
    }
    for (int m = threadIdx.x; m < M; m += blockDim.x) {
      double p = 0.0;
      if (m != i && ai[m]) {
        const double q = flat ? 1.0 / (double)r.n_nb : exp(-eta * (ti[m] - r.tmin) / scale) / z;
        p = ar * f1_of(m) + (free_mass > 0.0 ? free_mass * q : 0.0);
      }
      pi[m] = p;
    }
    if (threadIdx.x == 0) ok[i] = good ? 1 : 0;
    return;
  }
  double pii = (lo - T) / (r.tmin - r.C);
  if (pii > free_mass * (1.0 + kTie)) {
    if (threadIdx.x == 0) ok[i] = 0;
    return;
  }
  pii = fmin(pii, free_mass);
  for (int m = threadIdx.x; m < M; m += blockDim.x) {
    double p = 0.0;
    if (m == i) p = pii;
    else if (ai[m]) p = ar * f1_of(m) + (ti[m] <= r.tmin * (1.0 + kTie) ? (free_mass - pii) / r.n_fast : 0.0);
    pi[m] = p;
  }
  if (threadIdx.x == 0) ok[i] = 1;
}

// Y_P (Eq. 22) with p_i = 1/M: p_im gamma_im = (d_im+d_mi)/2, p_im gamma_im^2 = (d_im+d_mi)^2/(4 p_im).
__global__ void __launch_bounds__(kRowThreads) y_kernel(int M, const double* P, const uint8_t* adj, double ar, double* Y) {
  __shared__ double s_buf[33];
  const int i = blockIdx.x;
  double rowsum = 0.0;
  for (int m = threadIdx.x; m < M; m += blockDim.x) {
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
  rowsum = block_sum(rowsum, s_buf);
  if (threadIdx.x == 0) Y[(size_t)i * M + i] = 1.0 - rowsum;
}

// ---- Lanczos pieces (vectors of length M, fp64) -----------------------------------------------
// out = (Y - 11^T/M) v : one warp per row.
__global__ void __launch_bounds__(256) matvec_kernel(int M, const double* Y, const double* v, const double* vsum, double* out) {
  const int row = blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5), lane = threadIdx.x & 31;
  if (row >= M) return;
  const double* y = Y + (size_t)row * M;
  double acc = 0.0;
  for (int j = lane; j < M; j += 32) acc += y[j] * v[j];
  acc = warp_sum(acc);
  if (lane == 0) out[row] = acc - vsum[0] / M;
}

// dots[u] = sum_j V[u][j] * w[j] for u < n_vec : one CTA per vector.
__global__ void __launch_bounds__(256) dots_kernel(int M, const double* V, const double* w, double* dots) {
  __shared__ double s_buf[33];
  const double* v = V + (size_t)blockIdx.x * M;
  double acc = 0.0;
  for (int j = threadIdx.x; j < M; j += blockDim.x) acc += v[j] * w[j];
  acc = block_sum(acc, s_buf);
  if (threadIdx.x == 0) dots[blockIdx.x] = acc;
}

// w[j] -= sum_u dots[u] V[u][j]
__global__ void __launch_bounds__(256) project_out_kernel(int M, int n_vec, const double* V, const double* dots, double* w) {
  const int j = blockIdx.x * blockDim.x + threadIdx.x;
  if (j >= M) return;
  double acc = 0.0;
  for (int u = 0; u < n_vec; ++u) acc += dots[u] * V[(size_t)u * M + j];
  w[j] -= acc;
}

// alpha[step] = dots[step] (the Rayleigh coefficient taken before the projections)
__global__ void store_alpha_kernel(const double* dots, int step, double* alpha) { alpha[step] = dots[step]; }

// beta[step] = ||w||, next = w / beta, and its element sum (for the next matvec)
__global__ void __launch_bounds__(1024) normalise_kernel(int M, const double* w, double* next, double* beta, int step, double* vsum) {
  __shared__ double s_buf[33];
  double a = 0.0;
  for (int j = threadIdx.x; j < M; j += blockDim.x) a += w[j] * w[j];
  a = block_sum(a, s_buf);
  const double b = sqrt(a);
  double s = 0.0;
  for (int j = threadIdx.x; j < M; j += blockDim.x) {
    const double x = b > 0.0 ? w[j] / b : 0.0;
    next[j] = x;
    s += x;
  }
  s = block_sum(s, s_buf);
  if (threadIdx.x == 0) {
    beta[step] = b;
    vsum[0] = s;
  }
}

}  // namespace

#include "netmax_policy_gpu_host.inc"
