// NetMax round oracle -- TEST INFRASTRUCTURE, not the product.
//
// A plain, slow, sequential-in-spirit CPU statement of what one synchronous
// NetMax round computes, written from the paper (arXiv 2009.05766):
//
//   * peer selection            Algorithm 2 ("select a neighbour m with probability p_im")
//   * first-step update         Eq. 15:  x^{k+1/2} = x^k - alpha * g^k,  g = grad f + xi
//   * second-step (pull) update Eq. 16:  x^{k+1} = x^{k+1/2} - alpha*rho*gamma_im (x^{k+1/2} - x_m^k)
//                               with gamma_im = (d_im + d_mi) / (2 p_im)   (Section "Convergence analysis")
//
// Round semantics (a batching of the paper's one-worker-per-global-step process):
// in one round EVERY worker i performs one local iteration, and every pull reads the
// peer's replica as it was at the START of the round.  State is fp32 (the replicas'
// storage type); all arithmetic here is IEEE double, rounded to fp32 once per stored
// element.  Random numbers come from the Philox4x32-10 counter-based generator
// (Salmon, Moraes, Dror, Shaw: "Parallel random numbers: as easy as 1, 2, 3", SC'11),
// implemented here from its published definition.
//
// A second mode follows the paper's own process (Section II-B, Eq. 17): workers run
// asynchronously on simulated clocks, an iteration of worker i with peer m lasts t_im, and at
// every global step exactly ONE worker -- the one whose iteration finishes next -- updates
// its replica from the peer's CURRENT replica (nmo_async_*).
//
// Storage option (not in the paper, which trains in fp32): with bfloat16 storage the state
// holds bfloat16 values.  A stored value is then a quantised code, and the side that decides
// it must decide it in the precision of the simulator it checks: the update is evaluated in
// IEEE fp32, one operation at a time in the order
//   t = x - c;  g = fma(sigma, z, t);  h = fma(-alpha, g, x);  x' = fma(-w, h - x_m, h)
// (z = the double Box-Muller normal rounded to fp32), and x' is rounded to the nearest
// bfloat16, ties to even.  The fp32 value before that rounding is kept for the tests.
//
// Only tests, the smoke check and the benchmark's cpu_baseline leg may use this file.
// It shares no code with the CUDA library and includes none of its headers.
//
// Parity pins (see tests/): Philox against cuRAND's host generator; normals against
// the normal law; sampler against exact threshold sweeps and chi-square; the update
// against the M=2 closed form, D^k products, contraction and fixed points; the initial
// state (fill_normal) value by value against the composition of the two pinned primitives
// written out in numpy, against the normal law, and for the independence of its streams.
// Telemetry (consensus distance, mean loss) is not defined by the paper: parity unpinned
// by the paper; it is pinned against a direct numpy evaluation of its definition.

#include <algorithm>
#include <cmath>
#include <cstdint>
#include <cstring>
#include <thread>
#include <vector>

namespace {

// ---------------------------------------------------------------- Philox4x32-10
// One round: two 32x32->64 products of fixed odd multipliers with counter words 0 and 2;
// the high halves are xored with counter words 1, 3 and the round key, the low halves
// pass through, and the words are permuted.  The key is bumped by the two Weyl constants
// between rounds.  Ten rounds.
constexpr uint32_t kMul0 = 0xD2511F53u;
constexpr uint32_t kMul1 = 0xCD9E8D57u;
constexpr uint32_t kWeyl0 = 0x9E3779B9u;  // golden ratio
constexpr uint32_t kWeyl1 = 0xBB67AE85u;  // sqrt(3) - 1

void philox4x32_10(const uint32_t ctr[4], const uint32_t key[2], uint32_t out[4]) {
  uint32_t c0 = ctr[0], c1 = ctr[1], c2 = ctr[2], c3 = ctr[3];
  uint32_t k0 = key[0], k1 = key[1];
  for (int round = 0; round < 10; ++round) {
    if (round > 0) {
      k0 += kWeyl0;
      k1 += kWeyl1;
    }
    const uint64_t p0 = (uint64_t)kMul0 * c0;
    const uint64_t p1 = (uint64_t)kMul1 * c2;
    const uint32_t hi0 = (uint32_t)(p0 >> 32), lo0 = (uint32_t)p0;
    const uint32_t hi1 = (uint32_t)(p1 >> 32), lo1 = (uint32_t)p1;
    const uint32_t n0 = hi1 ^ c1 ^ k0;
    const uint32_t n1 = lo1;
    const uint32_t n2 = hi0 ^ c3 ^ k1;
    const uint32_t n3 = lo0;
    c0 = n0; c1 = n1; c2 = n2; c3 = n3;
  }
  out[0] = c0; out[1] = c1; out[2] = c2; out[3] = c3;
}

// Stream tags: the fourth counter word separates the independent streams.
enum : uint32_t { TAG_PEER = 1, TAG_NOISE = 2, TAG_X0 = 3, TAG_C = 4 };

// Counter layout: (column group e/4, worker i, round low word, tag | round high bits << 8).
inline void make_ctr(uint32_t group, uint32_t worker, uint64_t round, uint32_t tag, uint32_t ctr[4]) {
  ctr[0] = group;
  ctr[1] = worker;
  ctr[2] = (uint32_t)round;
  ctr[3] = tag | ((uint32_t)(round >> 32) << 8);
}

// Box-Muller on fixed-point uniforms that fp32 also represents exactly:
// u1 = (top23(a) + 1/2) / 2^23 in (0,1)  (2*top23+1 is a 24-bit integer),
// u2 = top24(b) / 2^24 in [0,1);  z0 = sqrt(-2 ln u1) cos(2 pi u2), z1 = ... sin(2 pi u2).
// Words (0,1) of a Philox block give the normals of lanes 0,1; words (2,3) lanes 2,3.
inline void normal_pair(uint32_t a, uint32_t b, double* z0, double* z1) {
  const double u1 = ((double)(a >> 9) + 0.5) * (1.0 / 8388608.0);
  const double u2 = (double)(b >> 8) * (1.0 / 16777216.0);
  const double rad = std::sqrt(-2.0 * std::log(u1));
  const double ang = 6.283185307179586476925286766559 * u2;
  *z0 = rad * std::cos(ang);
  *z1 = rad * std::sin(ang);
}

inline void normals4(const uint32_t r[4], double z[4]) {
  normal_pair(r[0], r[1], &z[0], &z[1]);
  normal_pair(r[2], r[3], &z[2], &z[3]);
}

// ------------------------------------------------------------------ sampler
// 32-bit fixed-point cumulative thresholds of one probability row:
//   cum_j = p_0 + ... + p_j (double, summed left to right),
//   T_j   = floor(cum_j * 2^32 + 1/2), made non-decreasing, saturated to 2^32-1 for
//           storage, and forced to the top for j >= the last index with p > 0.
// A draw u (uint32) selects m = min(#{j : T_j <= u}, last_nz).
void build_threshold_row(int M, const double* p, uint32_t* T, int32_t* last_nz) {
  int32_t last = -1;
  for (int j = 0; j < M; ++j)
    if (p[j] > 0.0) last = j;
  *last_nz = last;
  double cum = 0.0;
  uint64_t prev = 0;
  for (int j = 0; j < M; ++j) {
    cum += p[j];
    uint64_t t = (uint64_t)std::floor(cum * 4294967296.0 + 0.5);
    if (t < prev) t = prev;
    if (t > 0xFFFFFFFFull || j >= last) t = 0xFFFFFFFFull;
    T[j] = (uint32_t)t;
    prev = t;
  }
}

inline int32_t sample_row(const uint32_t* T, int M, int32_t last_nz, uint32_t u) {
  int32_t count = 0;
  for (int j = 0; j < M; ++j)
    if (T[j] <= u) ++count;
  return std::min(count, last_nz);
}

// Pull weight  w_im = alpha * rho * gamma_im = alpha*rho*(d_im + d_mi) / (2 p_im),
// computed in double and rounded to fp32 (the precision the replicas are updated in).
// Entries with p_im = 0 or m = i are 0 (never used: a self-draw skips the pull).
// fixed_w > 0 replaces it by one constant for every pull: the update rule of gossip / AD-PSGD
// style averaging (fixed_w = 1/2), which the paper's Section "Extension to existing
// decentralized PSGD approaches" puts in the same form x <- D(x - alpha g).
void build_weight_row(int M, int i, const double* P, const uint8_t* adj, double alpha, double rho, float* w,
                      double fixed_w = 0.0) {
  for (int m = 0; m < M; ++m) {
    const double p = P[(size_t)i * M + m];
    if (m == i || !(p > 0.0)) {
      w[m] = 0.0f;
      continue;
    }
    if (fixed_w > 0.0) {
      w[m] = (float)fixed_w;
      continue;
    }
    const double dsum = (double)adj[(size_t)i * M + m] + (double)adj[(size_t)m * M + i];
    w[m] = (float)(alpha * rho * dsum / (2.0 * p));
  }
}

// ------------------------------------------------------------------ simulator
// Nearest bfloat16 (the top 16 bits of the fp32 pattern), ties to even, returned as fp32.
// Finite inputs only.
inline float bf16_round(float v) {
  uint32_t u;
  std::memcpy(&u, &v, 4);
  const uint32_t keep_odd = (u >> 16) & 1u;  // makes an exact tie round to the even neighbour
  u = (u + 0x7FFFu + keep_odd) & 0xFFFF0000u;
  std::memcpy(&v, &u, 4);
  return v;
}

struct Sim {
  int M = 0;
  int64_t d = 0;           // logical vector length (defines the noise counters)
  int64_t ncols = 0;       // number of simulated columns (== d, or a sample of them)
  std::vector<int64_t> cols;  // logical element index of each simulated column
  double alpha = 0, rho = 0, sigma = 0;  // alpha, sigma already rounded to fp32 values
  double fixed_w = 0.0;                  // > 0: every pull uses this weight instead of Eq. 16's
  int objective = 1;
  int storage = 0;                       // 0: fp32 state, double arithmetic; 1: bfloat16 state, fp32 arithmetic
  std::vector<float> pre;                // storage 1: fp32 values of the last round before the bfloat16 rounding
  uint32_t key[2] = {0, 0};
  uint64_t round = 0;   // number of the next round: a word of every counter
  uint64_t round0 = 0;  // number of the first round (the trace and telemetry vectors start there)
  std::vector<uint32_t> T;
  std::vector<int32_t> last_nz;
  std::vector<float> w;
  std::vector<float> x, xn, c;  // [M][ncols]
  std::vector<int32_t> trace;   // [round][M], all rounds since creation
  std::vector<double> tel_consensus, tel_loss;  // per round, on the round-start state
  // asynchronous timeline
  bool async_on = false;
  double beta = 0.0;
  std::vector<double> t_iter;          // [M][M] iteration times, t_ii = compute-only
  std::vector<int64_t> local_n;        // [M] local iteration index n of the pending iteration
  std::vector<int32_t> pending_peer;   // [M] peer drawn for the pending iteration
  std::vector<float> pending_w;        // [M] its pull weight, from the policy in force when it started
  std::vector<double> pending_t;       // [M] its duration t_im, from the times in force when it started
  std::vector<double> finish;          // [M] simulated time at which the pending iteration ends
  std::vector<double> ema;             // [M][M] EMA of measured iteration times (Algorithm 2)
  std::vector<int64_t> ema_count;      // [M][M] samples folded into the EMA
  double now = 0.0;
  std::vector<int32_t> ev_worker, ev_peer;
  std::vector<int64_t> ev_n;
  std::vector<double> ev_time;
};

void sim_set_policy(Sim* s, const double* P, const uint8_t* adj, double rho) {
  const int M = s->M;
  s->rho = rho;
  s->T.assign((size_t)M * M, 0);
  s->last_nz.assign(M, 0);
  s->w.assign((size_t)M * M, 0.0f);
  for (int i = 0; i < M; ++i) {
    build_threshold_row(M, P + (size_t)i * M, s->T.data() + (size_t)i * M, &s->last_nz[i]);
    build_weight_row(M, i, P, adj, s->alpha, rho, s->w.data() + (size_t)i * M, s->fixed_w);
  }
}

void fill_normal(Sim* s, std::vector<float>& dst, double stddev, uint32_t tag) {
  for (int i = 0; i < s->M; ++i)
    for (int64_t k = 0; k < s->ncols; ++k) {
      const int64_t e = s->cols[k];
      uint32_t ctr[4], r[4];
      double z[4];
      make_ctr((uint32_t)(e >> 2), (uint32_t)i, 0, tag, ctr);
      philox4x32_10(ctr, s->key, r);
      normals4(r, z);
      // bfloat16 storage: fp32 normal times the fp32 scale (one fp32 product), then rounded
      dst[(size_t)i * s->ncols + k] =
          s->storage == 1 ? bf16_round((float)z[e & 3] * (float)stddev) : (float)(stddev * z[e & 3]);
    }
}

// Telemetry on the current state: consensus distance (1/M) sum_i ||x_i - xbar||^2 and
// mean loss (1/M) sum_i 1/2 ||x_i - c_i||^2 (the two terms of the paper's Eq. 1 that the
// simulator can observe).  Plain double sums over the simulated columns.
void telemetry(const Sim* s, double* consensus, double* loss) {
  const int M = s->M;
  double cons = 0.0, ls = 0.0;
  for (int64_t k = 0; k < s->ncols; ++k) {
    double mean = 0.0;
    for (int i = 0; i < M; ++i) mean += (double)s->x[(size_t)i * s->ncols + k];
    mean /= M;
    for (int i = 0; i < M; ++i) {
      const double xv = (double)s->x[(size_t)i * s->ncols + k];
      const double cv = (double)s->c[(size_t)i * s->ncols + k];
      cons += (xv - mean) * (xv - mean);
      ls += 0.5 * (xv - cv) * (xv - cv);
    }
  }
  *consensus = cons / M;
  *loss = ls / M;
}

// bfloat16 storage: Eq. 15 and Eq. 16 on one element in fp32, one operation at a time in the
// order the header states; `iter` is the round (or the worker's local iteration on the
// asynchronous timeline).  Returns the fp32 value before the rounding to bfloat16.
float update_fp32(const Sim* s, int i, uint64_t iter, int64_t e, float xv, float cv, float xmv, float alpha, float sigma,
                  float wf) {
  float h = xv;
  if (s->objective == 1) {
    uint32_t ctr[4], r[4];
    double z[4];
    make_ctr((uint32_t)(e >> 2), (uint32_t)i, iter, TAG_NOISE, ctr);
    philox4x32_10(ctr, s->key, r);
    normals4(r, z);
    const float t = xv - cv;
    const float g = std::fmaf(sigma, (float)z[e & 3], t);
    h = std::fmaf(-alpha, g, xv);  // Eq. 15
  }
  const float diff = h - xmv;
  return std::fmaf(-wf, diff, h);  // Eq. 16 (w = 0 on a self-draw)
}

void round_columns(Sim* s, const int32_t* peer, int64_t k0, int64_t k1) {
  const int M = s->M;
  const int64_t n = s->ncols;
  for (int i = 0; i < M; ++i) {
    const int m = peer[i];
    const double w = (double)s->w[(size_t)i * M + m];
    const float* xi = s->x.data() + (size_t)i * n;
    const float* xm = s->x.data() + (size_t)m * n;  // round-start snapshot of the peer
    const float* ci = s->c.data() + (size_t)i * n;
    float* out = s->xn.data() + (size_t)i * n;
    if (s->storage == 1) {  // bfloat16 state: fp32 arithmetic in the stated order, one rounding to bfloat16
      const float alpha = (float)s->alpha, sigma = (float)s->sigma, wf = (m != i) ? s->w[(size_t)i * M + m] : 0.0f;
      float* pre = s->pre.data() + (size_t)i * n;
      for (int64_t k = k0; k < k1; ++k) {
        const float xnew = update_fp32(s, i, s->round, s->cols[k], xi[k], ci[k], xm[k], alpha, sigma, wf);
        pre[k] = xnew;
        out[k] = bf16_round(xnew);
      }
      continue;
    }
    for (int64_t k = k0; k < k1; ++k) {
      const int64_t e = s->cols[k];
      const double xv = (double)xi[k];
      double g = 0.0;
      if (s->objective == 1) {
        uint32_t ctr[4], r[4];
        double z[4];
        make_ctr((uint32_t)(e >> 2), (uint32_t)i, s->round, TAG_NOISE, ctr);
        philox4x32_10(ctr, s->key, r);
        normals4(r, z);
        g = (xv - (double)ci[k]) + s->sigma * z[e & 3];  // grad of 1/2||x-c||^2, plus additive noise
      }
      const double h = xv - s->alpha * g;                        // Eq. 15
      double xnew = h;
      if (m != i) xnew = h - w * (h - (double)xm[k]);            // Eq. 16; a self-draw pulls nothing
      out[k] = (float)xnew;
    }
  }
}

void sim_round(Sim* s, int threads) {
  const int M = s->M;
  std::vector<int32_t> peer(M);
  for (int i = 0; i < M; ++i) {
    uint32_t ctr[4], r[4];
    make_ctr(0, (uint32_t)i, s->round, TAG_PEER, ctr);
    philox4x32_10(ctr, s->key, r);
    peer[i] = sample_row(s->T.data() + (size_t)i * M, M, s->last_nz[i], r[0]);
  }
  double cons, ls;
  telemetry(s, &cons, &ls);
  s->tel_consensus.push_back(cons);
  s->tel_loss.push_back(ls);
  s->trace.insert(s->trace.end(), peer.begin(), peer.end());

  threads = std::max(1, threads);
  if (threads == 1 || s->ncols < 4096) {
    round_columns(s, peer.data(), 0, s->ncols);
  } else {
    std::vector<std::thread> pool;
    const int64_t per = (s->ncols + threads - 1) / threads;
    for (int t = 0; t < threads; ++t) {
      const int64_t k0 = std::min<int64_t>(s->ncols, t * per), k1 = std::min<int64_t>(s->ncols, k0 + per);
      if (k0 < k1) pool.emplace_back(round_columns, s, peer.data(), k0, k1);
    }
    for (auto& th : pool) th.join();
  }
  s->x.swap(s->xn);
  s->round += 1;
}

// ---------------------------------------------------------------- asynchronous timeline
// Worker i's iteration n: peer m drawn from P[i,:] with the PEER stream at counter (0, i, n),
// duration t_im (Section II-B: t_im = max{C_i, N_im}); the next iteration starts when this
// one ends.  Algorithm 2 takes a new policy (P[i], rho) at the top of an iteration, before the
// peer is selected, and its UpdateTimeVector records how long the iteration took: so the pull
// weight alpha rho gamma_im and the duration t_im of an iteration are those in force when it
// STARTS, whatever changes while it is in flight.
void async_start_iteration(Sim* s, int i, double start) {
  uint32_t ctr[4], r[4];
  make_ctr(0, (uint32_t)i, (uint64_t)s->local_n[i], TAG_PEER, ctr);
  philox4x32_10(ctr, s->key, r);
  const int m = sample_row(s->T.data() + (size_t)i * s->M, s->M, s->last_nz[i], r[0]);
  s->pending_peer[i] = m;
  s->pending_w[i] = (m != i) ? s->w[(size_t)i * s->M + m] : 0.0f;
  s->pending_t[i] = s->t_iter[(size_t)i * s->M + m];
  s->finish[i] = start + s->pending_t[i];
}

// One global step (Eq. 17): the worker whose iteration finishes first (ties: lowest index)
// applies  x_i <- (1 - w_im)(x_i - alpha g_i) + w_im x_m  with the peer's current replica;
// every other replica is unchanged.  Then it records the iteration time (Algorithm 2,
// UpdateTimeVector: T_i[m] <- beta T_i[m] + (1 - beta) t_im) and starts its next iteration.
void async_step(Sim* s) {
  const int M = s->M;
  int i = 0;
  for (int j = 1; j < M; ++j)
    if (s->finish[j] < s->finish[i]) i = j;
  const int m = s->pending_peer[i];
  const int64_t nloc = s->local_n[i];
  const float wf = s->pending_w[i];  // fixed when the iteration started (0 on a self-draw)
  const double w = (double)wf;
  const int64_t n = s->ncols;
  float* xi = s->x.data() + (size_t)i * n;
  const float* xm = s->x.data() + (size_t)m * n;
  const float* ci = s->c.data() + (size_t)i * n;
  for (int64_t k = 0; k < n; ++k) {
    const int64_t e = s->cols[k];
    if (s->storage == 1) {  // bfloat16 state: the same fp32 evaluation as in a round, rounded once
      const float xnew = update_fp32(s, i, (uint64_t)nloc, e, xi[k], ci[k], xm[k], (float)s->alpha, (float)s->sigma, wf);
      s->pre[(size_t)i * n + k] = xnew;
      xi[k] = bf16_round(xnew);
      continue;
    }
    const double xv = (double)xi[k];
    double g = 0.0;
    if (s->objective == 1) {
      uint32_t ctr[4], r[4];
      double z[4];
      make_ctr((uint32_t)(e >> 2), (uint32_t)i, (uint64_t)nloc, TAG_NOISE, ctr);
      philox4x32_10(ctr, s->key, r);
      normals4(r, z);
      g = (xv - (double)ci[k]) + s->sigma * z[e & 3];
    }
    const double h = xv - s->alpha * g;
    double xnew = h;
    if (m != i) xnew = h - w * (h - (double)xm[k]);
    xi[k] = (float)xnew;
  }
  s->now = s->finish[i];
  s->ev_worker.push_back(i);
  s->ev_peer.push_back(m);
  s->ev_n.push_back(nloc);
  s->ev_time.push_back(s->now);
  const size_t at = (size_t)i * M + m;
  s->ema[at] = s->beta * s->ema[at] + (1.0 - s->beta) * s->pending_t[i];  // the time this iteration took
  s->ema_count[at] += 1;
  s->local_n[i] = nloc + 1;
  async_start_iteration(s, i, s->now);
}

}  // namespace

extern "C" {

void nmo_philox4x32_10(const uint32_t* ctr, const uint32_t* key, uint32_t* out) { philox4x32_10(ctr, key, out); }

// out[4n]: blocks for counters (c0_first + j, c1, c2, c3), j = 0..n-1.
void nmo_philox_blocks(uint64_t seed, uint32_t c0_first, uint32_t c1, uint32_t c2, uint32_t c3, int64_t n,
                       uint32_t* out) {
  const uint32_t key[2] = {(uint32_t)seed, (uint32_t)(seed >> 32)};
  for (int64_t j = 0; j < n; ++j) {
    const uint32_t ctr[4] = {c0_first + (uint32_t)j, c1, c2, c3};
    philox4x32_10(ctr, key, out + 4 * j);
  }
}

// Normals of the noise stream: z[n] for elements e0..e0+n-1 of worker i at a round.
void nmo_noise(uint64_t seed, int32_t worker, uint64_t round, int64_t e0, int64_t n, double* z) {
  const uint32_t key[2] = {(uint32_t)seed, (uint32_t)(seed >> 32)};
  for (int64_t e = e0; e < e0 + n; ++e) {
    uint32_t ctr[4], r[4];
    double zz[4];
    make_ctr((uint32_t)(e >> 2), (uint32_t)worker, round, TAG_NOISE, ctr);
    philox4x32_10(ctr, key, r);
    normals4(r, zz);
    z[e - e0] = zz[e & 3];
  }
}

void nmo_normals_from_words(const uint32_t* r4, double* z4) { normals4(r4, z4); }

void nmo_build_thresholds(int32_t M, const double* P, uint32_t* T, int32_t* last_nz) {
  for (int i = 0; i < M; ++i) build_threshold_row(M, P + (size_t)i * M, T + (size_t)i * M, last_nz + i);
}

int32_t nmo_sample(const uint32_t* Trow, int32_t M, int32_t last_nz, uint32_t u) { return sample_row(Trow, M, last_nz, u); }

void nmo_build_weights(int32_t M, const double* P, const uint8_t* adj, double alpha, double rho, float* w) {
  for (int i = 0; i < M; ++i) build_weight_row(M, i, P, adj, alpha, rho, w + (size_t)i * M);
}

// Peer draws only (no replica state): out[n_rounds][M].
void nmo_peer_draws(int32_t M, const double* P, uint64_t seed, uint64_t first_round, int64_t n_rounds, int32_t* out) {
  std::vector<uint32_t> T((size_t)M * M);
  std::vector<int32_t> last(M);
  nmo_build_thresholds(M, P, T.data(), last.data());
  const uint32_t key[2] = {(uint32_t)seed, (uint32_t)(seed >> 32)};
  for (int64_t r = 0; r < n_rounds; ++r)
    for (int i = 0; i < M; ++i) {
      uint32_t ctr[4], w[4];
      make_ctr(0, (uint32_t)i, first_round + (uint64_t)r, TAG_PEER, ctr);
      philox4x32_10(ctr, key, w);
      out[(size_t)r * M + i] = sample_row(T.data() + (size_t)i * M, M, last[i], w[0]);
    }
}

// cols == nullptr: simulate all d columns; else the ncols listed logical element indices.
void* nmo_sim_create(int32_t M, int64_t d, const int64_t* cols, int64_t ncols, const double* P, const uint8_t* adj,
                     double alpha, double rho, double sigma, int32_t objective, uint64_t seed) {
  Sim* s = new Sim();
  s->M = M;
  s->d = d;
  if (cols) {
    s->ncols = ncols;
    s->cols.assign(cols, cols + ncols);
  } else {
    s->ncols = d;
    s->cols.resize(d);
    for (int64_t e = 0; e < d; ++e) s->cols[e] = e;
  }
  s->alpha = (double)(float)alpha;  // the update runs on fp32 parameters
  s->sigma = (double)(float)sigma;
  s->objective = objective;
  s->key[0] = (uint32_t)seed;
  s->key[1] = (uint32_t)(seed >> 32);
  s->x.assign((size_t)M * s->ncols, 0.0f);
  s->xn.assign((size_t)M * s->ncols, 0.0f);
  s->c.assign((size_t)M * s->ncols, 0.0f);
  sim_set_policy(s, P, adj, rho);
  return s;
}

void nmo_sim_destroy(void* h) { delete (Sim*)h; }
// Takes effect at the next nmo_sim_set_policy.
void nmo_sim_set_fixed_weight(void* h, double fixed_w) { ((Sim*)h)->fixed_w = fixed_w; }
void nmo_sim_set_policy(void* h, const double* P, const uint8_t* adj, double rho) { sim_set_policy((Sim*)h, P, adj, rho); }

// x_i(0) = x0_std * z, c_i = c_std * z from the X0 / C streams (round word 0).
void nmo_sim_init(void* h, double x0_std, double c_std) {
  Sim* s = (Sim*)h;
  fill_normal(s, s->x, x0_std, TAG_X0);
  fill_normal(s, s->c, c_std, TAG_C);
}

void nmo_sim_set_x(void* h, const float* x) {
  Sim* s = (Sim*)h;
  for (size_t k = 0; k < s->x.size(); ++k) s->x[k] = s->storage == 1 ? bf16_round(x[k]) : x[k];
}
void nmo_sim_set_c(void* h, const float* c) {
  Sim* s = (Sim*)h;
  for (size_t k = 0; k < s->c.size(); ++k) s->c[k] = s->storage == 1 ? bf16_round(c[k]) : c[k];
}
// Before any state is set.  1: bfloat16 storage with fp32 arithmetic (see the header).
void nmo_sim_set_storage(void* h, int32_t storage) {
  Sim* s = (Sim*)h;
  s->storage = storage;
  s->pre.assign(storage == 1 ? s->x.size() : 0, 0.0f);
}
// bfloat16 storage: the last round's new parameters before they were rounded to bfloat16.
void nmo_sim_get_unrounded(void* h, float* out) { Sim* s = (Sim*)h; std::memcpy(out, s->pre.data(), s->pre.size() * sizeof(float)); }
void nmo_bf16_round(const float* in, int64_t n, float* out) { for (int64_t k = 0; k < n; ++k) out[k] = bf16_round(in[k]); }
void nmo_sim_get_x(void* h, float* x) { Sim* s = (Sim*)h; std::memcpy(x, s->x.data(), s->x.size() * sizeof(float)); }
void nmo_sim_get_c(void* h, float* c) { Sim* s = (Sim*)h; std::memcpy(c, s->c.data(), s->c.size() * sizeof(float)); }

void nmo_sim_round(void* h, int64_t n_rounds, int32_t threads) {
  for (int64_t r = 0; r < n_rounds; ++r) sim_round((Sim*)h, threads);
}

// Rounds run since creation (the trace holds that many).
int64_t nmo_sim_rounds_done(void* h) { return (int64_t)(((Sim*)h)->round - ((Sim*)h)->round0); }
// Before any round: number the rounds from `first` on (the round number enters every counter).
void nmo_sim_set_first_round(void* h, uint64_t first) { ((Sim*)h)->round = ((Sim*)h)->round0 = first; }

void nmo_sim_get_trace(void* h, int64_t first, int64_t n, int32_t* out) {
  Sim* s = (Sim*)h;
  std::memcpy(out, s->trace.data() + (size_t)first * s->M, (size_t)n * s->M * sizeof(int32_t));
}

void nmo_sim_get_telemetry(void* h, int64_t first, int64_t n, double* consensus, double* loss) {
  Sim* s = (Sim*)h;
  for (int64_t r = 0; r < n; ++r) {
    consensus[r] = s->tel_consensus[first + r];
    loss[r] = s->tel_loss[first + r];
  }
}

void nmo_sim_telemetry_now(void* h, double* consensus, double* loss) { telemetry((Sim*)h, consensus, loss); }

// ---- asynchronous timeline
void nmo_async_begin(void* h, const double* t_iter, double beta) {
  Sim* s = (Sim*)h;
  const int M = s->M;
  s->async_on = true;
  s->beta = beta;
  s->t_iter.assign(t_iter, t_iter + (size_t)M * M);
  s->local_n.assign(M, 0);
  s->pending_peer.assign(M, 0);
  s->pending_w.assign(M, 0.0f);
  s->pending_t.assign(M, 0.0);
  s->finish.assign(M, 0.0);
  s->ema.assign((size_t)M * M, 0.0);
  s->ema_count.assign((size_t)M * M, 0);
  s->now = 0.0;
  for (int i = 0; i < M; ++i) async_start_iteration(s, i, 0.0);
}

void nmo_async_set_times(void* h, const double* t_iter) {
  Sim* s = (Sim*)h;
  s->t_iter.assign(t_iter, t_iter + (size_t)s->M * s->M);
}

void nmo_async_steps(void* h, int64_t n) {
  for (int64_t k = 0; k < n; ++k) async_step((Sim*)h);
}

int64_t nmo_async_steps_done(void* h) { return (int64_t)((Sim*)h)->ev_worker.size(); }
double nmo_async_now(void* h) { return ((Sim*)h)->now; }
// Simulated time of the next global step (the earliest pending finish time).
double nmo_async_next_time(void* h) {
  Sim* s = (Sim*)h;
  return *std::min_element(s->finish.begin(), s->finish.end());
}

void nmo_async_trace(void* h, int64_t first, int64_t n, int32_t* worker, int32_t* peer, int64_t* local_iter, double* time) {
  Sim* s = (Sim*)h;
  for (int64_t k = 0; k < n; ++k) {
    worker[k] = s->ev_worker[first + k];
    peer[k] = s->ev_peer[first + k];
    local_iter[k] = s->ev_n[first + k];
    time[k] = s->ev_time[first + k];
  }
}

void nmo_async_ema(void* h, double* ema, int64_t* count) {
  Sim* s = (Sim*)h;
  std::memcpy(ema, s->ema.data(), s->ema.size() * sizeof(double));
  std::memcpy(count, s->ema_count.data(), s->ema_count.size() * sizeof(int64_t));
}

}  // extern "C"
