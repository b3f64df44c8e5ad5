// C-ABI implementation of the NetMax round simulator (see include/netmax.h).
//
// Host side: validation, the 32-bit cumulative-threshold and pull-weight tables, buffer
// layout, launches.  Every step of a round runs in the kernels of netmax_kernels.cuh.
#include "../../include/netmax.h"

#include <algorithm>
#include <cmath>
#include <cstdarg>
#include <cstdio>
#include <cstring>
#include <mutex>
#include <new>
#include <queue>
#include <string>
#include <vector>

#include <cuda_runtime.h>

#include "netmax_kernels.cuh"
#include "netmax_policy.h"

using namespace netmax;

namespace {

thread_local std::string g_error;  // failures of calls that have no context

constexpr int kThreads = 256;
constexpr int64_t kMaxM = 16384;
constexpr int64_t kMaxD = ((int64_t)1 << 30) - 32;  // a padded row stays below 2^32 bytes

size_t align_up(size_t v, size_t a) { return (v + a - 1) / a * a; }

struct DeviceGuard {
  int prev = -1;
  bool ok = true;
  explicit DeviceGuard(int dev) {
    if (cudaGetDevice(&prev) != cudaSuccess) { prev = -1; }
    if (prev != dev) ok = (cudaSetDevice(dev) == cudaSuccess);
  }
  ~DeviceGuard() {
    int cur = -1;
    if (prev >= 0 && cudaGetDevice(&cur) == cudaSuccess && cur != prev) cudaSetDevice(prev);
  }
};

struct ResidentPlan {  // launch shape of resident_rounds_kernel
  bool ok = false;
  int threads = 0, grid = 0, G = 0, log2G = 0, draw_chunk = 0;
  size_t smem = 0;
  int64_t n_tiles = 0, max_rounds = 0;
  int64_t min_rounds = 1;  // rounds a call must run to repay loading and storing the tiles
};

struct FusedPlan {  // launch shape of fused_rounds_kernel
  bool ok = false;
  int threads = 0, grid = 0, max_rounds = 0;
  int slots = 0;  // rounds the kernel's table of draws is sized for
  size_t smem = 0;
  int64_t n_tiles = 0;
};

struct ClusterPlan {  // launch shape of cluster_rounds_kernel
  bool ok = false;
  int threads = 0, grid = 0, C = 0, rpc = 0, max_rounds = 0;
  size_t smem = 0;
  int64_t n_tiles = 0;
};

struct Layout {
  int64_t ld = 0, ldq = 0, nq = 0;  // row stride in elements / in 16-byte column groups; column groups in use
  int elem = 4, halves = 1;         // bytes per stored element; Philox blocks (4 elements) per column group
  size_t plane = 0;                 // bytes of one [M][ld] array
  size_t off_x0 = 0, off_x1 = 0, off_c = 0, off_thr = 0, off_last = 0, off_w = 0, off_trace = 0, off_wring = 0, off_tel = 0,
         off_partials = 0, off_ticket = 0, off_colpart = 0, off_coltick = 0, off_pipe_tel = 0, total = 0;
};

constexpr int kMaxGrid = 148 * 16;  // upper bound on resident CTAs of the round kernel
constexpr int64_t kMaxRoundsPerLaunch = 4096;  // rounds one cooperative launch runs at most
constexpr size_t kColPartBytes = (size_t)8 << 20;  // column partials of the row-split (short vector) shape
constexpr int kMaxChunks = 32;  // column chunks of a pipelined host round trip

Layout make_layout(int64_t M, int64_t d, int64_t trace_rounds, int storage) {
  Layout L;
  L.elem = storage == NETMAX_STORAGE_BF16 ? 2 : 4;
  L.halves = storage == NETMAX_STORAGE_BF16 ? 2 : 1;
  const int64_t per_group = 16 / L.elem;
  L.ld = (int64_t)align_up((size_t)d, (size_t)(128 / L.elem));  // rows start on 128-byte boundaries
  L.ldq = L.ld / per_group;
  L.nq = (d + per_group - 1) / per_group;
  size_t o = 0;
  auto take = [&](size_t bytes) { size_t at = o; o = align_up(o + bytes, 256); return at; };
  const size_t plane = (size_t)M * L.ld * L.elem;
  L.plane = plane;
  L.off_x0 = take(plane);
  L.off_x1 = take(plane);
  L.off_c = take(plane);
  L.off_thr = take((size_t)M * M * sizeof(uint32_t));
  L.off_last = take((size_t)M * sizeof(int32_t));
  L.off_w = take((size_t)M * M * sizeof(float));
  L.off_trace = take((size_t)trace_rounds * M * sizeof(int32_t));
  L.off_wring = take((size_t)trace_rounds * M * sizeof(float));  // pull weight of every draw in the trace ring
  L.off_tel = take((size_t)trace_rounds * 2 * sizeof(double));
  L.off_partials = take((size_t)kMaxGrid * 2 * sizeof(double) * kFusedMaxRounds);  // per round of a fused launch; two sets for multi-round launches
  L.off_ticket = take(256);
  L.off_colpart = take(kColPartBytes);
  L.off_coltick = take((size_t)kMaxGrid * sizeof(unsigned int));
  L.off_pipe_tel = take((size_t)kMaxChunks * trace_rounds * 2 * sizeof(double));  // per-chunk telemetry of a pipelined round trip
  L.total = o;
  return L;
}

}  // namespace

namespace netmax {
void set_global_error(const std::string& msg) { g_error = msg; }
}  // namespace netmax

struct netmax_ctx {
  int32_t M = 0;
  int64_t d = 0;
  uint32_t q_offset = 0;  // element_offset / 4: added to the column-group word of the counters
  Layout L;
  int device = 0;
  cudaStream_t stream = nullptr;
  bool own_memory = false;
  unsigned char* base = nullptr;
  int storage = NETMAX_STORAGE_F32;
  unsigned char *x[2] = {nullptr, nullptr}, *c = nullptr;  // [M][ld] fp32 or bfloat16, as `storage` says
  uint32_t* thr = nullptr;
  int32_t* last_nz = nullptr;
  float* wtab = nullptr;
  int32_t* trace = nullptr;
  float* wring = nullptr;
  double* tel = nullptr;
  double* partials = nullptr;
  unsigned int* ticket = nullptr;
  float4* colpart = nullptr;
  unsigned int* grid_barrier = nullptr;  // arrival counter of multi-round launches
  unsigned int* dev_error = nullptr;     // raised by a kernel whose bounded wait gave up
  bool cooperative = false;              // device supports cooperative launches
  uint32_t inject_absent_ctas = 0;       // test hook: applied to the next multi-round launch, then cleared
  double* measure_out = nullptr;         // device: (consensus, loss) of netmax_measure
  // host copies of the tables in force (the asynchronous timeline draws peers on the host)
  std::vector<uint32_t> h_thr;
  std::vector<int32_t> h_last;
  std::vector<float> h_w;
  std::vector<double> t_iter;  // iteration times derived from the link speeds in force
  // asynchronous timeline (one worker per global step)
  bool async_on = false;
  double beta = 0.0;
  double now = 0.0;
  int64_t steps = 0;
  std::vector<int64_t> local_n;
  std::vector<int32_t> pending_peer;
  std::vector<float> pending_weight;    // Eq. 16's weight for the pending iteration, under the policy it started with
  std::vector<double> pending_duration; // t_im of the pending iteration, under the times it started with
  std::vector<double> finish;
  // pending iterations ordered by (finish time, worker): exactly one entry per worker
  std::priority_queue<std::pair<double, int>, std::vector<std::pair<double, int>>, std::greater<std::pair<double, int>>> queue;
  std::vector<double> ema;
  std::vector<int64_t> ema_count;
  double monitor_period = 0.0, monitor_next = 0.0;  // Network Monitor on the simulated clock (0: off)
  int64_t monitor_refreshes = 0;
  int64_t ev_cap = 0;
  std::vector<int32_t> ev_worker, ev_peer;
  std::vector<int64_t> ev_n;
  std::vector<double> ev_time;
  unsigned int* coltick = nullptr;
  double* pipe_tel = nullptr;                      // [kMaxChunks][trace_rounds][2]
  cudaStream_t up_stream = nullptr, down_stream = nullptr;  // host round trips: uploads and downloads beside the context's stream
  int cur = 0;  // index of the buffer holding the current replicas
  int64_t rounds = 0;  // number of the next round (absolute)
  int64_t round0 = 0;  // number of the context's first round
  int64_t trace_rounds = 0;
  double alpha = 0, rho = 0, sigma = 0;
  double pull_weight = 0;  // > 0: fixed weight of every pull
  int objective = 1;
  uint64_t seed = 0;
  int policy_K = 20, policy_R = 20;
  double policy_rho_upper = 0.0;
  int fuse_rounds = 0;  // 0: automatic, 1: one launch per round, 2..kFusedMaxRounds: rounds per fused launch
  bool fused_planned = false;
  FusedPlan fused;
  bool resident_planned = false;
  ResidentPlan resident;
  bool cluster_planned = false;
  ClusterPlan cluster;
  PhiloxKeys keys;
  std::vector<double> P;      // policy in force
  std::vector<uint8_t> adj;   // link graph in force
  int sm_count = 148;
  int64_t launches = 0;
  std::string error;
};

namespace {

int fail(netmax_ctx* ctx, int code, const char* fmt, ...) {
  char buf[512];
  va_list ap;
  va_start(ap, fmt);
  vsnprintf(buf, sizeof buf, fmt, ap);
  va_end(ap);
  if (ctx) ctx->error = buf; else g_error = buf;
  return code;
}

#define NM_CUDA(ctx, call)                                                                         \
  do {                                                                                             \
    cudaError_t e_ = (call);                                                                       \
    if (e_ != cudaSuccess)                                                                         \
      return fail(ctx, e_ == cudaErrorMemoryAllocation ? NETMAX_OOM : NETMAX_CUDA_ERROR, "%s: %s", \
                  #call, cudaGetErrorString(e_));                                                  \
  } while (0)

// Link graph from speeds: d_im = 1 iff i != m and the speed is positive (symmetrised).
int build_adjacency(netmax_ctx* ctx, int32_t M, const double* speed, std::vector<uint8_t>& adj) {
  adj.assign((size_t)M * M, 0);
  for (int i = 0; i < M; ++i)
    for (int m = 0; m < M; ++m) {
      if (i == m) continue;
      if (!speed) { adj[(size_t)i * M + m] = 1; continue; }
      const double a = speed[(size_t)i * M + m], b = speed[(size_t)m * M + i];
      if (!std::isfinite(a) || !std::isfinite(b)) return fail(ctx, NETMAX_INVALID_ARG, "link speed (%d,%d) is not finite", i, m);
      adj[(size_t)i * M + m] = (a > 0.0 && b > 0.0) ? 1 : 0;
    }
  // connectivity (Assumption 1) by a depth-first walk from worker 0
  std::vector<int> stack{0};
  std::vector<uint8_t> seen(M, 0);
  seen[0] = 1;
  int count = 1;
  while (!stack.empty()) {
    const int v = stack.back();
    stack.pop_back();
    for (int m = 0; m < M; ++m)
      if (adj[(size_t)v * M + m] && !seen[m]) { seen[m] = 1; ++count; stack.push_back(m); }
  }
  if (count != M) return fail(ctx, NETMAX_NOT_CONNECTED, "link graph is not connected (%d of %d workers reachable)", count, M);
  return NETMAX_OK;
}

int validate_policy(netmax_ctx* ctx, int32_t M, const double* P, const std::vector<uint8_t>& adj) {
  for (int i = 0; i < M; ++i) {
    double sum = 0.0;
    for (int m = 0; m < M; ++m) {
      const double p = P[(size_t)i * M + m];
      if (!(p >= 0.0) || !std::isfinite(p)) return fail(ctx, NETMAX_BAD_PROB_ROW, "P[%d,%d] = %g is negative or not finite", i, m, p);
      if (p > 0.0 && m != i && !adj[(size_t)i * M + m])
        return fail(ctx, NETMAX_BAD_PROB_ROW, "P[%d,%d] > 0 on a missing link (Eq. 12)", i, m);
      sum += p;
    }
    if (std::fabs(sum - 1.0) > 1e-9) return fail(ctx, NETMAX_BAD_PROB_ROW, "row %d of P sums to %.12g", i, sum);
  }
  return NETMAX_OK;
}

// rho <= 0: the largest rho that keeps Eq. 11 (p_im > alpha rho (d_im + d_mi)) with a 1e-6 margin.
double default_rho(int32_t M, const double* P, const std::vector<uint8_t>& adj, double alpha) {
  double best = INFINITY;
  for (int i = 0; i < M; ++i)
    for (int m = 0; m < M; ++m) {
      const double p = P[(size_t)i * M + m];
      if (i == m || !(p > 0.0)) continue;
      const double dsum = (double)adj[(size_t)i * M + m] + (double)adj[(size_t)m * M + i];
      best = std::min(best, p / (alpha * dsum));
    }
  return std::isfinite(best) ? (1.0 - 1e-6) * best : 0.0;
}

// A caller's rho must keep Eq. 11, p_im >= alpha rho (d_im + d_mi) on every link in use (taken
// closed, as Algorithm 3's rows may sit on the floor): otherwise the pull weight of Eq. 16
// exceeds 1/2, entries of Y_P (Eq. 22) can turn negative and Theorem 3's lambda_2 < 1 is lost.
// With a fixed pull weight rho is unused and nothing is checked.
int check_rho(netmax_ctx* ctx, int32_t M, const double* P, const std::vector<uint8_t>& adj, double alpha, double rho,
              double pull_weight) {
  if (pull_weight > 0.0) return NETMAX_OK;
  for (int i = 0; i < M; ++i)
    for (int m = 0; m < M; ++m) {
      const double p = P[(size_t)i * M + m];
      if (i == m || !(p > 0.0)) continue;
      const double floor_im = alpha * rho * ((double)adj[(size_t)i * M + m] + (double)adj[(size_t)m * M + i]);
      if (floor_im > p * (1.0 + 1e-9))
        return fail(ctx, NETMAX_INVALID_ARG, "rho = %g breaks Eq. 11 on link (%d,%d): alpha rho (d_im + d_mi) = %g > p_im = %g",
                    rho, i, m, floor_im, p);
    }
  return NETMAX_OK;
}

// T_j = floor(cum_j 2^32 + 1/2) over the left-to-right double prefix sums of the row,
// non-decreasing, saturated, and pinned to the top from the last positive entry on.
void build_tables(int32_t M, const double* P, const std::vector<uint8_t>& adj, double alpha32, double rho,
                  double pull_weight, std::vector<uint32_t>& thr, std::vector<int32_t>& last_nz, std::vector<float>& w) {
  thr.resize((size_t)M * M);
  last_nz.resize(M);
  w.resize((size_t)M * M);
  for (int i = 0; i < M; ++i) {
    const double* p = P + (size_t)i * M;
    int32_t last = -1;
    for (int j = 0; j < M; ++j) if (p[j] > 0.0) last = j;
    last_nz[i] = last;
    double cum = 0.0;
    uint64_t prev = 0;
    for (int j = 0; j < M; ++j) {
      cum += p[j];
      uint64_t t = (uint64_t)std::floor(cum * 4294967296.0 + 0.5);
      t = std::max(t, prev);
      if (t > 0xFFFFFFFFull || j >= last) t = 0xFFFFFFFFull;
      thr[(size_t)i * M + j] = (uint32_t)t;
      prev = t;
      float wv = 0.0f;
      if (j != i && p[j] > 0.0) {
        const double dsum = (double)adj[(size_t)i * M + j] + (double)adj[(size_t)j * M + i];
        wv = pull_weight > 0.0 ? (float)pull_weight                         // fixed-weight averaging
                               : (float)(alpha32 * rho * dsum / (2.0 * p[j]));  // alpha rho gamma_im (Eq. 16)
      }
      w[(size_t)i * M + j] = wv;
    }
  }
}

int upload_policy(netmax_ctx* ctx) {
  std::vector<uint32_t>& thr = ctx->h_thr;
  std::vector<int32_t>& last = ctx->h_last;
  std::vector<float>& w = ctx->h_w;
  build_tables(ctx->M, ctx->P.data(), ctx->adj, (double)(float)ctx->alpha, ctx->rho, ctx->pull_weight, thr, last, w);
  // pageable sources: the copies are complete (staged) when these calls return
  NM_CUDA(ctx, cudaMemcpyAsync(ctx->thr, thr.data(), thr.size() * sizeof(uint32_t), cudaMemcpyHostToDevice, ctx->stream));
  NM_CUDA(ctx, cudaMemcpyAsync(ctx->last_nz, last.data(), last.size() * sizeof(int32_t), cudaMemcpyHostToDevice, ctx->stream));
  NM_CUDA(ctx, cudaMemcpyAsync(ctx->wtab, w.data(), w.size() * sizeof(float), cudaMemcpyHostToDevice, ctx->stream));
  NM_CUDA(ctx, cudaStreamSynchronize(ctx->stream));
  return NETMAX_OK;
}

// Iteration times of the link speeds in force (equal speeds when none were given).
int refresh_iteration_times(netmax_ctx* ctx, const double* speed) {
  const int32_t M = ctx->M;
  std::vector<double> flat;
  if (!speed) {
    flat.assign((size_t)M * M, 1.0);
    speed = flat.data();
  }
  std::vector<uint8_t> adj2((size_t)M * M);
  ctx->t_iter.assign((size_t)M * M, 0.0);
  int rc = netmax_iteration_times(M, ctx->d, speed, ctx->t_iter.data(), adj2.data());
  if (rc) return fail(ctx, rc, "%s", netmax_last_error(nullptr));
  return NETMAX_OK;
}

// Chooses P and rho: the caller's, or Algorithm 3's.  speed == NULL keeps the iteration times
// in force (or, at creation, takes equal speeds).
int resolve_policy(netmax_ctx* ctx, const double* speed, const double* prob, double rho) {
  const int32_t M = ctx->M;
  if (speed || ctx->t_iter.empty()) {
    int rc = refresh_iteration_times(ctx, speed);
    if (rc) return rc;
  }
  if (prob) {
    int rc = validate_policy(ctx, M, prob, ctx->adj);
    if (rc) return rc;
    if (rho > 0.0) {
      rc = check_rho(ctx, M, prob, ctx->adj, ctx->alpha, rho, ctx->pull_weight);
      if (rc) return rc;
    }
    ctx->P.assign(prob, prob + (size_t)M * M);
    ctx->rho = rho > 0.0 ? rho : default_rho(M, prob, ctx->adj, ctx->alpha);
    return NETMAX_OK;
  }
  ctx->P.assign((size_t)M * M, 0.0);
  double rho_sel = 0.0;
  if (ctx->pull_weight > 0.0) {
    // constant pull weight: Algorithm 3 in the form the paper's extension section prescribes (a floor
    // on p_im in rho's place, balanced columns); rho plays no part in the update
    double floor_sel = 0.0;
    int rc = netmax_policy_generate_fixed_weight(M, ctx->t_iter.data(), ctx->adj.data(), ctx->pull_weight, ctx->policy_K,
                                                 ctx->policy_R, ctx->policy_rho_upper, ctx->P.data(), &floor_sel, nullptr);
    if (rc) return fail(ctx, rc, "%s", netmax_last_error(nullptr));
    ctx->rho = rho > 0.0 ? rho : 0.0;
    return NETMAX_OK;
  }
  // Algorithm 3: on the device from 512 workers up (where the host generator takes seconds)
  int ndev = 0;
  const bool on_device = M >= 512 && cudaGetDeviceCount(&ndev) == cudaSuccess && ctx->device < ndev;
  if (!on_device) cudaGetLastError();
  int rc = on_device ? netmax_policy_generate_device(M, ctx->t_iter.data(), ctx->adj.data(), ctx->alpha, ctx->policy_K,
                                                     ctx->policy_R, ctx->policy_rho_upper, ctx->device, ctx->stream, ctx->P.data(), &rho_sel, nullptr)
                     : netmax_policy_generate_ex(M, ctx->t_iter.data(), ctx->adj.data(), ctx->alpha, ctx->policy_K,
                                                 ctx->policy_R, ctx->policy_rho_upper, ctx->P.data(), &rho_sel, nullptr);
  if (rc) return fail(ctx, rc, "%s", netmax_last_error(nullptr));
  if (rho > 0.0) {  // the caller's rho with Algorithm 3's P: it must still respect that P
    rc = check_rho(ctx, M, ctx->P.data(), ctx->adj, ctx->alpha, rho, ctx->pull_weight);
    if (rc) return rc;
  }
  ctx->rho = rho > 0.0 ? rho : rho_sel;
  return NETMAX_OK;
}

int launch_init(netmax_ctx* ctx, unsigned char* dst, double stddev, uint32_t tag) {
  NM_CUDA(ctx, cudaMemsetAsync(dst, 0, ctx->L.plane, ctx->stream));
  if (stddev == 0.0) return NETMAX_OK;
  InitParams p;
  p.dst = reinterpret_cast<float4*>(dst);
  p.ldq = ctx->L.ldq;
  p.nq = ctx->L.nq;
  p.M = ctx->M;
  p.tail = (int32_t)(ctx->d % (4 * ctx->L.halves));
  p.stddev = (float)stddev;
  p.tag = tag;
  p.q_offset = ctx->q_offset;
  p.keys = ctx->keys;
  const int64_t total = (int64_t)ctx->M * ctx->L.nq;
  const int grid = (int)std::min<int64_t>((total + kThreads - 1) / kThreads, (int64_t)ctx->sm_count * 16);
  if (ctx->L.halves == 2) init_normal_kernel<2><<<grid, kThreads, 0, ctx->stream>>>(p);
  else init_normal_kernel<1><<<grid, kThreads, 0, ctx->stream>>>(p);
  ctx->launches += 1;
  NM_CUDA(ctx, cudaGetLastError());
  return NETMAX_OK;
}

int launch_sampler(netmax_ctx* ctx, uint64_t first_round, int64_t n_rounds, int32_t* out, float* w_out, int64_t slot0,
                   int64_t ring) {
  if (n_rounds <= 0) return NETMAX_OK;
  SampleParams p;
  p.thresholds = ctx->thr;
  p.last_nz = ctx->last_nz;
  p.out = out;
  p.w_out = w_out;
  p.wtab = ctx->wtab;
  p.slot0 = slot0;
  p.ring = ring;
  p.first_round = first_round;
  p.n_rounds = n_rounds;
  p.M = ctx->M;
  p.keys = ctx->keys;
  const int64_t total = n_rounds * (int64_t)ctx->M;
  const int grid = (int)std::min<int64_t>((total + kThreads - 1) / kThreads, (int64_t)ctx->sm_count * 32);
  sample_peers_kernel<<<grid, kThreads, 0, ctx->stream>>>(p);
  ctx->launches += 1;
  NM_CUDA(ctx, cudaGetLastError());
  return NETMAX_OK;
}

struct RoundPlan {
  int cg = kThreads, rl = 1, rg = 1, rows_per_group = 0;
  bool short_vectors = false;  // fewer than two streaming tiles per SM: the L2-resident shape
  int grid = 1;
  size_t smem = 0;
  int64_t n_tiles = 0;
};

using RoundKernel = void (*)(const RoundParams);

using StepKernel = void (*)(const StepParams);

// halves: 1 for fp32 state, 2 for bfloat16 state (Philox blocks per 16-byte column group)
template <int kHalves>
StepKernel pick_step_kernel_h(int objective) {
  return objective == 1 ? step_kernel<1, true, kHalves> : step_kernel<0, true, kHalves>;
}
StepKernel pick_step_kernel(int objective, int halves) {
  return halves == 2 ? pick_step_kernel_h<2>(objective) : pick_step_kernel_h<1>(objective);
}

template <int kHalves>
RoundKernel pick_kernel_h(int objective, bool short_vectors) {
  if (objective == 2) return short_vectors ? round_kernel<2, true, 4, kHalves> : round_kernel<2, true, 1, kHalves>;
  if (short_vectors) return objective == 1 ? round_kernel<1, true, 4, kHalves> : round_kernel<0, true, 4, kHalves>;
#ifdef NETMAX_BF16_LONG_RIF
  if (kHalves == 2) return objective == 1 ? round_kernel<1, true, NETMAX_BF16_LONG_RIF, kHalves> : round_kernel<0, true, NETMAX_BF16_LONG_RIF, kHalves>;
#endif
  return objective == 1 ? round_kernel<1, true, 1, kHalves> : round_kernel<0, true, 1, kHalves>;
}
RoundKernel pick_kernel(int objective, bool short_vectors, int halves) {
  return halves == 2 ? pick_kernel_h<2>(objective, short_vectors) : pick_kernel_h<1>(objective, short_vectors);
}

using MultiRoundKernel = void (*)(const MultiRoundParams);

MultiRoundKernel pick_multi_kernel(int objective, int halves) {
  if (halves == 2) return objective == 1 ? multi_round_kernel<1, true, 2> : multi_round_kernel<0, true, 2>;
  return objective == 1 ? multi_round_kernel<1, true, 1> : multi_round_kernel<0, true, 1>;
}

using FusedKernel = void (*)(const FusedParams);

template <int kRounds>
FusedKernel pick_fused_kernel_r(int objective, int halves) {
  if (halves == 2) return objective == 1 ? fused_rounds_kernel<1, true, true, kRounds> : fused_rounds_kernel<0, true, true, kRounds>;
  return objective == 1 ? fused_rounds_kernel<1, true, false, kRounds> : fused_rounds_kernel<0, true, false, kRounds>;
}
// The instance for launches of `rounds` rounds (both instances share one shared-memory layout, FusedParams::slots).
FusedKernel pick_fused_kernel(int objective, int halves, int rounds) {
  return rounds <= 4 ? pick_fused_kernel_r<4>(objective, halves) : pick_fused_kernel_r<kFusedMaxRounds>(objective, halves);
}

using ResidentKernel = void (*)(const ResidentParams);

ResidentKernel pick_resident_kernel(int objective, int halves) {
  if (halves == 2) return objective == 1 ? resident_rounds_kernel<1, true, true> : resident_rounds_kernel<0, true, true>;
  return objective == 1 ? resident_rounds_kernel<1, true, false> : resident_rounds_kernel<0, true, false>;
}

// The kernels' noise scale: sigma (at its fp32 rounding, the value the update is defined with)
// times the constant factor sqrt(2 ln 2) of the Box-Muller radius, which the fast normal generator
// leaves out, rounded once to fp32.
float noise_scale(const netmax_ctx* ctx) { return (float)((double)(float)ctx->sigma * kNormalScale); }

int floor_pow2(int64_t v) {
  int r = 1;
  while ((int64_t)r * 2 <= v) r *= 2;
  return r;
}

// Tile shape.  Long vectors: all M rows x cg column groups, cg the largest power of two
// (<= 256 threads' worth, i.e. 4 KB of a row) that keeps the tile's share of x within 96 KB, so
// that a row fetched for its own update is still in cache when another row pulls it as a peer
// (measured optimum on cfg 2-4: wider tiles stream better until the peer reads start to miss).
// Short vectors (fewer than two such tiles per SM; everything is L2-resident then): 128-byte
// column segments where M allows, no idle row lanes, and the rows split into rg groups so that
// about two CTAs per SM have work.  The same shape serves many workers with vectors of any length:
// beyond 768 rows the 96 KB rule leaves a tile less than 128 bytes of every row, and a stream of
// 64- or 16-byte pieces costs more than peer rows that come from L2 instead of L1 (4096 x 4096
// elements: 135 us per round with 16-byte pieces, 34 with 128-byte pieces and two row groups;
// 1024 x 65536: 250 against 184).
int plan_round(netmax_ctx* ctx, RoundPlan& plan, int objective) {
  const int64_t M = ctx->M, nq = ctx->L.nq;
  const int64_t target = 2 * (int64_t)ctx->sm_count;  // the short-vector kernel runs 2 CTAs per SM
  int cg = kThreads;
  while (cg > 1 && (int64_t)cg * 16 * M > 96 * 1024) cg >>= 1;
  int rg = 1;
  if ((nq + cg - 1) / cg < 2 * (int64_t)ctx->sm_count || kThreads / cg > M || cg < 8) {
    plan.short_vectors = true;
    // Candidates in order of preference; the score is the number of CTAs with work, up to the target.
    // First among segments of at least 128 bytes only: a narrower one that happens to give more CTAs
    // loses more at the DRAM pins than it wins (8192 x 2048 elements: 144 us per round with 16-byte
    // pieces and 512 CTAs, 50 with 256-byte pieces and 256 CTAs).  With more workers than resident
    // columns can hold, this kernel is the one that runs by default, and 256-byte pieces measured
    // best there (8192 x 2048: 50 against 55 us; 16384 x 1024: 73 against 84).
    static const int wide_first[] = {8, 16, 32, 64, 128, 256};
    static const int wide_first_large[] = {16, 8, 32, 64, 128, 256};
    static const int any_width[] = {8, 4, 2, 16, 32, 64, 128, 256, 1};
    int64_t best_score = -1;
    auto consider = [&](int cand) {
      const int rl = kThreads / cand;
      if (rl > M && cand != kThreads) return;  // row lanes without rows
      const int64_t nct = (nq + cand - 1) / cand;
      int g = (int)std::min<int64_t>(std::min<int64_t>(32, std::max<int64_t>(1, M / rl)), floor_pow2(std::max<int64_t>(1, target / nct)));
      while (g > 1 && (size_t)nct * g * cand * 32 * ctx->L.halves > kColPartBytes) g >>= 1;
      if (nct * g > kMaxGrid) return;
      const int64_t score = std::min<int64_t>(nct * g, target);
      if (score > best_score) {
        best_score = score;
        cg = cand;
        rg = g;
      }
    };
    for (int cand : (M > 4700 ? wide_first_large : wide_first)) consider(cand);
    if (best_score * 20 < target * 17) {  // fewer than 85 % of the CTAs the SMs can hold: narrower pieces may do better
      best_score = -1;
      for (int cand : any_width) consider(cand);
    }
  }
  plan.cg = cg;
  plan.rl = kThreads / cg;
  plan.rg = rg;
  plan.rows_per_group = (int)((M + rg - 1) / rg);
  plan.n_tiles = (nq + cg - 1) / cg * rg;
  plan.smem = align_up((size_t)M * 8, 16) + (plan.rl > 1 ? (size_t)kThreads * 32 * ctx->L.halves : 0) + 64 * sizeof(double);
  RoundKernel k = pick_kernel(objective, plan.short_vectors, ctx->L.halves);
  // (the kernels also hold a little static shared memory, so the opt-in is needed somewhat below 48 KB of dynamic)
  if (plan.smem > 40 * 1024)
    NM_CUDA(ctx, cudaFuncSetAttribute(k, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)plan.smem));
  int per_sm = 0;
  NM_CUDA(ctx, cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, k, kThreads, plan.smem));
  if (per_sm < 1) return fail(ctx, NETMAX_CUDA_ERROR, "round kernel does not fit on an SM (smem %zu)", plan.smem);
  if (plan.short_vectors && ctx->cooperative) {  // the multi-round kernel needs all of its CTAs resident
    MultiRoundKernel mk = pick_multi_kernel(objective == 2 ? 0 : objective, ctx->L.halves);
    if (plan.smem > 40 * 1024)
      NM_CUDA(ctx, cudaFuncSetAttribute(mk, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)plan.smem));
    int per_sm_multi = 0;
    NM_CUDA(ctx, cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm_multi, mk, kThreads, plan.smem));
    per_sm = std::min(per_sm, per_sm_multi);
    if (per_sm < 1) return fail(ctx, NETMAX_CUDA_ERROR, "multi-round kernel does not fit on an SM (smem %zu)", plan.smem);
  }
  plan.grid = (int)std::min<int64_t>(plan.n_tiles, std::min<int64_t>((int64_t)per_sm * ctx->sm_count, kMaxGrid));
  return NETMAX_OK;
}

// Rounds whose draws the resident kernel stages in shared memory at a time: about 8 KB worth
// for up to 512 workers, none beyond (threads then fetch the draws of their own rows).
int resident_draw_chunk(int64_t M) { return M <= 512 ? (int)std::max<int64_t>(2, 1024 / M) : 0; }

size_t resident_smem(int64_t M, int threads, int G) {
  return (size_t)48 * M * G + 2 * sizeof(float) * resident_scratch_floats(threads, G) + 128 * sizeof(float) +
         (size_t)resident_draw_chunk(M) * M * 8;
}

// Short vectors whose M rows of at least one column group fit in a CTA's shared memory run all
// rounds of a call on resident columns (resident_rounds_kernel).  Small M: a thread per column
// group, as few threads per CTA as keep the CTA count within a few per SM (the problem is
// latency-bound: spread it over the SMs).  Larger M: G column groups per CTA, the rows of each
// split over the threads; G as large as fits, but no larger than leaves every SM a tile.
int plan_resident_uncached(netmax_ctx* ctx, const RoundPlan& plan, ResidentPlan& f) {
  f = ResidentPlan();
  if (!plan.short_vectors) return NETMAX_OK;
  const int64_t M = ctx->M, nq = (ctx->d + 3) / 4;
  const size_t limit = (size_t)224 * 1024;
  int threads = 0, G = 0;
  if (resident_smem(M, 32, 32) <= (size_t)100 * 1024) {
    // small M.  The problem is latency-bound: give a thread as few rows as still leaves about two
    // warps per scheduler busy, i.e. split the rows of a group over RL lanes (a power of two)
    const int64_t target_threads = (int64_t)ctx->sm_count * 256;
    const int64_t rows_per_thread = std::max<int64_t>(1, M * nq / target_threads);
    int RL = 1;
    while (RL < 32 && RL < M && (M + RL - 1) / RL > rows_per_thread) RL <<= 1;
    for (int cand : {32, 64, 128, 256}) {
      const int g = cand / RL;
      if (g < 1 || (RL > 1 && g > 32)) break;
      if (resident_smem(M, cand, g) > (size_t)100 * 1024) break;
      threads = cand;
      G = g;
      if ((nq + g - 1) / g <= (int64_t)8 * ctx->sm_count) break;
    }
  }
  if (threads == 0) {  // rows of a group split over the threads
    G = 32;
    while (G > 1 && (size_t)48 * M * G > (size_t)190 * 1024) G >>= 1;
    while (G > 1 && (nq + G - 1) / G < ctx->sm_count) G >>= 1;
    threads = (int)std::min<int64_t>(512, std::max<int64_t>(64, floor_pow2(M * G / 2)));
    threads = std::max(threads, G);
    if (resident_smem(M, threads, G) > limit) return NETMAX_OK;
  }
  f.threads = threads;
  f.G = G;
  f.log2G = 0;
  while ((1 << f.log2G) < G) ++f.log2G;
  f.draw_chunk = (int)std::min<int64_t>(resident_draw_chunk(M), ctx->trace_rounds);
  f.smem = resident_smem(M, threads, G);
  f.n_tiles = (nq + G - 1) / G;
  f.max_rounds = std::max<int64_t>(1, std::min<int64_t>(kMaxRoundsPerLaunch, (int64_t)(kColPartBytes / 16) / f.n_tiles));
  // A call pays once for bringing its tiles on chip and back -- narrow columns of all M rows, which stream
  // badly (about 1.1 TB/s with one column group per tile) -- and then saves on every round.  Rounds from
  // which that paid in measurements (us per round, resident columns against the per-round kernels, calls of
  // 1 / 2 / 4 / many rounds): 4 x 4096 elements 13.4 / 7.0 / 4.1 / 0.9 against 10.3 / 8.2 / 6.0 / 3.8;
  // 4096 x 1024: 57 / 33 / 21 / 9.5 against 29 / 23 / 19 / 16; 4096 x 4096: 219 / 128 / 80 / 33 against
  // 66 / 61 / 58 / 54; 4096 x 16384: 837 / 492 / 310 / 136 against 195 / 192 / 190 / 188.
  const int64_t elements = M * ctx->d;
  f.min_rounds = elements <= ((int64_t)1 << 20) ? 2 : elements <= ((int64_t)1 << 22) ? 6 : elements <= ((int64_t)1 << 24) ? 8 : 16;
  ResidentKernel k = pick_resident_kernel(ctx->objective, ctx->L.halves);
  NM_CUDA(ctx, cudaFuncSetAttribute(k, cudaFuncAttributePreferredSharedMemoryCarveout, (int)cudaSharedmemCarveoutMaxShared));
  NM_CUDA(ctx, cudaFuncSetAttribute(k, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)f.smem));
  int per_sm = 0;
  NM_CUDA(ctx, cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, k, threads, f.smem));
  if (per_sm < 1) return NETMAX_OK;
  f.grid = (int)std::min<int64_t>(f.n_tiles, (int64_t)per_sm * ctx->sm_count);
  f.ok = true;
  return NETMAX_OK;
}

int plan_resident(netmax_ctx* ctx, const RoundPlan& plan, ResidentPlan& f) {
  if (ctx->resident_planned) {
    f = ctx->resident;
    return NETMAX_OK;
  }
  int rc = plan_resident_uncached(ctx, plan, f);
  if (rc == NETMAX_OK) {
    ctx->resident = f;
    ctx->resident_planned = true;
  }
  return rc;
}

int plan_fused_uncached(netmax_ctx* ctx, const RoundPlan& plan, FusedPlan& f) {
  f = FusedPlan();
  if (ctx->fuse_rounds == 1 || plan.short_vectors) return NETMAX_OK;
  const int64_t M = ctx->M;
  const int want_rounds = ctx->fuse_rounds >= 2 ? std::min(ctx->fuse_rounds, kFusedMaxRounds) : kFusedMaxRounds;
  // 256 or 128 threads per CTA (a multiple of four warps keeps the SM's four schedulers evenly
  // loaded: 3 x 96 threads measured 587 us per cfg3 round against 508 for 2 x 128), whichever
  // puts more threads on an SM with at least two CTAs (one loads its tile while the other
  // computes; M = 16: 1 x 256 threads 529 us).  Every thread needs 48 M bytes of shared memory,
  // and the kernel's ~100 registers cap an SM at 16 warps (capping it at 96 or 80 registers for
  // 18-20 warps measured slower: 135 and 157 us against 128 per cfg2 round).  Beyond 18 workers only
  // 64-thread CTAs fit, three per SM up to M = 24 and two up to M = 36: four to six warps per SM, and
  // still 9 to 21 % faster than the same rows split over a cluster (M x 4,000,002 elements, us per round:
  // M = 20: 132 against 144, 28: 182 against 214, 36: 227 against 287) -- no barrier, no pull that leaves
  // the CTA.  A single such CTA per SM (M = 37 ... 73) is slower than the cluster shape (M = 40: 330
  // against 309), so the kernel is used down to 128 threads per SM.
  FusedKernel k = pick_fused_kernel(ctx->objective, ctx->L.halves, kFusedMaxRounds);  // (the instance with more registers)
  NM_CUDA(ctx, cudaFuncSetAttribute(k, cudaFuncAttributePreferredSharedMemoryCarveout, (int)cudaSharedmemCarveoutMaxShared));
  NM_CUDA(ctx, cudaFuncSetAttribute(pick_fused_kernel(ctx->objective, ctx->L.halves, 4), cudaFuncAttributePreferredSharedMemoryCarveout,
                                    (int)cudaSharedmemCarveoutMaxShared));
  // The table of draws at the head of the shared memory takes 16 M bytes per round of the launch: room for
  // as many rounds as were asked for, unless the smaller table of four rounds lets more threads live on an SM
  // (M = 36: the last kilobytes decide between two CTAs and one).
  int threads = 0, per_sm = 0, slots = 0;
  size_t fixed = 0;
  for (int rounds : {want_rounds, std::min(want_rounds, 4)}) {
    const size_t fixed_r = align_up((size_t)rounds * M * 16, 128) + 64 * sizeof(double);
    int threads_r = 0, per_sm_r = 0;
    for (int cand : {256, 128, 64}) {
      const size_t smem = fixed_r + (size_t)48 * M * cand;
      if (smem > (size_t)227 * 1024) continue;
      NM_CUDA(ctx, cudaFuncSetAttribute(k, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
      int n = 0;
      NM_CUDA(ctx, cudaOccupancyMaxActiveBlocksPerMultiprocessor(&n, k, cand, smem));
      const bool better = (n >= 2) != (per_sm_r >= 2) ? n >= 2 : n * cand > per_sm_r * threads_r;
      if (n >= 1 && (threads_r == 0 || better)) { threads_r = cand; per_sm_r = n; }
    }
    if (threads_r != 0 && per_sm_r * threads_r > per_sm * threads) {
      threads = threads_r;
      per_sm = per_sm_r;
      slots = rounds;
      fixed = fixed_r;
    }
  }
  if (threads == 0 || per_sm * threads < 128) return NETMAX_OK;  // too few warps to hide the arithmetic latency
  f.threads = threads;
  f.slots = slots;
  f.smem = fixed + (size_t)48 * M * threads;
  f.max_rounds = slots;
  f.n_tiles = ((ctx->d + 3) / 4 + threads - 1) / threads;
  NM_CUDA(ctx, cudaFuncSetAttribute(k, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)f.smem));
  f.grid = (int)std::min<int64_t>(f.n_tiles, std::min<int64_t>((int64_t)per_sm * ctx->sm_count, kMaxGrid));
  f.ok = true;
  return NETMAX_OK;
}

// Several rounds per launch over shared-memory-resident tiles (fused_rounds_kernel): long
// vectors, fp32 state, and few enough workers that the slabs (48 bytes per worker and thread)
// of at least eight warps fit on an SM.  The plan is kept until fuse_rounds changes.
int plan_fused(netmax_ctx* ctx, const RoundPlan& plan, FusedPlan& f) {
  if (ctx->fused_planned) {
    f = ctx->fused;
    return NETMAX_OK;
  }
  int rc = plan_fused_uncached(ctx, plan, f);
  if (rc == NETMAX_OK) {
    ctx->fused = f;
    ctx->fused_planned = true;
  }
  return rc;
}

using ClusterKernel = void (*)(const ClusterParams);

ClusterKernel pick_cluster_kernel(int objective) {
  return objective == 1 ? cluster_rounds_kernel<1, true> : cluster_rounds_kernel<0, true>;
}

#ifndef NETMAX_CLUSTER_SIZE
#define NETMAX_CLUSTER_SIZE 0  // 0: chosen from the number of workers (cluster_size below); 2, 4, 8: fixed
#endif
#ifndef NETMAX_CLUSTER_THREADS
#define NETMAX_CLUSTER_THREADS 0  // 0: the smallest of 64, 128, 256 threads per CTA whose slabs fit
#endif

size_t cluster_smem(int rpc, int threads) {
  return align_up((size_t)kClusterMaxRounds * rpc * 16, 128) + (size_t)3 * rpc * threads * 16 + (size_t)2 * threads * 16 +
         64 * sizeof(double);
}

// CTAs per cluster for M workers, 0 for "one launch per round instead".  A CTA needs enough rows between
// two cluster barriers to pay for them (a barrier costs about 1,500 cycles even for the last CTA to arrive)
// and few enough that eight CTAs of 64 threads still fit on an SM; a ragged last CTA makes the others
// wait; smaller clusters have cheaper barriers and more pulls that stay in the CTA.  The sweet spot is
// eight rows per CTA in as few CTAs as possible, but the details do not follow a formula, so the size is
// the one measured fastest: every size from 2 to 8, M x 2,000,002 elements, four rounds per launch against
// one launch per round (profiles/cluster_rounds_kernel_cfg4.md has the sweep).  Entered only where the
// cluster shape took less than 0.97 of the per-round time: 0.83-0.93 for M = 37 ... 66, 0.92-0.97 for most
// of 68 ... 88, nothing beyond.  Clusters of 16 (not portable) fit too few at a time: 1.3-2.1 x slower.
// `forced` (the caller asked for fused rounds): any M up to 8 x 18 rows gets the table's size or else the
// one whose CTAs hold closest to eight rows.
int cluster_size(int64_t M, bool forced) {
  if (NETMAX_CLUSTER_SIZE != 0) return NETMAX_CLUSTER_SIZE;
  static const unsigned char by_workers[] = {
      // M = 37 ... 88 (up to 36 workers fused_rounds_kernel holds all rows in one CTA)
      5, 5, 5, 5, 4, 4, 4, 4, 5, 6, 6, 6, 5, 5, 5, 5, 5, 5, 5, 7, 6, 6, 6, 6, 8, 8,
      8, 8, 6, 6, 0, 4, 7, 7, 0, 7, 7, 7, 7, 7, 7, 0, 0, 8, 0, 0, 0, 8, 8, 8, 8, 8};
  if (M >= 37 && M < 37 + (int64_t)sizeof by_workers && by_workers[M - 37] != 0) return by_workers[M - 37];
  if (!forced) return 0;
  int best = 0;
  int64_t best_gap = 0;
  for (int c = 2; c <= 8; ++c) {
    const int64_t rpc = (M + c - 1) / c, gap = rpc > 8 ? rpc - 8 : 8 - rpc;
    if (rpc <= 18 && (best == 0 || gap < best_gap)) {
      best = c;
      best_gap = gap;
    }
  }
  return best;
}

// Long fp32 vectors with more workers than fused_rounds_kernel can hold per thread (M > 36): the rows
// of a tile are split over the CTAs of a cluster (cluster_rounds_kernel), up to 18 rows per CTA.
int plan_cluster_uncached(netmax_ctx* ctx, const RoundPlan& plan, const FusedPlan& fused, ClusterPlan& f) {
  f = ClusterPlan();
  if (ctx->fuse_rounds == 1 || plan.short_vectors || fused.ok || ctx->storage != NETMAX_STORAGE_F32) return NETMAX_OK;
  const int64_t M = ctx->M;
  const int C = cluster_size(M, ctx->fuse_rounds >= 2);
  if (C == 0) return NETMAX_OK;
  const int rpc = (int)((M + C - 1) / C);
  if (rpc > 18) return NETMAX_OK;
  ClusterKernel k = pick_cluster_kernel(ctx->objective);
  NM_CUDA(ctx, cudaFuncSetAttribute(k, cudaFuncAttributePreferredSharedMemoryCarveout, (int)cudaSharedmemCarveoutMaxShared));
  // Small CTAs, many per SM: a CTA that waits at the cluster barrier leaves its SM to the others.  Measured
  // on 64 x 11.2 M elements, clusters of 8: 64 threads (8 CTAs per SM) 1.39 ms per round, 128 threads 1.43,
  // 256 threads 1.69, 32 threads 2.08; clusters of 4 with 64 threads 1.54 (one launch per round: 1.62).
  for (int cand : {64, 128, 256}) {
    if (NETMAX_CLUSTER_THREADS != 0 && cand != NETMAX_CLUSTER_THREADS) continue;
    const size_t smem = cluster_smem(rpc, cand);
    if (smem > (size_t)113 * 1024) continue;  // at least two CTAs per SM
    NM_CUDA(ctx, cudaFuncSetAttribute(k, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)(C * ctx->sm_count));
    cfg.blockDim = dim3((unsigned)cand);
    cfg.dynamicSmemBytes = smem;
    cudaLaunchAttribute attr;
    attr.id = cudaLaunchAttributeClusterDimension;
    attr.val.clusterDim.x = (unsigned)C;
    attr.val.clusterDim.y = 1;
    attr.val.clusterDim.z = 1;
    cfg.attrs = &attr;
    cfg.numAttrs = 1;
    int clusters = 0;
    if (cudaOccupancyMaxActiveClusters(&clusters, k, &cfg) != cudaSuccess) { cudaGetLastError(); continue; }
    if (clusters < 1) continue;
    f.threads = cand;
    f.C = C;
    f.rpc = rpc;
    f.smem = smem;
    f.n_tiles = ((ctx->d + 3) / 4 + cand - 1) / cand;
    f.max_rounds = ctx->fuse_rounds >= 2 ? std::min(ctx->fuse_rounds, kClusterMaxRounds) : kClusterMaxRounds;
    f.grid = (int)std::min<int64_t>(f.n_tiles, (int64_t)clusters) * C;
    f.ok = true;
    break;
  }
  return NETMAX_OK;
}

int plan_cluster(netmax_ctx* ctx, const RoundPlan& plan, const FusedPlan& fused, ClusterPlan& f) {
  if (ctx->cluster_planned) {
    f = ctx->cluster;
    return NETMAX_OK;
  }
  int rc = plan_cluster_uncached(ctx, plan, fused, f);
  if (rc == NETMAX_OK) {
    ctx->cluster = f;
    ctx->cluster_planned = true;
  }
  return rc;
}

// What every launch of the round kernels shares: buffers, tile shape, step sizes, keys.
RoundParams make_round_params(const netmax_ctx* ctx, const RoundPlan& plan) {
  RoundParams p;
  std::memset(&p, 0, sizeof p);
  p.c = reinterpret_cast<const float4*>(ctx->c);
  p.wtab = ctx->wtab;
  p.partials = ctx->partials;
  p.ticket = ctx->ticket;
  p.ldq = ctx->L.ldq;
  p.row_bytes = (uint32_t)(ctx->L.ld * ctx->L.elem);
  p.nq = ctx->L.nq;
  p.n_tiles = plan.n_tiles;
  p.M = ctx->M;
  p.tail = (int32_t)(ctx->d % (4 * ctx->L.halves));
  p.cg = plan.cg;
  p.rl = plan.rl;
  p.rg = plan.rg;
  p.rows_per_group = plan.rows_per_group;
  p.colpart = ctx->colpart;
  p.coltick = ctx->coltick;
  p.alpha = (float)ctx->alpha;
  p.sigma = noise_scale(ctx);
  p.inv_M = 1.0f / (float)ctx->M;
  p.q_offset = ctx->q_offset;
  p.keys = ctx->keys;
  return p;
}

// A range of column groups (four fp32 elements each) of every replica: the whole vector, or one
// chunk of a pipelined host round trip.  Given the draws, columns evolve independently, so the
// kernels run on a range exactly as on the whole: shifted base pointers, the range's group count,
// and the Philox block offset moved along.
struct ColumnRange {
  int64_t q0 = 0, nq4 = 0;  // first group and number of groups (four elements each)
  int32_t tail4 = 0;        // live elements of the range's last group (0: all four); non-zero only at the end of the rows
  bool whole = true;        // the whole vector (the only form bfloat16 state takes)
};

// Enqueues rounds [first, first + n) -- their draws are in the trace ring -- for one column range on
// `stream`: up to four rounds per launch where tiles stay resident (fused_rounds_kernel, or
// cluster_rounds_kernel for more workers), else one launch per round.  `cur` is the buffer that holds
// the range's values at round `first`; it is flipped launch by launch.  Telemetry of the range goes
// to tel (ring-indexed like the context's).
int launch_long_rounds(netmax_ctx* ctx, cudaStream_t stream, const RoundPlan& plan, const FusedPlan& fused,
                       const ClusterPlan& cluster, RoundParams p, const ColumnRange& range, double* tel, uint64_t first,
                       int64_t n, int& cur) {
  RoundKernel kernel = pick_kernel(ctx->objective, plan.short_vectors, ctx->L.halves);
  const size_t shift = range.whole ? 0 : (size_t)range.q0 * 16;  // bytes into every row (fp32 state when not whole)
  const unsigned char* cbase = ctx->c + shift;
  if (!range.whole) {
    p.nq = range.nq4;
    p.n_tiles = (range.nq4 + plan.cg - 1) / plan.cg * plan.rg;
    p.tail = range.tail4;
    p.q_offset = ctx->q_offset + (uint32_t)range.q0;
    p.c = reinterpret_cast<const float4*>(cbase);
  }
  const int round_grid = (int)std::min<int64_t>(plan.grid, p.n_tiles);
  uint64_t r = first;
  for (int64_t b = 0; b < n;) {
    const unsigned char* xin = ctx->x[cur] + shift;
    unsigned char* xout = ctx->x[cur ^ 1] + shift;
    if ((fused.ok || cluster.ok) && n - b >= 2) {  // the next rounds in one launch over resident tiles
      // launches of even length (20 rounds at 8 per launch: 7 + 7 + 6, not 8 + 8 + 4)
      const int64_t per_launch = fused.ok ? fused.max_rounds : cluster.max_rounds;
      const int64_t launches_left = (n - b + per_launch - 1) / per_launch;
      const int chunk = (int)((n - b + launches_left - 1) / launches_left);
      const int threads = fused.ok ? fused.threads : cluster.threads;
      FusedParams fp;
      fp.x_cur = reinterpret_cast<const float4*>(xin);
      fp.x_nxt = reinterpret_cast<float4*>(xout);
      fp.c = reinterpret_cast<const float4*>(cbase);
      fp.trace = ctx->trace;
      fp.wtab = ctx->wtab;
      fp.tel = tel;
      fp.partials = ctx->partials;
      fp.ticket = ctx->ticket;
      fp.slot0 = (int64_t)(r % (uint64_t)ctx->trace_rounds);
      fp.ring = ctx->trace_rounds;
      fp.first_round = r;
      fp.n_rounds = chunk;
      fp.slots = fused.ok ? fused.slots : kClusterMaxRounds;
      fp.nq = range.nq4;
      fp.n_tiles = (range.nq4 + threads - 1) / threads;
      fp.row_bytes = p.row_bytes;
      fp.M = p.M;
      fp.tail = range.tail4;
      fp.alpha = p.alpha;
      fp.sigma = p.sigma;
      fp.inv_M = p.inv_M;
      fp.q_offset = ctx->q_offset + (uint32_t)range.q0;
      fp.keys = p.keys;
      if (!fused.ok) {  // rows split over the CTAs of a cluster
        ClusterParams cpar;
        cpar.f = fp;
        cpar.rpc = cluster.rpc;
        ClusterKernel ck = pick_cluster_kernel(ctx->objective);
        NM_CUDA(ctx, cudaFuncSetAttribute(ck, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)cluster.smem));
        cudaLaunchConfig_t lc = {};
        lc.gridDim = dim3((unsigned)(std::min<int64_t>(cluster.grid / cluster.C, fp.n_tiles) * cluster.C));
        lc.blockDim = dim3((unsigned)cluster.threads);
        lc.dynamicSmemBytes = cluster.smem;
        lc.stream = stream;
        cudaLaunchAttribute attr;
        attr.id = cudaLaunchAttributeClusterDimension;
        attr.val.clusterDim.x = (unsigned)cluster.C;
        attr.val.clusterDim.y = 1;
        attr.val.clusterDim.z = 1;
        lc.attrs = &attr;
        lc.numAttrs = 1;
        NM_CUDA(ctx, cudaLaunchKernelEx(&lc, ck, cpar));
      } else {
        // (the attribute belongs to the kernel, not to this context: another context may have lowered it)
        // (one instance for all launches of the call: the larger one unless the whole call is four rounds or fewer)
        FusedKernel fk = pick_fused_kernel(ctx->objective, ctx->L.halves, (int)std::min<int64_t>(n, fused.max_rounds));
        NM_CUDA(ctx, cudaFuncSetAttribute(fk, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)fused.smem));
        fk<<<(unsigned)std::min<int64_t>(fused.grid, fp.n_tiles), fused.threads, fused.smem, stream>>>(fp);
      }
      ctx->launches += 1;
      cur ^= 1;
      r += (uint64_t)chunk;
      b += chunk;
      continue;
    }
    const int64_t slot = (int64_t)(r % (uint64_t)ctx->trace_rounds);
    p.x_cur = reinterpret_cast<const float4*>(xin);
    p.x_nxt = reinterpret_cast<float4*>(xout);
    p.peers = ctx->trace + slot * ctx->M;
    p.tel_out = tel + 2 * slot;
    p.round_lo = (uint32_t)r;
    p.ctr3 = philox_ctr3(kTagNoise, r);
    kernel<<<round_grid, kThreads, plan.smem, stream>>>(p);
    ctx->launches += 1;
    cur ^= 1;
    r += 1;
    b += 1;
  }
  NM_CUDA(ctx, cudaGetLastError());
  return NETMAX_OK;
}

}  // namespace

extern "C" {

int netmax_config_init(netmax_config* cfg) {
  if (!cfg) return fail(nullptr, NETMAX_INVALID_ARG, "cfg is NULL");
  std::memset(cfg, 0, sizeof *cfg);
  cfg->objective = 1;
  cfg->trace_rounds = 1024;
  cfg->policy_K = 20;
  cfg->policy_R = 20;
  return NETMAX_OK;
}

static int check_sizes(const netmax_config* cfg) {
  if (!cfg) return fail(nullptr, NETMAX_INVALID_ARG, "cfg is NULL");
  if (cfg->storage != NETMAX_STORAGE_F32 && cfg->storage != NETMAX_STORAGE_BF16)
    return fail(nullptr, NETMAX_INVALID_ARG, "storage = %d is neither NETMAX_STORAGE_F32 nor NETMAX_STORAGE_BF16", cfg->storage);
  if (cfg->storage == NETMAX_STORAGE_BF16 && cfg->element_offset % 8 != 0)
    return fail(nullptr, NETMAX_INVALID_ARG, "element_offset = %lld must be a multiple of 8 with bfloat16 storage", (long long)cfg->element_offset);
  if (cfg->M < 2 || cfg->M > kMaxM) return fail(nullptr, NETMAX_INVALID_ARG, "M = %d outside [2, %lld]", cfg->M, (long long)kMaxM);
  if (cfg->d < 1 || cfg->d >= kMaxD) return fail(nullptr, NETMAX_INVALID_ARG, "d = %lld outside [1, 2^30 - 32)", (long long)cfg->d);
  if (cfg->element_offset < 0 || cfg->element_offset % 4 != 0 || cfg->element_offset + cfg->d >= kMaxD)
    return fail(nullptr, NETMAX_INVALID_ARG, "element_offset = %lld must be a non-negative multiple of 4 with offset + d < 2^30 - 32", (long long)cfg->element_offset);
  if (cfg->trace_rounds < 1) return fail(nullptr, NETMAX_INVALID_ARG, "trace_rounds = %lld < 1", (long long)cfg->trace_rounds);
  if (cfg->fuse_rounds < 0 || cfg->fuse_rounds > kFusedMaxRounds)
    return fail(nullptr, NETMAX_INVALID_ARG, "fuse_rounds = %d outside [0, %d]", cfg->fuse_rounds, kFusedMaxRounds);
  if (cfg->first_round < 0 || cfg->first_round >= ((int64_t)1 << 56))
    return fail(nullptr, NETMAX_INVALID_ARG, "first_round = %lld outside [0, 2^56)", (long long)cfg->first_round);
  return NETMAX_OK;
}

int netmax_workspace_size(const netmax_config* cfg, size_t* bytes) {
  int rc = check_sizes(cfg);
  if (rc) return rc;
  if (!bytes) return fail(nullptr, NETMAX_INVALID_ARG, "bytes is NULL");
  *bytes = make_layout(cfg->M, cfg->d, cfg->trace_rounds, cfg->storage).total;
  return NETMAX_OK;
}

int netmax_create_ex(const netmax_config* cfg, netmax_ctx** out) {
  if (!out) return fail(nullptr, NETMAX_INVALID_ARG, "out is NULL");
  *out = nullptr;
  int rc = check_sizes(cfg);
  if (rc) return rc;
  if (!(cfg->lr > 0.0) || !std::isfinite(cfg->lr)) return fail(nullptr, NETMAX_INVALID_ARG, "lr = %g must be positive and finite", cfg->lr);
  if (!(cfg->sigma >= 0.0) || !std::isfinite(cfg->sigma)) return fail(nullptr, NETMAX_INVALID_ARG, "sigma = %g must be >= 0 and finite", cfg->sigma);
  if (!(cfg->x0_std >= 0.0) || !std::isfinite(cfg->x0_std) || !(cfg->c_std >= 0.0) || !std::isfinite(cfg->c_std))
    return fail(nullptr, NETMAX_INVALID_ARG, "x0_std and c_std must be >= 0 and finite");
  if (!std::isfinite(cfg->rho)) return fail(nullptr, NETMAX_INVALID_ARG, "rho is not finite");
  if (!(cfg->pull_weight >= 0.0 && cfg->pull_weight < 1.0))
    return fail(nullptr, NETMAX_INVALID_ARG, "pull_weight = %g outside [0, 1)", cfg->pull_weight);
  if (cfg->objective != 0 && cfg->objective != 1) return fail(nullptr, NETMAX_INVALID_ARG, "objective = %d is not 0 or 1", cfg->objective);
  if (cfg->device < 0) return fail(nullptr, NETMAX_INVALID_ARG, "device = %d", cfg->device);

  netmax_ctx* ctx = new (std::nothrow) netmax_ctx();
  if (!ctx) return fail(nullptr, NETMAX_OOM, "host allocation failed");
  auto bail = [&](int code) {
    g_error = ctx->error;
    netmax_destroy(ctx);
    return code;
  };
  ctx->M = cfg->M;
  ctx->d = cfg->d;
  ctx->q_offset = (uint32_t)(cfg->element_offset / 4);
  ctx->device = cfg->device;
  ctx->stream = (cudaStream_t)cfg->stream;
  ctx->trace_rounds = cfg->trace_rounds;
  ctx->alpha = cfg->lr;
  ctx->sigma = cfg->sigma;
  ctx->pull_weight = cfg->pull_weight;
  ctx->objective = cfg->objective;
  ctx->seed = cfg->seed;
  ctx->policy_K = cfg->policy_K > 0 ? cfg->policy_K : 20;
  ctx->policy_R = cfg->policy_R > 0 ? cfg->policy_R : 20;
  ctx->policy_rho_upper = cfg->policy_rho_upper > 0.0 ? cfg->policy_rho_upper : 0.0;
  ctx->keys = make_philox_keys(cfg->seed);
  ctx->storage = cfg->storage;
  ctx->fuse_rounds = cfg->fuse_rounds;
  ctx->round0 = ctx->rounds = cfg->first_round;
  ctx->L = make_layout(cfg->M, cfg->d, cfg->trace_rounds, cfg->storage);

  rc = build_adjacency(ctx, cfg->M, cfg->link_speed_gbps, ctx->adj);
  if (rc) return bail(rc);
  rc = resolve_policy(ctx, cfg->link_speed_gbps, cfg->prob, cfg->rho);
  if (rc) return bail(rc);

  int ndev = 0;
  if (cudaGetDeviceCount(&ndev) != cudaSuccess || ndev < 1) {
    cudaGetLastError();
    ctx->error = "no CUDA device is available";
    return bail(NETMAX_CUDA_ERROR);
  }
  if (cfg->device >= ndev) { ctx->error = "device ordinal out of range"; return bail(NETMAX_INVALID_ARG); }
  DeviceGuard guard(cfg->device);
  if (!guard.ok) { ctx->error = "cudaSetDevice failed"; return bail(NETMAX_CUDA_ERROR); }
  cudaDeviceProp prop;
  if (cudaGetDeviceProperties(&prop, cfg->device) == cudaSuccess) {
    ctx->sm_count = prop.multiProcessorCount;
    ctx->cooperative = prop.cooperativeLaunch != 0;
  }
  if (cfg->workspace) {
    if (((uintptr_t)cfg->workspace & 255) != 0) { ctx->error = "workspace is not 256-byte aligned"; return bail(NETMAX_INVALID_ARG); }
    if (cfg->workspace_bytes < ctx->L.total) {
      char buf[128];
      snprintf(buf, sizeof buf, "workspace holds %zu bytes, %zu needed", cfg->workspace_bytes, ctx->L.total);
      ctx->error = buf;
      return bail(NETMAX_OOM);
    }
    ctx->base = (unsigned char*)cfg->workspace;
  } else {
    void* ptr = nullptr;
    cudaError_t e = cudaMalloc(&ptr, ctx->L.total);
    if (e != cudaSuccess) {
      cudaGetLastError();
      char buf[160];
      snprintf(buf, sizeof buf, "cudaMalloc of %zu bytes failed: %s", ctx->L.total, cudaGetErrorString(e));
      ctx->error = buf;
      return bail(NETMAX_OOM);
    }
    ctx->base = (unsigned char*)ptr;
    ctx->own_memory = true;
  }
  const Layout& L = ctx->L;
  ctx->x[0] = ctx->base + L.off_x0;
  ctx->x[1] = ctx->base + L.off_x1;
  ctx->c = ctx->base + L.off_c;
  ctx->thr = (uint32_t*)(ctx->base + L.off_thr);
  ctx->last_nz = (int32_t*)(ctx->base + L.off_last);
  ctx->wtab = (float*)(ctx->base + L.off_w);
  ctx->trace = (int32_t*)(ctx->base + L.off_trace);
  ctx->wring = (float*)(ctx->base + L.off_wring);
  ctx->tel = (double*)(ctx->base + L.off_tel);
  ctx->partials = (double*)(ctx->base + L.off_partials);
  ctx->ticket = (unsigned int*)(ctx->base + L.off_ticket);
  ctx->colpart = (float4*)(ctx->base + L.off_colpart);
  ctx->grid_barrier = ctx->ticket + 16;
  ctx->dev_error = ctx->ticket + 32;
  ctx->measure_out = (double*)(ctx->ticket + 48);
  ctx->coltick = (unsigned int*)(ctx->base + L.off_coltick);
  ctx->pipe_tel = (double*)(ctx->base + L.off_pipe_tel);

  auto step = [&](cudaError_t e, const char* what) {
    if (e == cudaSuccess) return true;
    ctx->error = std::string(what) + ": " + cudaGetErrorString(e);
    return false;
  };
  if (!step(cudaMemsetAsync(ctx->ticket, 0, 256, ctx->stream), "cudaMemsetAsync(ticket)")) return bail(NETMAX_CUDA_ERROR);
  if (!step(cudaMemsetAsync(ctx->coltick, 0, (size_t)kMaxGrid * sizeof(unsigned int), ctx->stream), "cudaMemsetAsync(coltick)")) return bail(NETMAX_CUDA_ERROR);
  if (!step(cudaMemsetAsync(ctx->x[1], 0, L.plane, ctx->stream), "cudaMemsetAsync(x)")) return bail(NETMAX_CUDA_ERROR);
  if (!step(cudaMemsetAsync(ctx->tel, 0, (size_t)ctx->trace_rounds * 2 * sizeof(double), ctx->stream), "cudaMemsetAsync(tel)")) return bail(NETMAX_CUDA_ERROR);
  rc = upload_policy(ctx);
  if (rc) return bail(rc);
  rc = launch_init(ctx, ctx->x[0], cfg->x0_std, kTagX0);
  if (rc) return bail(rc);
  rc = launch_init(ctx, ctx->c, cfg->c_std, kTagC);
  if (rc) return bail(rc);
  if (!step(cudaStreamSynchronize(ctx->stream), "cudaStreamSynchronize")) return bail(NETMAX_CUDA_ERROR);
  *out = ctx;
  return NETMAX_OK;
}

int netmax_create(int32_t M, int64_t d, const double* link_speed_gbps, const double* prob, double lr, uint64_t seed,
                  netmax_ctx** out) {
  netmax_config cfg;
  netmax_config_init(&cfg);
  cfg.M = M;
  cfg.d = d;
  cfg.link_speed_gbps = link_speed_gbps;
  cfg.prob = prob;
  cfg.lr = lr;
  cfg.seed = seed;
  cfg.x0_std = 1.0;
  cfg.c_std = 1.0;
  int dev = 0;
  if (cudaGetDevice(&dev) == cudaSuccess) cfg.device = dev; else cudaGetLastError();
  return netmax_create_ex(&cfg, out);
}

void netmax_destroy(netmax_ctx* ctx) {
  if (!ctx) return;
  if (ctx->up_stream || ctx->down_stream) {
    DeviceGuard guard(ctx->device);
    if (ctx->up_stream) cudaStreamDestroy(ctx->up_stream);
    if (ctx->down_stream) cudaStreamDestroy(ctx->down_stream);
    cudaGetLastError();
  }
  if (ctx->own_memory && ctx->base) {
    DeviceGuard guard(ctx->device);
    cudaStreamSynchronize(ctx->stream);
    cudaFree(ctx->base);
    cudaGetLastError();
  }
  delete ctx;
}

int netmax_set_policy(netmax_ctx* ctx, const double* link_speed_gbps, const double* prob, double rho) {
  if (!ctx) return fail(nullptr, NETMAX_INVALID_ARG, "ctx is NULL");
  if (!std::isfinite(rho)) return fail(ctx, NETMAX_INVALID_ARG, "rho is not finite");
  DeviceGuard guard(ctx->device);
  std::vector<uint8_t> old_adj = ctx->adj;
  std::vector<double> old_P = ctx->P, old_t = ctx->t_iter;
  const double old_rho = ctx->rho;
  int rc = NETMAX_OK;
  if (link_speed_gbps) rc = build_adjacency(ctx, ctx->M, link_speed_gbps, ctx->adj);
  if (!rc) rc = resolve_policy(ctx, link_speed_gbps, prob, rho);
  if (rc) {  // leave the policy in force untouched
    ctx->adj.swap(old_adj);
    ctx->P.swap(old_P);
    ctx->t_iter.swap(old_t);
    ctx->rho = old_rho;
    return rc;
  }
  // rounds already enqueued still read the old tables: wait for them before overwriting
  NM_CUDA(ctx, cudaStreamSynchronize(ctx->stream));
  return upload_policy(ctx);
}

int netmax_get_policy(netmax_ctx* ctx, double* prob_out, double* rho_out) {
  if (!ctx) return fail(nullptr, NETMAX_INVALID_ARG, "ctx is NULL");
  if (prob_out) std::memcpy(prob_out, ctx->P.data(), ctx->P.size() * sizeof(double));
  if (rho_out) *rho_out = ctx->rho;
  return NETMAX_OK;
}

// After a synchronisation: has a kernel's bounded wait given up since the last check?
static int check_device_error(netmax_ctx* ctx) {
  unsigned int flag = 0;
  NM_CUDA(ctx, cudaMemcpy(&flag, ctx->dev_error, sizeof flag, cudaMemcpyDeviceToHost));
  if (flag == 0) return NETMAX_OK;
  cudaMemset(ctx->dev_error, 0, sizeof flag);
  return fail(ctx, NETMAX_CUDA_ERROR, "a multi-round launch gave up waiting at its grid barrier; replicas are not valid");
}

// Host transfers of a bfloat16 context go through fp32 on the device: the buffer of the double
// buffer that holds no replicas at the moment serves as the staging area, a chunk of rows at a
// time, and is cleared again afterwards.  Nothing is allocated.
static int64_t staging_rows(const netmax_ctx* ctx) {
  return std::max<int64_t>(1, (int64_t)(ctx->L.plane / ((size_t)ctx->d * sizeof(float))));
}

static int convert_grid(const netmax_ctx* ctx, int64_t total) {
  return (int)std::min<int64_t>((total + kThreads - 1) / kThreads, (int64_t)ctx->sm_count * 16);
}

static int copy_in(netmax_ctx* ctx, unsigned char* dst, const float* host) {
  if (!ctx) return fail(nullptr, NETMAX_INVALID_ARG, "ctx is NULL");
  if (!host) return fail(ctx, NETMAX_INVALID_ARG, "host pointer is NULL");
  DeviceGuard guard(ctx->device);
  if (ctx->storage == NETMAX_STORAGE_BF16) {
    float* stage = reinterpret_cast<float*>(ctx->x[ctx->cur ^ 1]);
    const int64_t chunk = staging_rows(ctx);
    for (int64_t r0 = 0; r0 < ctx->M; r0 += chunk) {
      const int64_t rows = std::min<int64_t>(chunk, ctx->M - r0);
      NM_CUDA(ctx, cudaMemcpyAsync(stage, host + (size_t)r0 * ctx->d, (size_t)rows * ctx->d * sizeof(float), cudaMemcpyHostToDevice, ctx->stream));
      narrow_rows_kernel<<<convert_grid(ctx, rows * ctx->d), kThreads, 0, ctx->stream>>>(
          stage, reinterpret_cast<unsigned short*>(dst) + (size_t)r0 * ctx->L.ld, rows, ctx->d, ctx->L.ld);
      ctx->launches += 1;
      NM_CUDA(ctx, cudaGetLastError());
    }
    NM_CUDA(ctx, cudaMemsetAsync(stage, 0, ctx->L.plane, ctx->stream));
    return NETMAX_OK;
  }
  NM_CUDA(ctx, cudaMemcpy2DAsync(dst, (size_t)ctx->L.ld * sizeof(float), host, (size_t)ctx->d * sizeof(float),
                                 (size_t)ctx->d * sizeof(float), (size_t)ctx->M, cudaMemcpyHostToDevice, ctx->stream));
  return NETMAX_OK;
}

static int copy_out(netmax_ctx* ctx, const unsigned char* src, float* host) {
  if (!ctx) return fail(nullptr, NETMAX_INVALID_ARG, "ctx is NULL");
  if (!host) return fail(ctx, NETMAX_INVALID_ARG, "host pointer is NULL");
  DeviceGuard guard(ctx->device);
  if (ctx->storage == NETMAX_STORAGE_BF16) {
    float* stage = reinterpret_cast<float*>(ctx->x[ctx->cur ^ 1]);
    const int64_t chunk = staging_rows(ctx);
    for (int64_t r0 = 0; r0 < ctx->M; r0 += chunk) {
      const int64_t rows = std::min<int64_t>(chunk, ctx->M - r0);
      widen_rows_kernel<<<convert_grid(ctx, rows * ctx->d), kThreads, 0, ctx->stream>>>(
          reinterpret_cast<const unsigned short*>(src) + (size_t)r0 * ctx->L.ld, stage, rows, ctx->d, ctx->L.ld);
      ctx->launches += 1;
      NM_CUDA(ctx, cudaGetLastError());
      NM_CUDA(ctx, cudaMemcpyAsync(host + (size_t)r0 * ctx->d, stage, (size_t)rows * ctx->d * sizeof(float), cudaMemcpyDeviceToHost, ctx->stream));
    }
    NM_CUDA(ctx, cudaMemsetAsync(stage, 0, ctx->L.plane, ctx->stream));
    NM_CUDA(ctx, cudaStreamSynchronize(ctx->stream));
    return check_device_error(ctx);
  }
  NM_CUDA(ctx, cudaMemcpy2DAsync(host, (size_t)ctx->d * sizeof(float), src, (size_t)ctx->L.ld * sizeof(float),
                                 (size_t)ctx->d * sizeof(float), (size_t)ctx->M, cudaMemcpyDeviceToHost, ctx->stream));
  NM_CUDA(ctx, cudaStreamSynchronize(ctx->stream));
  return check_device_error(ctx);
}

int netmax_set_replicas(netmax_ctx* ctx, const float* host_x) { return copy_in(ctx, ctx ? ctx->x[ctx->cur] : nullptr, host_x); }
int netmax_set_centres(netmax_ctx* ctx, const float* host_c) { return copy_in(ctx, ctx ? ctx->c : nullptr, host_c); }
int netmax_read_replicas(netmax_ctx* ctx, float* host_out) { return copy_out(ctx, ctx ? ctx->x[ctx->cur] : nullptr, host_out); }
int netmax_read_centres(netmax_ctx* ctx, float* host_out) { return copy_out(ctx, ctx ? ctx->c : nullptr, host_out); }

int netmax_round(netmax_ctx* ctx, int64_t n_rounds) {
  if (!ctx) return fail(nullptr, NETMAX_INVALID_ARG, "ctx is NULL");
  if (n_rounds < 0) return fail(ctx, NETMAX_INVALID_ARG, "n_rounds = %lld < 0", (long long)n_rounds);
  if (ctx->async_on) return fail(ctx, NETMAX_INVALID_ARG, "the context runs the asynchronous timeline; use netmax_async_steps");
  if (n_rounds == 0) return NETMAX_OK;
  if ((uint64_t)(ctx->rounds + n_rounds) >= ((uint64_t)1 << 56)) return fail(ctx, NETMAX_INVALID_ARG, "round counter would exceed 2^56");
  DeviceGuard guard(ctx->device);
  RoundPlan plan;
  int rc = plan_round(ctx, plan, ctx->objective);
  if (rc) return rc;
  FusedPlan fused;
  rc = plan_fused(ctx, plan, fused);
  if (rc) return rc;
  ResidentPlan resident;
  rc = plan_resident(ctx, plan, resident);
  if (rc) return rc;
  if (ctx->fuse_rounds == 1) resident.ok = false;  // one launch per round was asked for
  ClusterPlan cluster;
  rc = plan_cluster(ctx, plan, fused, cluster);
  if (rc) return rc;

  RoundParams p = make_round_params(ctx, plan);

  int64_t done = 0;
  while (done < n_rounds) {
    // peers of a batch of rounds in one launch (counter-based draws do not depend on x),
    // at most one lap of the ring at a time
    const int64_t batch = std::min<int64_t>(n_rounds - done, ctx->trace_rounds);
    rc = launch_sampler(ctx, (uint64_t)ctx->rounds, batch, ctx->trace, ctx->wring, ctx->rounds % ctx->trace_rounds,
                        ctx->trace_rounds);
    if (rc) return rc;
    if (resident.ok && batch >= resident.min_rounds) {
      // short vectors: every round of the batch on shared-memory-resident columns
      ResidentKernel rk = pick_resident_kernel(ctx->objective, ctx->L.halves);
      int64_t b = 0;
      while (b < batch) {
        const int64_t chunk = std::min<int64_t>(batch - b, resident.max_rounds);
        ResidentParams rp;
        rp.x_cur = reinterpret_cast<const char*>(ctx->x[ctx->cur]);
        rp.x_nxt = reinterpret_cast<char*>(ctx->x[ctx->cur ^ 1]);
        rp.c = reinterpret_cast<const char*>(ctx->c);
        rp.trace = ctx->trace;
        rp.wring = ctx->wring;
        rp.partials = reinterpret_cast<double*>(ctx->colpart);
        rp.slot0 = ctx->rounds % ctx->trace_rounds;
        rp.ring = ctx->trace_rounds;
        rp.first_round = (uint64_t)ctx->rounds;
        rp.n_rounds = (int32_t)chunk;
        rp.nq = (ctx->d + 3) / 4;
        rp.n_tiles = resident.n_tiles;
        rp.row_bytes = p.row_bytes;
        rp.M = p.M;
        rp.tail = (int32_t)(ctx->d % 4);
        rp.G = resident.G;
        rp.log2G = resident.log2G;
        rp.draw_chunk = resident.draw_chunk;
        rp.alpha = p.alpha;
        rp.sigma = p.sigma;
        rp.inv_M = p.inv_M;
        rp.q_offset = p.q_offset;
        rp.keys = p.keys;
        NM_CUDA(ctx, cudaFuncSetAttribute(rk, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)resident.smem));
        rk<<<resident.grid, resident.threads, resident.smem, ctx->stream>>>(rp);
        const int warps_per_block = kThreads / 32;
        sum_tile_partials_kernel<<<(unsigned)((chunk + warps_per_block - 1) / warps_per_block), kThreads, 0, ctx->stream>>>(
            rp.partials, rp.n_tiles, rp.n_rounds, (double)p.inv_M, ctx->tel, rp.slot0, rp.ring);
        ctx->launches += 2;
        NM_CUDA(ctx, cudaGetLastError());
        ctx->cur ^= 1;
        ctx->rounds += chunk;
        b += chunk;
      }
      done += batch;
      continue;
    }
    if (plan.short_vectors && ctx->cooperative && batch >= 2) {
      // short, L2-resident problem: all rounds of the batch in cooperative launches
      int64_t b = 0;
      while (b < batch) {
        const int64_t chunk = std::min<int64_t>(batch - b, kMaxRoundsPerLaunch);
        MultiRoundParams mp;
        mp.r = p;
        mp.r.x_cur = reinterpret_cast<const float4*>(ctx->x[ctx->cur]);
        mp.r.x_nxt = reinterpret_cast<float4*>(ctx->x[ctx->cur ^ 1]);
        mp.r.peers = nullptr;
        mp.r.tel_out = nullptr;
        mp.trace = ctx->trace;
        mp.tel = ctx->tel;
        mp.partials2 = ctx->partials;
        mp.barrier = ctx->grid_barrier;
        mp.error = ctx->dev_error;
        mp.slot0 = ctx->rounds % ctx->trace_rounds;
        mp.ring = ctx->trace_rounds;
        mp.first_round = (uint64_t)ctx->rounds;
        mp.n_rounds = (int32_t)chunk;
        mp.absent_ctas = ctx->inject_absent_ctas;
        ctx->inject_absent_ctas = 0;
        NM_CUDA(ctx, cudaMemsetAsync(ctx->grid_barrier, 0, sizeof(unsigned int), ctx->stream));
        void* args[] = {&mp};
        NM_CUDA(ctx, cudaLaunchCooperativeKernel((const void*)pick_multi_kernel(ctx->objective, ctx->L.halves), dim3(plan.grid), dim3(kThreads),
                                                 args, plan.smem, ctx->stream));
        ctx->launches += 1;
        ctx->cur ^= (int)(chunk & 1);
        ctx->rounds += chunk;
        b += chunk;
      }
      done += batch;
      continue;
    }
    {  // long vectors: fused, cluster-resident or one launch per round, over all columns
      ColumnRange all;
      all.q0 = 0;
      all.nq4 = (ctx->d + 3) / 4;
      all.tail4 = (int32_t)(ctx->d % 4);
      all.whole = true;
      int cur = ctx->cur;
      rc = launch_long_rounds(ctx, ctx->stream, plan, fused, cluster, p, all, ctx->tel, (uint64_t)ctx->rounds, batch, cur);
      if (rc) return rc;
      ctx->cur = cur;
      ctx->rounds += batch;
    }
    NM_CUDA(ctx, cudaGetLastError());
    done += batch;
  }
  return NETMAX_OK;
}

int64_t netmax_rounds_done(const netmax_ctx* ctx) { return ctx ? ctx->rounds : -1; }

// ---- host round trip, pipelined over column chunks ----------------------------------------------
int netmax_round_from_host(netmax_ctx* ctx, const float* host_x, const float* host_c, int64_t n_rounds, float* host_out,
                           int32_t n_chunks) {
  if (!ctx) return fail(nullptr, NETMAX_INVALID_ARG, "ctx is NULL");
  if (n_rounds < 0) return fail(ctx, NETMAX_INVALID_ARG, "n_rounds = %lld < 0", (long long)n_rounds);
  if (!host_out) return fail(ctx, NETMAX_INVALID_ARG, "host_out is NULL");
  if (n_chunks < 0 || n_chunks > kMaxChunks) return fail(ctx, NETMAX_INVALID_ARG, "n_chunks = %d outside [0, %d]", n_chunks, kMaxChunks);
  if (ctx->async_on) return fail(ctx, NETMAX_INVALID_ARG, "the context runs the asynchronous timeline; use netmax_async_steps");
  DeviceGuard guard(ctx->device);
  RoundPlan plan;
  int rc = plan_round(ctx, plan, ctx->objective);
  if (rc) return rc;
  const int64_t nq4 = (ctx->d + 3) / 4;
  const int64_t unit = 256;  // chunk boundaries on 4 KB of every row
  int chunks = n_chunks > 0 ? n_chunks : 8;
  chunks = (int)std::min<int64_t>(chunks, (nq4 + unit - 1) / unit);
  const bool pipelined = ctx->storage == NETMAX_STORAGE_F32 && !plan.short_vectors && n_rounds >= 1 &&
                         n_rounds <= ctx->trace_rounds && chunks >= 2 &&
                         (uint64_t)(ctx->rounds + n_rounds) < ((uint64_t)1 << 56);
  if (!pipelined) {  // the same three steps one after the other
    if (host_x) { rc = netmax_set_replicas(ctx, host_x); if (rc) return rc; }
    if (host_c) { rc = netmax_set_centres(ctx, host_c); if (rc) return rc; }
    rc = netmax_round(ctx, n_rounds);
    if (rc) return rc;
    return netmax_read_replicas(ctx, host_out);
  }
  FusedPlan fused;
  rc = plan_fused(ctx, plan, fused);
  if (rc) return rc;
  ClusterPlan cluster;
  rc = plan_cluster(ctx, plan, fused, cluster);
  if (rc) return rc;
  if (!ctx->up_stream) NM_CUDA(ctx, cudaStreamCreateWithFlags(&ctx->up_stream, cudaStreamNonBlocking));
  if (!ctx->down_stream) NM_CUDA(ctx, cudaStreamCreateWithFlags(&ctx->down_stream, cudaStreamNonBlocking));

  const int64_t per_chunk = ((nq4 + chunks - 1) / chunks + unit - 1) / unit * unit;
  chunks = (int)((nq4 + per_chunk - 1) / per_chunk);
  std::vector<cudaEvent_t> events(2 * chunks + 1, nullptr);
  auto cleanup = [&]() {
    for (cudaEvent_t e : events)
      if (e) cudaEventDestroy(e);
  };
  for (auto& e : events) {
    cudaError_t ce = cudaEventCreateWithFlags(&e, cudaEventDisableTiming);
    if (ce != cudaSuccess) { cleanup(); return fail(ctx, NETMAX_CUDA_ERROR, "cudaEventCreate: %s", cudaGetErrorString(ce)); }
  }
  // from here on a failure still has to wait for what is in flight before the events go away
  auto bail = [&](int code) {
    cudaStreamSynchronize(ctx->up_stream);
    cudaStreamSynchronize(ctx->stream);
    cudaStreamSynchronize(ctx->down_stream);
    cleanup();
    return code;
  };
#define NM_PIPE(call)                                                                                   \
  do {                                                                                                  \
    cudaError_t e_ = (call);                                                                            \
    if (e_ != cudaSuccess) return bail(fail(ctx, NETMAX_CUDA_ERROR, "%s: %s", #call, cudaGetErrorString(e_))); \
  } while (0)

  const uint64_t first = (uint64_t)ctx->rounds;
  rc = launch_sampler(ctx, first, n_rounds, ctx->trace, ctx->wring, ctx->rounds % ctx->trace_rounds, ctx->trace_rounds);
  if (rc) return bail(rc);
  // uploads must not overtake earlier work of the context that still reads the buffers
  NM_PIPE(cudaEventRecord(events[2 * chunks], ctx->stream));
  NM_PIPE(cudaStreamWaitEvent(ctx->up_stream, events[2 * chunks], 0));
  const RoundParams p = make_round_params(ctx, plan);
  const size_t dev_pitch = (size_t)ctx->L.ld * sizeof(float), host_pitch = (size_t)ctx->d * sizeof(float);
  int cur_end = ctx->cur;
  for (int k = 0; k < chunks; ++k) {
    ColumnRange range;
    range.q0 = (int64_t)k * per_chunk;
    range.nq4 = std::min<int64_t>(per_chunk, nq4 - range.q0);
    range.tail4 = (k == chunks - 1) ? (int32_t)(ctx->d % 4) : 0;
    range.whole = false;
    const int64_t e0 = range.q0 * 4, cols = std::min<int64_t>(range.nq4 * 4, ctx->d - e0);
    const size_t width = (size_t)cols * sizeof(float), at = (size_t)e0 * sizeof(float);
    if (host_x)
      NM_PIPE(cudaMemcpy2DAsync(ctx->x[ctx->cur] + at, dev_pitch, host_x + e0, host_pitch, width, (size_t)ctx->M,
                                cudaMemcpyHostToDevice, ctx->up_stream));
    if (host_c)
      NM_PIPE(cudaMemcpy2DAsync(ctx->c + at, dev_pitch, host_c + e0, host_pitch, width, (size_t)ctx->M, cudaMemcpyHostToDevice,
                                ctx->up_stream));
    NM_PIPE(cudaEventRecord(events[2 * k], ctx->up_stream));
    NM_PIPE(cudaStreamWaitEvent(ctx->stream, events[2 * k], 0));
    int cur = ctx->cur;
    rc = launch_long_rounds(ctx, ctx->stream, plan, fused, cluster, p, range, ctx->pipe_tel + (size_t)k * ctx->trace_rounds * 2,
                            first, n_rounds, cur);
    if (rc) return bail(rc);
    cur_end = cur;
    NM_PIPE(cudaEventRecord(events[2 * k + 1], ctx->stream));
    NM_PIPE(cudaStreamWaitEvent(ctx->down_stream, events[2 * k + 1], 0));
    NM_PIPE(cudaMemcpy2DAsync(host_out + e0, host_pitch, ctx->x[cur_end] + at, dev_pitch, width, (size_t)ctx->M,
                              cudaMemcpyDeviceToHost, ctx->down_stream));
  }
  // the rounds' telemetry: the chunks' shares added in chunk order
  sum_chunk_telemetry_kernel<<<(unsigned)((n_rounds + kThreads - 1) / kThreads), kThreads, 0, ctx->stream>>>(
      ctx->pipe_tel, chunks, ctx->trace_rounds, (int64_t)(first % (uint64_t)ctx->trace_rounds), n_rounds, ctx->tel);
  ctx->launches += 1;
  NM_PIPE(cudaGetLastError());
  ctx->cur = cur_end;
  ctx->rounds += n_rounds;
  NM_PIPE(cudaStreamSynchronize(ctx->down_stream));
  NM_PIPE(cudaStreamSynchronize(ctx->stream));
#undef NM_PIPE
  cleanup();
  return check_device_error(ctx);
}

int netmax_set_fuse_rounds(netmax_ctx* ctx, int32_t fuse_rounds) {
  if (!ctx) return fail(nullptr, NETMAX_INVALID_ARG, "ctx is NULL");
  if (fuse_rounds < 0 || fuse_rounds > kFusedMaxRounds)
    return fail(ctx, NETMAX_INVALID_ARG, "fuse_rounds = %d outside [0, %d]", fuse_rounds, kFusedMaxRounds);
  ctx->fuse_rounds = fuse_rounds;
  ctx->fused_planned = false;
  ctx->cluster_planned = false;
  return NETMAX_OK;
}

int netmax_read_columns(netmax_ctx* ctx, const int64_t* host_cols, int64_t n_cols, float* host_out) {
  if (!ctx) return fail(nullptr, NETMAX_INVALID_ARG, "ctx is NULL");
  if (n_cols < 0 || (n_cols > 0 && (!host_cols || !host_out))) return fail(ctx, NETMAX_INVALID_ARG, "bad column list");
  if (n_cols == 0) return NETMAX_OK;
  for (int64_t k = 0; k < n_cols; ++k)
    if (host_cols[k] < 0 || host_cols[k] >= ctx->d) return fail(ctx, NETMAX_INVALID_ARG, "cols[%lld] = %lld outside [0, d)", (long long)k, (long long)host_cols[k]);
  DeviceGuard guard(ctx->device);
  int64_t* d_cols = nullptr;
  float* d_out = nullptr;
  NM_CUDA(ctx, cudaMalloc(&d_cols, (size_t)n_cols * sizeof(int64_t)));
  cudaError_t e = cudaMalloc(&d_out, (size_t)n_cols * ctx->M * sizeof(float));
  if (e != cudaSuccess) { cudaFree(d_cols); cudaGetLastError(); return fail(ctx, NETMAX_OOM, "cudaMalloc failed: %s", cudaGetErrorString(e)); }
  int rc = NETMAX_OK;
  const int64_t total = n_cols * ctx->M;
  const int grid = (int)std::min<int64_t>((total + kThreads - 1) / kThreads, 4096);
  e = cudaMemcpyAsync(d_cols, host_cols, (size_t)n_cols * sizeof(int64_t), cudaMemcpyHostToDevice, ctx->stream);
  if (e == cudaSuccess) {
    gather_columns_kernel<<<grid, kThreads, 0, ctx->stream>>>(ctx->x[ctx->cur], ctx->storage == NETMAX_STORAGE_BF16, ctx->L.ld, ctx->M, d_cols, n_cols, d_out);
    ctx->launches += 1;
    e = cudaGetLastError();
  }
  if (e == cudaSuccess) e = cudaMemcpyAsync(host_out, d_out, (size_t)total * sizeof(float), cudaMemcpyDeviceToHost, ctx->stream);
  if (e == cudaSuccess) e = cudaStreamSynchronize(ctx->stream);
  if (e != cudaSuccess) rc = fail(ctx, NETMAX_CUDA_ERROR, "read_columns: %s", cudaGetErrorString(e));
  cudaFree(d_cols);
  cudaFree(d_out);
  return rc ? rc : check_device_error(ctx);
}

// ---- sampled read-back that allocates nothing -------------------------------------------
// Staging area of netmax_read_columns_static: the column list, then the gathered values.
// It is part of the library image, so every device that loads the library holds it.
struct StaticGatherScratch {
  int64_t cols[NETMAX_STATIC_MAX_COLS];
  float values[NETMAX_STATIC_MAX_VALUES];
};
static __device__ __align__(256) unsigned char g_gather_scratch[sizeof(StaticGatherScratch)];

// In host code g_gather_scratch is only a stand-in for the symbol; the address a kernel or a
// copy can use comes from cudaGetSymbolAddress, looked up once per device (that device
// current) and cached here.
static std::mutex g_gather_mu;
static StaticGatherScratch* g_gather_ptr[64] = {};

static int gather_scratch_address(netmax_ctx* ctx, StaticGatherScratch** out) {
  std::lock_guard<std::mutex> lock(g_gather_mu);
  const bool cached = ctx->device >= 0 && ctx->device < 64;
  if (cached && g_gather_ptr[ctx->device]) {
    *out = g_gather_ptr[ctx->device];
    return NETMAX_OK;
  }
  void* ptr = nullptr;
  NM_CUDA(ctx, cudaGetSymbolAddress(&ptr, g_gather_scratch));
  if (!ptr) return fail(ctx, NETMAX_CUDA_ERROR, "cudaGetSymbolAddress returned a null address");
  if (cached) g_gather_ptr[ctx->device] = (StaticGatherScratch*)ptr;
  *out = (StaticGatherScratch*)ptr;
  return NETMAX_OK;
}

int netmax_read_columns_static(netmax_ctx* ctx, const int64_t* host_cols, int64_t n_cols, float* host_out) {
  if (!ctx) return fail(nullptr, NETMAX_INVALID_ARG, "ctx is NULL");
  if (n_cols < 0 || (n_cols > 0 && (!host_cols || !host_out))) return fail(ctx, NETMAX_INVALID_ARG, "bad column list");
  if (n_cols > NETMAX_STATIC_MAX_COLS)
    return fail(ctx, NETMAX_INVALID_ARG, "read_columns_static: n_cols = %lld exceeds the fixed staging area (%d columns); split the list",
                (long long)n_cols, NETMAX_STATIC_MAX_COLS);
  if (n_cols * (int64_t)ctx->M > NETMAX_STATIC_MAX_VALUES)
    return fail(ctx, NETMAX_INVALID_ARG, "read_columns_static: M * n_cols = %lld exceeds the fixed staging area (%d values); split the list",
                (long long)(n_cols * (int64_t)ctx->M), NETMAX_STATIC_MAX_VALUES);
  if (n_cols == 0) return NETMAX_OK;
  for (int64_t k = 0; k < n_cols; ++k)
    if (host_cols[k] < 0 || host_cols[k] >= ctx->d) return fail(ctx, NETMAX_INVALID_ARG, "cols[%lld] = %lld outside [0, d)", (long long)k, (long long)host_cols[k]);
  DeviceGuard guard(ctx->device);
  StaticGatherScratch* scratch = nullptr;
  int rc = gather_scratch_address(ctx, &scratch);
  if (rc) return rc;
  const int64_t total = n_cols * ctx->M;
  const int grid = (int)std::min<int64_t>((total + kThreads - 1) / kThreads, 4096);
  NM_CUDA(ctx, cudaMemcpyAsync(scratch->cols, host_cols, (size_t)n_cols * sizeof(int64_t), cudaMemcpyHostToDevice, ctx->stream));
  gather_columns_kernel<<<grid, kThreads, 0, ctx->stream>>>(ctx->x[ctx->cur], ctx->storage == NETMAX_STORAGE_BF16, ctx->L.ld, ctx->M, scratch->cols, n_cols, scratch->values);
  ctx->launches += 1;
  cudaError_t e = cudaGetLastError();
  if (e == cudaSuccess) e = cudaMemcpyAsync(host_out, scratch->values, (size_t)total * sizeof(float), cudaMemcpyDeviceToHost, ctx->stream);
  // whatever happened, leave the shared array idle: the next call, perhaps on another stream, reuses it
  const cudaError_t es = cudaStreamSynchronize(ctx->stream);
  if (e == cudaSuccess) e = es;
  if (e != cudaSuccess) return fail(ctx, NETMAX_CUDA_ERROR, "read_columns_static: %s", cudaGetErrorString(e));
  return check_device_error(ctx);
}

static int ring_range(netmax_ctx* ctx, int64_t first, int64_t n) {
  if (first < ctx->round0 || n < 0 || first + n > ctx->rounds || first < ctx->rounds - ctx->trace_rounds)
    return fail(ctx, NETMAX_TRACE_RANGE, "rounds [%lld, %lld) are not in the ring (rounds done %lld, capacity %lld)",
                (long long)first, (long long)(first + n), (long long)ctx->rounds, (long long)ctx->trace_rounds);
  return NETMAX_OK;
}

int netmax_peer_trace(netmax_ctx* ctx, int64_t first_round, int64_t n, int32_t* host_out) {
  if (!ctx) return fail(nullptr, NETMAX_INVALID_ARG, "ctx is NULL");
  int rc = ring_range(ctx, first_round, n);
  if (rc) return rc;
  if (n == 0) return NETMAX_OK;
  if (!host_out) return fail(ctx, NETMAX_INVALID_ARG, "host_out is NULL");
  DeviceGuard guard(ctx->device);
  NM_CUDA(ctx, cudaStreamSynchronize(ctx->stream));
  rc = check_device_error(ctx);
  if (rc) return rc;
  const size_t row = (size_t)ctx->M * sizeof(int32_t);
  int64_t r = first_round;
  while (r < first_round + n) {  // at most two contiguous pieces of the ring
    const int64_t slot = r % ctx->trace_rounds;
    const int64_t piece = std::min<int64_t>(first_round + n - r, ctx->trace_rounds - slot);
    NM_CUDA(ctx, cudaMemcpy(host_out + (size_t)(r - first_round) * ctx->M, ctx->trace + (size_t)slot * ctx->M, piece * row, cudaMemcpyDeviceToHost));
    r += piece;
  }
  return NETMAX_OK;
}

int netmax_telemetry(netmax_ctx* ctx, int64_t first_round, int64_t n, double* host_consensus, double* host_loss) {
  if (!ctx) return fail(nullptr, NETMAX_INVALID_ARG, "ctx is NULL");
  int rc = ring_range(ctx, first_round, n);
  if (rc) return rc;
  if (n == 0) return NETMAX_OK;
  DeviceGuard guard(ctx->device);
  NM_CUDA(ctx, cudaStreamSynchronize(ctx->stream));
  rc = check_device_error(ctx);
  if (rc) return rc;
  std::vector<double> ring((size_t)ctx->trace_rounds * 2);
  NM_CUDA(ctx, cudaMemcpy(ring.data(), ctx->tel, ring.size() * sizeof(double), cudaMemcpyDeviceToHost));
  for (int64_t k = 0; k < n; ++k) {
    const int64_t slot = (first_round + k) % ctx->trace_rounds;
    if (host_consensus) host_consensus[k] = ring[2 * slot];
    if (host_loss) host_loss[k] = ring[2 * slot + 1];
  }
  return NETMAX_OK;
}

int netmax_replicas_device(netmax_ctx* ctx, const float** x, int64_t* ld) {
  if (!ctx) return fail(nullptr, NETMAX_INVALID_ARG, "ctx is NULL");
  if (!x || !ld) return fail(ctx, NETMAX_INVALID_ARG, "output pointer is NULL");
  *x = reinterpret_cast<const float*>(ctx->x[ctx->cur]);
  *ld = ctx->L.ld;
  return NETMAX_OK;
}

int netmax_sample_peers(netmax_ctx* ctx, int64_t first_round, int64_t n_rounds, int32_t* device_out) {
  if (!ctx) return fail(nullptr, NETMAX_INVALID_ARG, "ctx is NULL");
  if (first_round < 0 || n_rounds < 0 || (n_rounds > 0 && !device_out)) return fail(ctx, NETMAX_INVALID_ARG, "bad range or NULL output");
  DeviceGuard guard(ctx->device);
  return launch_sampler(ctx, (uint64_t)first_round, n_rounds, device_out, nullptr, 0, INT64_MAX);
}

// ---- telemetry on demand --------------------------------------------------------------------
int netmax_measure(netmax_ctx* ctx, double* consensus, double* loss) {
  if (!ctx) return fail(nullptr, NETMAX_INVALID_ARG, "ctx is NULL");
  DeviceGuard guard(ctx->device);
  RoundPlan plan;
  int rc = plan_round(ctx, plan, 2);  // 2: the measuring instantiation of the round kernel
  if (rc) return rc;
  RoundKernel kernel = pick_kernel(2, plan.short_vectors, ctx->L.halves);
  RoundParams p;
  std::memset(&p, 0, sizeof p);
  p.x_cur = reinterpret_cast<const float4*>(ctx->x[ctx->cur]);
  p.x_nxt = nullptr;
  p.c = reinterpret_cast<const float4*>(ctx->c);
  p.peers = nullptr;
  p.wtab = ctx->wtab;
  p.partials = ctx->partials;
  p.ticket = ctx->ticket;
  p.tel_out = ctx->measure_out;
  p.ldq = ctx->L.ldq;
  p.row_bytes = (uint32_t)(ctx->L.ld * ctx->L.elem);
  p.nq = ctx->L.nq;
  p.n_tiles = plan.n_tiles;
  p.M = ctx->M;
  p.tail = (int32_t)(ctx->d % (4 * ctx->L.halves));
  p.cg = plan.cg;
  p.rl = plan.rl;
  p.rg = plan.rg;
  p.rows_per_group = plan.rows_per_group;
  p.colpart = ctx->colpart;
  p.coltick = ctx->coltick;
  p.inv_M = 1.0f / (float)ctx->M;
  p.keys = ctx->keys;
  kernel<<<plan.grid, kThreads, plan.smem, ctx->stream>>>(p);
  ctx->launches += 1;
  NM_CUDA(ctx, cudaGetLastError());
  double out[2] = {0.0, 0.0};
  NM_CUDA(ctx, cudaMemcpyAsync(out, ctx->measure_out, sizeof out, cudaMemcpyDeviceToHost, ctx->stream));
  NM_CUDA(ctx, cudaStreamSynchronize(ctx->stream));
  if (consensus) *consensus = out[0];
  if (loss) *loss = out[1];
  return check_device_error(ctx);
}

// ---- asynchronous timeline --------------------------------------------------------------------
// First word of the Philox block of the peer stream at counter (0, worker, iteration): the host
// twin of the device sampler (same published algorithm, 32x32->64 products and xors).
static uint32_t host_peer_word(const PhiloxKeys& keys, uint32_t worker, uint64_t iter) {
  uint32_t c0 = 0, c1 = worker, c2 = (uint32_t)iter, c3 = philox_ctr3(kTagPeer, iter);
  for (int r = 0; r < 10; ++r) {
    const uint64_t p0 = (uint64_t)kPhiloxMul0 * c0, p1 = (uint64_t)kPhiloxMul1 * c2;
    const uint32_t n0 = (uint32_t)(p1 >> 32) ^ c1 ^ keys.k0[r];
    const uint32_t n2 = (uint32_t)(p0 >> 32) ^ c3 ^ keys.k1[r];
    c0 = n0;
    c1 = (uint32_t)p1;
    c2 = n2;
    c3 = (uint32_t)p0;
  }
  return c0;
}

// Draws the peer of worker i's next local iteration (Algorithm 2) and sets when it will finish.
// The policy is read at the top of an iteration and the moving average records the time the
// iteration took, so the pull weight and the duration are latched here: a policy or time
// matrix that arrives while the iteration is in flight does not touch them.
static void async_start_iteration(netmax_ctx* ctx, int i, double start) {
  const int32_t M = ctx->M;
  const uint32_t u = host_peer_word(ctx->keys, (uint32_t)i, (uint64_t)ctx->local_n[i]);
  const uint32_t* row = ctx->h_thr.data() + (size_t)i * M;
  const int32_t count = (int32_t)(std::upper_bound(row, row + M, u) - row);  // #{j : T[j] <= u}
  const int32_t m = std::min(count, ctx->h_last[i]);
  const size_t link = (size_t)i * M + m;
  ctx->pending_peer[i] = m;
  ctx->pending_weight[i] = (m == i) ? 0.0f : ctx->h_w[link];
  ctx->pending_duration[i] = ctx->t_iter[link];
  ctx->finish[i] = start + ctx->pending_duration[i];
}

int netmax_async_begin(netmax_ctx* ctx, const double* t_iter, double beta) {
  if (!ctx) return fail(nullptr, NETMAX_INVALID_ARG, "ctx is NULL");
  if (ctx->rounds != ctx->round0) return fail(ctx, NETMAX_INVALID_ARG, "netmax_async_begin must precede any netmax_round");
  if (!(beta >= 0.0 && beta < 1.0)) return fail(ctx, NETMAX_INVALID_ARG, "beta = %g outside [0, 1)", beta);
  const int32_t M = ctx->M;
  if (t_iter) {
    for (size_t k = 0; k < (size_t)M * M; ++k) {
      const int i = (int)(k / M), m = (int)(k % M);
      const bool used = (i == m) || ctx->adj[k];
      if (used && !(t_iter[k] > 0.0 && std::isfinite(t_iter[k])))
        return fail(ctx, NETMAX_INVALID_ARG, "t_iter[%d,%d] = %g must be positive and finite", i, m, t_iter[k]);
    }
    ctx->t_iter.assign(t_iter, t_iter + (size_t)M * M);
  }
  ctx->async_on = true;
  ctx->beta = beta;
  ctx->now = 0.0;
  ctx->steps = 0;
  ctx->local_n.assign(M, 0);
  ctx->pending_peer.assign(M, 0);
  ctx->pending_weight.assign(M, 0.0f);
  ctx->pending_duration.assign(M, 0.0);
  ctx->finish.assign(M, 0.0);
  ctx->ema.assign((size_t)M * M, 0.0);
  ctx->ema_count.assign((size_t)M * M, 0);
  ctx->ev_cap = std::max<int64_t>(ctx->trace_rounds * (int64_t)M, 1024);
  ctx->ev_worker.assign(ctx->ev_cap, 0);
  ctx->ev_peer.assign(ctx->ev_cap, 0);
  ctx->ev_n.assign(ctx->ev_cap, 0);
  ctx->ev_time.assign(ctx->ev_cap, 0.0);
  ctx->queue = decltype(ctx->queue)();
  for (int i = 0; i < M; ++i) {
    async_start_iteration(ctx, i, 0.0);
    ctx->queue.emplace(ctx->finish[i], i);
  }
  return NETMAX_OK;
}

int netmax_async_set_times(netmax_ctx* ctx, const double* t_iter) {
  if (!ctx) return fail(nullptr, NETMAX_INVALID_ARG, "ctx is NULL");
  if (!t_iter) return fail(ctx, NETMAX_INVALID_ARG, "t_iter is NULL");
  ctx->t_iter.assign(t_iter, t_iter + (size_t)ctx->M * ctx->M);
  return NETMAX_OK;
}

// Network Monitor (Algorithm 1): collect the workers' moving averages of iteration times, run
// Algorithm 3 on them and send P and rho back.  An average that has seen n samples is read as
// T / (1 - beta^n) (Algorithm 2 starts T at 0); a link that was never sampled is taken at its
// current iteration time.  An infeasible grid leaves the policy in force.
static int monitor_refresh(netmax_ctx* ctx) {
  const int32_t M = ctx->M;
  std::vector<double> t((size_t)M * M, 0.0);
  for (size_t at = 0; at < (size_t)M * M; ++at) {
    const int i = (int)(at / M), m = (int)(at % M);
    if (i != m && !ctx->adj[at]) continue;
    const int64_t n = ctx->ema_count[at];
    t[at] = n > 0 ? ctx->ema[at] / (1.0 - std::pow(ctx->beta, (double)n)) : ctx->t_iter[at];
  }
  std::vector<double> P((size_t)M * M);
  double rho = 0.0;
  int ndev = 0;
  const bool fixed = ctx->pull_weight > 0.0;  // constant pull weight: the extension section's form of Algorithm 3
  const bool on_device = !fixed && M >= 512 && cudaGetDeviceCount(&ndev) == cudaSuccess && ctx->device < ndev;
  double floor_sel = 0.0;
  int rc = fixed ? netmax_policy_generate_fixed_weight(M, t.data(), ctx->adj.data(), ctx->pull_weight, ctx->policy_K, ctx->policy_R,
                                                       ctx->policy_rho_upper, P.data(), &floor_sel, nullptr)
           : on_device ? netmax_policy_generate_device(M, t.data(), ctx->adj.data(), ctx->alpha, ctx->policy_K, ctx->policy_R,
                                                     ctx->policy_rho_upper, ctx->device, ctx->stream, P.data(), &rho, nullptr)
                     : netmax_policy_generate_ex(M, t.data(), ctx->adj.data(), ctx->alpha, ctx->policy_K, ctx->policy_R,
                                                 ctx->policy_rho_upper, P.data(), &rho, nullptr);
  if (rc == NETMAX_INFEASIBLE) return NETMAX_OK;
  if (rc) return fail(ctx, rc, "%s", netmax_last_error(nullptr));
  ctx->P.swap(P);
  if (!fixed) ctx->rho = rho;
  ctx->monitor_refreshes += 1;
  NM_CUDA(ctx, cudaStreamSynchronize(ctx->stream));
  return upload_policy(ctx);
}

int netmax_async_monitor(netmax_ctx* ctx, double period_s) {
  if (!ctx) return fail(nullptr, NETMAX_INVALID_ARG, "ctx is NULL");
  if (!ctx->async_on) return fail(ctx, NETMAX_INVALID_ARG, "call netmax_async_begin first");
  if (!(period_s >= 0.0) || !std::isfinite(period_s)) return fail(ctx, NETMAX_INVALID_ARG, "period_s = %g", period_s);
  ctx->monitor_period = period_s;
  ctx->monitor_next = ctx->now + period_s;
  return NETMAX_OK;
}

int64_t netmax_async_monitor_refreshes(const netmax_ctx* ctx) { return ctx ? ctx->monitor_refreshes : -1; }

int netmax_async_steps(netmax_ctx* ctx, int64_t n_steps) {
  if (!ctx) return fail(nullptr, NETMAX_INVALID_ARG, "ctx is NULL");
  if (!ctx->async_on) return fail(ctx, NETMAX_INVALID_ARG, "call netmax_async_begin first");
  if (n_steps < 0) return fail(ctx, NETMAX_INVALID_ARG, "n_steps = %lld < 0", (long long)n_steps);
  DeviceGuard guard(ctx->device);
  const int32_t M = ctx->M;
  StepKernel kernel = pick_step_kernel(ctx->objective, ctx->L.halves);
  StepParams p;
  p.x = reinterpret_cast<float4*>(ctx->x[ctx->cur]);
  p.c = reinterpret_cast<const float4*>(ctx->c);
  p.nq = ctx->L.nq;
  p.row_bytes = (uint32_t)(ctx->L.ld * ctx->L.elem);
  p.tail = (int32_t)(ctx->d % (4 * ctx->L.halves));
  p.alpha = (float)ctx->alpha;
  p.sigma = noise_scale(ctx);
  p.q_offset = ctx->q_offset;
  p.n_events = 0;
  p.keys = ctx->keys;
  std::vector<uint8_t> writes(M, 0), reads(M, 0);
  auto flush = [&]() -> int {
    if (p.n_events == 0) return NETMAX_OK;
    const int64_t want = (ctx->L.nq + kThreads - 1) / kThreads;
    const int64_t cap = std::max<int64_t>(1, (int64_t)8 * ctx->sm_count / p.n_events);
    dim3 grid((unsigned)std::min<int64_t>(want, cap), (unsigned)p.n_events);
    kernel<<<grid, kThreads, 0, ctx->stream>>>(p);
    ctx->launches += 1;
    NM_CUDA(ctx, cudaGetLastError());
    for (int e = 0; e < p.n_events; ++e) {
      writes[p.ev[e].worker] = 0;
      reads[p.ev[e].worker] = 0;
      reads[p.ev[e].peer] = 0;
    }
    p.n_events = 0;
    return NETMAX_OK;
  };
  for (int64_t k = 0; k < n_steps; ++k) {
    // the next global step: the worker whose iteration finishes first (ties: lowest index)
    const int i = ctx->queue.top().second;
    // the Network Monitor wakes up before any step at or after its next period boundary
    while (ctx->monitor_period > 0.0 && ctx->finish[i] >= ctx->monitor_next) {
      int rc = flush();
      if (!rc) rc = monitor_refresh(ctx);
      if (rc) return rc;
      ctx->monitor_next += ctx->monitor_period;
    }
    const int m = ctx->pending_peer[i];
    // a launch holds steps on disjoint replicas only: this one must not write a row that an
    // earlier step of the launch reads or writes, nor read a row that one writes
    if (p.n_events == kMaxStepEvents || writes[i] || reads[i] || writes[m]) {
      int rc = flush();
      if (rc) return rc;
    }
    const uint64_t n = (uint64_t)ctx->local_n[i];
    StepEvent& e = p.ev[p.n_events++];
    e.worker = i;
    e.peer = m;
    e.iter_lo = (uint32_t)n;
    e.ctr3 = philox_ctr3(kTagNoise, n);
    e.w = ctx->pending_weight[i];
    writes[i] = 1;
    reads[i] = 1;
    reads[m] = 1;
    // bookkeeping of Algorithm 2: the clock, the EMA of the iteration time, the next iteration
    ctx->now = ctx->finish[i];
    const int64_t slot = ctx->steps % ctx->ev_cap;
    ctx->ev_worker[slot] = i;
    ctx->ev_peer[slot] = m;
    ctx->ev_n[slot] = (int64_t)n;
    ctx->ev_time[slot] = ctx->now;
    const size_t at = (size_t)i * M + m;
    ctx->ema[at] = ctx->beta * ctx->ema[at] + (1.0 - ctx->beta) * ctx->pending_duration[i];
    ctx->ema_count[at] += 1;
    ctx->local_n[i] += 1;
    ctx->steps += 1;
    async_start_iteration(ctx, i, ctx->now);
    ctx->queue.pop();
    ctx->queue.emplace(ctx->finish[i], i);
  }
  return flush();
}

int netmax_async_time(netmax_ctx* ctx, double* sim_time, int64_t* steps_done) {
  if (!ctx) return fail(nullptr, NETMAX_INVALID_ARG, "ctx is NULL");
  if (!ctx->async_on) return fail(ctx, NETMAX_INVALID_ARG, "call netmax_async_begin first");
  if (sim_time) *sim_time = ctx->now;
  if (steps_done) *steps_done = ctx->steps;
  return NETMAX_OK;
}

int netmax_async_trace(netmax_ctx* ctx, int64_t first_step, int64_t n, int32_t* worker, int32_t* peer, int64_t* local_iter,
                       double* finish_time) {
  if (!ctx) return fail(nullptr, NETMAX_INVALID_ARG, "ctx is NULL");
  if (!ctx->async_on) return fail(ctx, NETMAX_INVALID_ARG, "call netmax_async_begin first");
  if (first_step < 0 || n < 0 || first_step + n > ctx->steps || first_step < ctx->steps - ctx->ev_cap)
    return fail(ctx, NETMAX_TRACE_RANGE, "steps [%lld, %lld) are not in the ring (steps done %lld, capacity %lld)",
                (long long)first_step, (long long)(first_step + n), (long long)ctx->steps, (long long)ctx->ev_cap);
  for (int64_t k = 0; k < n; ++k) {
    const int64_t slot = (first_step + k) % ctx->ev_cap;
    if (worker) worker[k] = ctx->ev_worker[slot];
    if (peer) peer[k] = ctx->ev_peer[slot];
    if (local_iter) local_iter[k] = ctx->ev_n[slot];
    if (finish_time) finish_time[k] = ctx->ev_time[slot];
  }
  return NETMAX_OK;
}

int netmax_async_ema(netmax_ctx* ctx, double* ema_out, int64_t* samples_out) {
  if (!ctx) return fail(nullptr, NETMAX_INVALID_ARG, "ctx is NULL");
  if (!ctx->async_on) return fail(ctx, NETMAX_INVALID_ARG, "call netmax_async_begin first");
  if (ema_out) std::memcpy(ema_out, ctx->ema.data(), ctx->ema.size() * sizeof(double));
  if (samples_out) std::memcpy(samples_out, ctx->ema_count.data(), ctx->ema_count.size() * sizeof(int64_t));
  return NETMAX_OK;
}

int netmax_debug_absent_ctas(netmax_ctx* ctx, int32_t n) {
  if (!ctx) return fail(nullptr, NETMAX_INVALID_ARG, "ctx is NULL");
  if (n < 0 || n > 1024) return fail(ctx, NETMAX_INVALID_ARG, "n = %d outside [0, 1024]", n);
  ctx->inject_absent_ctas = (uint32_t)n;
  return NETMAX_OK;
}

int64_t netmax_kernel_launches(const netmax_ctx* ctx) { return ctx ? ctx->launches : -1; }

const char* netmax_last_error(const netmax_ctx* ctx) { return ctx ? ctx->error.c_str() : g_error.c_str(); }

}  // extern "C"
