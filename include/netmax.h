/*
 * netmax.h -- C ABI of the NetMax round simulator for one NVIDIA B200 (sm_100a).
 *
 * NetMax (arXiv 2009.05766) is decentralised consensus SGD: worker i repeatedly (a) picks a
 * peer m with probability p_im from its row of the communication policy matrix P
 * (Algorithm 2, "select a neighbour m with probability p_im"), (b) takes a local SGD step
 * x_i^{k+1/2} = x_i^k - alpha g_i^k (Eq. 15), and (c) pulls the peer's parameters,
 * x_i^{k+1} = x_i^{k+1/2} - alpha rho gamma_im (x_i^{k+1/2} - x_m^k),
 * gamma_im = (d_im + d_mi) / (2 p_im) (Eq. 16).  This library keeps all M replicas in one
 * GPU's memory and advances them in synchronous ROUNDS: in a round every worker does one
 * such iteration, and every pull reads the peer's replica as it was at the start of the
 * round.  Objectives are f_i(x) = 1/2 ||x - c_i||^2 with additive N(0, sigma^2) gradient
 * noise (the paper's additive-noise assumption), or zero gradients.
 *
 * Conventions
 *   - Every function returns NETMAX_OK (0) or a negative netmax_status; none throws,
 *     aborts or leaves the CUDA context in a sticky error state of its own making.
 *   - "host" pointers are ordinary CPU memory, "device" pointers are CUDA device memory on
 *     the context's device.  Inputs are borrowed for the duration of the call and copied;
 *     outputs are caller-allocated and caller-owned.
 *   - Matrices are row-major M x M; replica arrays are dense row-major M x d (no padding).
 *   - Rounds are numbered from netmax_config.first_round (default 0) over the life of a context.  All random numbers are
 *     Philox4x32-10 blocks addressed by (seed, stream, worker, round, element), so splitting
 *     netmax_round(a + b) into netmax_round(a); netmax_round(b) changes no bit.
 *   - Work is enqueued on the context's stream.  Calls that return data to the host
 *     synchronise that stream first.  A context is not thread-safe.
 */
#ifndef NETMAX_H_
#define NETMAX_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum netmax_status {
  NETMAX_OK = 0,
  NETMAX_INVALID_ARG = -1,    /* null pointer, size out of range, non-finite parameter        */
  NETMAX_BAD_PROB_ROW = -2,   /* a row of P has a negative entry or does not sum to 1 (1e-9)  */
  NETMAX_OOM = -3,            /* device or host allocation failed / workspace too small       */
  NETMAX_CUDA_ERROR = -4,     /* a CUDA call failed; see netmax_last_error                    */
  NETMAX_TRACE_RANGE = -5,    /* requested rounds are not (or no longer) in the ring          */
  NETMAX_NOT_CONNECTED = -6,  /* the link graph is not connected (Assumption 1)               */
  NETMAX_INFEASIBLE = -7      /* Algorithm 3 found no feasible (rho, t_bar) grid point        */
} netmax_status;

typedef struct netmax_ctx netmax_ctx; /* opaque; created and destroyed by the library */

/*
 * Precision of the state kept in device memory (netmax_config.storage).  The paper trains in
 * fp32, which is the default.  NETMAX_STORAGE_BF16 is an option of this library: replicas and
 * centres are held as bfloat16 (half the memory and half the traffic per element), Eq. 15 and
 * Eq. 16 are still evaluated in fp32, in the order
 *   t = x - c;  g = fma(sigma, z, t);  h = fma(-alpha, g, x);  x' = fma(-w, h - x_m, h),
 * and each new parameter is rounded once to the nearest bfloat16 (ties to even) when it is
 * stored.  An update smaller than half a bfloat16 unit of the parameter is therefore lost --
 * the known price of narrow storage.  Host-side arrays stay fp32 in every call: values passed
 * in are rounded to bfloat16, values read back are widened exactly.
 */
enum { NETMAX_STORAGE_F32 = 0, NETMAX_STORAGE_BF16 = 1 };

/*
 * Full configuration of a context (Algorithm 2's inputs alpha, rho and P, plus what the
 * simulator adds: sizes, the synthetic objective, the seed and where to run).
 */
typedef struct netmax_config {
  int32_t M;                     /* workers, 2 <= M <= 16384                                          */
  int64_t d;                     /* parameters per replica, 1 <= d < 2^30 - 32                        */
  int64_t element_offset;        /* logical index of this context's first element inside a longer global
                                    vector (a multiple of 4 -- of 8 with bfloat16 storage --, offset + d <
                                    2^30 - 32; default 0).  Only the
                                    noise / initialisation counters use it: contexts that hold disjoint
                                    column ranges of one problem (one per GPU) then draw the streams the
                                    single-context run would, and never need to exchange data            */
  const double* link_speed_gbps; /* host, M*M, symmetric, diagonal ignored; speed <= 0 means "no link"
                                    (d_im = 0).  NULL means fully connected with equal speeds          */
  const double* prob;            /* host, M*M, row i = P[i,:].  NULL: run Algorithm 3 on the iteration
                                    times derived from link_speed_gbps (policy_K x policy_R grid); with
                                    pull_weight > 0 in the form for a constant weight
                                    (netmax_policy_generate_fixed_weight)                              */
  double lr;                     /* alpha > 0; the update uses its fp32 rounding                       */
  double rho;                    /* rho; <= 0: with prob given, the largest rho meeting Eq. 11 with a
                                    1e-6 margin, min_{p_im>0} p_im / (alpha (d_im+d_mi)); with prob
                                    NULL, the rho Algorithm 3 selects.  A rho > 0 that breaks Eq. 11
                                    (alpha rho (d_im+d_mi) > p_im on a link with p_im > 0, i.e. a pull
                                    weight above 1/2) is rejected with NETMAX_INVALID_ARG unless
                                    pull_weight replaces Eq. 16's weight                               */
  double pull_weight;            /* 0 (default): Eq. 16's weight alpha rho (d_im+d_mi)/(2 p_im).  In (0, 1):
                                    every pull uses this constant instead -- the update rule of gossip /
                                    AD-PSGD style averaging (1/2), which the paper's section on extending
                                    existing decentralised PSGD approaches writes in the same form
                                    x <- D (x - alpha g); rho is then unused                             */
  double sigma;                  /* std of the gradient noise; the update uses its fp32 rounding       */
  double x0_std, c_std;          /* x_i(0) ~ N(0, x0_std^2), c_i ~ N(0, c_std^2), drawn from the seed  */
  int32_t objective;             /* 0: zero gradients (sigma ignored); 1: f_i = 1/2 ||x - c_i||^2      */
  uint64_t seed;                 /* Philox key                                                         */
  int32_t device;                /* CUDA device ordinal                                                */
  void* stream;                  /* cudaStream_t to enqueue on (NULL: the legacy default stream)       */
  int64_t trace_rounds;          /* capacity of the peer-trace / telemetry ring, in rounds (>= 1)      */
  int32_t policy_K, policy_R;    /* Algorithm 3 grid sizes when prob is NULL (<= 0: 20 x 20)           */
  double policy_rho_upper;       /* upper end of Algorithm 3's rho grid (<= 0: default cap; see
                                    netmax_policy_generate_ex); with pull_weight > 0 the upper end of
                                    the floor grid of netmax_policy_generate_fixed_weight              */
  void* workspace;               /* device memory for ALL of the context's device buffers, 256-byte
                                    aligned, at least netmax_workspace_size() bytes, owned by the
                                    caller and kept alive until netmax_destroy.  NULL: the library
                                    allocates with cudaMalloc and frees in netmax_destroy              */
  size_t workspace_bytes;
  int32_t storage;               /* NETMAX_STORAGE_F32 (default) or NETMAX_STORAGE_BF16: see above       */
  int32_t fuse_rounds;           /* rounds that one launch may advance a tile of long vectors while it is
                                    resident on chip (see netmax_round): 0 (default) automatic, 1 never
                                    (one launch per round; short vectors then do not keep columns in shared
                                    memory either), 2..8 at most that many (four over a cluster).  Replicas and peer traces do
                                    not depend on it                                                     */
  int64_t first_round;           /* number of the context's first round, 0 <= first_round < 2^56 (default 0).  Rounds are
                                    numbered from here; the round number is a word of every Philox counter, so a run
                                    that is resumed from saved replicas at round r (netmax_set_replicas) with
                                    first_round = r continues the streams of the run it was saved from               */
} netmax_config;

/* Fills *cfg with defaults: rho = 0 (automatic), sigma = 0, stds 0, objective 1, seed 0,
 * device 0, stream NULL, trace_rounds 1024, policy grid 20 x 20, no workspace, offset 0,
 * fp32 storage, first round 0. */
int netmax_config_init(netmax_config* cfg);

/* Device bytes a context with this M, d, trace_rounds and storage needs (only those fields are read). */
int netmax_workspace_size(const netmax_config* cfg, size_t* bytes);

/*
 * Creates a context: validates, builds the 32-bit cumulative-threshold table and the
 * pull-weight table w_im = alpha rho (d_im + d_mi) / (2 p_im) (Eq. 16) on the host, uploads
 * them, and fills x(0) and c on the device from the seed.  *out is NULL on failure.
 */
int netmax_create_ex(const netmax_config* cfg, netmax_ctx** out);

/* Short form: objective 1, sigma = 0, x0_std = c_std = 1, automatic rho, current device,
 * default stream, library-allocated memory.  link_speed_gbps and prob as in netmax_config. */
int netmax_create(int32_t M, int64_t d, const double* link_speed_gbps, const double* prob, double lr,
                  uint64_t seed, netmax_ctx** out);

void netmax_destroy(netmax_ctx* ctx);

/*
 * Replaces P, the link graph and rho between rounds (Algorithm 2: "if received new policy").
 * Arguments as in netmax_config; prob == NULL reruns Algorithm 3; link_speed_gbps == NULL
 * keeps the current graph.  Takes effect from the next round.
 */
int netmax_set_policy(netmax_ctx* ctx, const double* link_speed_gbps, const double* prob, double rho);

/* Reads back the policy in force: prob_out (host, M*M) and *rho_out; either may be NULL. */
int netmax_get_policy(netmax_ctx* ctx, double* prob_out, double* rho_out);

/* Overwrite all replicas / all centres from dense host arrays of M*d floats.  A bfloat16
 * context rounds them on the device; the buffer of the double buffer that holds no replicas
 * at that moment is the staging area, so nothing is allocated. */
int netmax_set_replicas(netmax_ctx* ctx, const float* host_x);
int netmax_set_centres(netmax_ctx* ctx, const float* host_c);

/*
 * Runs n_rounds rounds (n_rounds >= 0), asynchronously on the context's stream.  Per round:
 * the peer of every worker is drawn (Algorithm 2), then ONE fused kernel applies Eq. 15 and
 * Eq. 16 to every element of every replica, reading the round-start buffer and writing the
 * other one, and reduces that round's telemetry.  The peers of up to trace_rounds rounds are
 * drawn ahead in one sampler launch (the draws are counter-based and do not depend on x).
 * Short vectors (a round of a few microseconds) whose M rows of at least one four-element column
 * group fit in a CTA's shared memory (M up to about 4700) run all rounds of a call on
 * shared-memory-resident columns: CTAs own disjoint columns and never exchange anything.  A call
 * has to run enough rounds to repay bringing the columns on chip (2 for up to a million elements,
 * up to 16 for the largest problems); shorter calls take the per-round kernels.
 * Other short-vector shapes (and fuse_rounds = 1) run all rounds of a call in one cooperative
 * launch with a grid-wide barrier per round; its waits are bounded, and one that runs out is
 * reported by the next synchronising call as NETMAX_CUDA_ERROR (the replicas are then not
 * valid).
 * Long vectors with at most 36 workers advance up to eight rounds per launch
 * (netmax_config.fuse_rounds): given the draws, Eq. 16 acts on every column separately, so a
 * tile holding all M rows of a column range stays in shared memory for those rounds and HBM
 * sees x and c once per launch instead of once per round.  With 37 to 144 workers (fp32 state)
 * the rows of such a tile are split over the CTAs of a thread-block cluster (4 to 8 of them,
 * by the number of workers), a pull reads the peer's row from the shared memory of the CTA
 * that holds it, and a launch advances up to four rounds; with fuse_rounds = 0 this shape is taken only where it was measured faster than
 * one launch per round (37 to 66 workers and most counts up to 88), with fuse_rounds >= 2
 * wherever it fits.
 * Whatever the launch shape and however a run is split into calls, replicas and peer traces
 * are the same bit for bit; telemetry sums are accumulated in an order that depends on the
 * launch shape and agree to fp32 rounding of their partial sums (2e-5 relative or better).
 */
int netmax_round(netmax_ctx* ctx, int64_t n_rounds);

/*
 * A whole step through host buffers in one call: replaces the replicas by host_x and the centres by
 * host_c (either may be NULL: keep what the context holds), runs n_rounds rounds and copies the
 * resulting replicas to host_out -- what netmax_set_replicas, netmax_set_centres, netmax_round and
 * netmax_read_replicas do one after the other, with the same replicas, peer trace, telemetry and
 * round counter bit for bit.  Given the draws, Eq. 15-16 act on every column separately, so the work
 * is cut into n_chunks column ranges (0: automatic; at most 32) and pipelined: while the rounds of
 * one range run on the context's stream, the next range is uploaded and the previous one downloaded
 * on two streams of the library's own.  All arrays are dense M*d floats on the host; pinned memory
 * lets the copies overlap.  Ranges are pipelined for fp32 state, long vectors and
 * 1 <= n_rounds <= trace_rounds; otherwise the call runs the four steps in turn.  Synchronises.
 */
int netmax_round_from_host(netmax_ctx* ctx, const float* host_x, const float* host_c, int64_t n_rounds, float* host_out,
                           int32_t n_chunks);

/* Changes netmax_config.fuse_rounds for the rounds that follow (0 automatic, 1 one launch per
 * round, 2..8 at most that many rounds per launch). */
int netmax_set_fuse_rounds(netmax_ctx* ctx, int32_t fuse_rounds);

/* Number of the next round: netmax_config.first_round plus the rounds enqueued so far. */
int64_t netmax_rounds_done(const netmax_ctx* ctx);

/* Synchronises, then copies the current replicas to host_out (M*d floats, dense; bfloat16
 * state is widened exactly). */
int netmax_read_replicas(netmax_ctx* ctx, float* host_out);
/* Same for the centres c_i. */
int netmax_read_centres(netmax_ctx* ctx, float* host_out);

/*
 * Copies the values of the listed logical element indices (0 <= cols[k] < d) of every
 * replica to host_out (M*n_cols floats, row-major): a cheap way to inspect large replicas.
 */
int netmax_read_columns(netmax_ctx* ctx, const int64_t* host_cols, int64_t n_cols, float* host_out);

/*
 * netmax_read_columns without any allocation.  (The paper has no counterpart: this is a
 * convenience of the library, like netmax_read_columns itself.)
 *
 * netmax_read_columns stages the column list and the gathered values in temporaries that it
 * cudaMallocs and frees on every call.  Some callers must not do that: a process whose
 * device memory is entirely handed to a pool allocator (the reason netmax_config.workspace
 * exists) can see cudaMalloc fail or take memory the pool counts on; a monitoring loop that
 * polls a few parameters between rounds does not want the device-wide synchronisation that
 * cudaMalloc / cudaFree imply; and code that runs where the CUDA runtime forbids allocation
 * cannot call it at all.  This variant runs the same gather kernel, but stages through a
 * fixed array that lives in the library image (a file-scope __device__ array of
 * NETMAX_STATIC_MAX_COLS * 8 + NETMAX_STATIC_MAX_VALUES * 4 bytes, about 1.03 MB, present on
 * every GPU that loads the library until the process exits).  It calls no cudaMalloc,
 * cudaFree or other allocating routine.
 *
 * Arguments and result are those of netmax_read_columns.  Limits: n_cols <=
 * NETMAX_STATIC_MAX_COLS and M * n_cols <= NETMAX_STATIC_MAX_VALUES; beyond either the call
 * returns NETMAX_INVALID_ARG and touches nothing (split the list and call again).
 *
 * The first call on a device looks up the array's device address (cudaGetSymbolAddress,
 * once per device, cached); make that first call before any stream capture begins.  All
 * calls, from every context on the device, share the one array: it still holds the previous
 * call's data (nothing in it needs to start at zero, every slot that is read back is
 * written first), and two calls whose GPU work overlaps -- different streams, or different
 * host threads -- race on it.  Calls on one stream are ordered and safe.  Synchronises the
 * context's stream before returning, like netmax_read_columns.
 */
#define NETMAX_STATIC_MAX_COLS 4096
#define NETMAX_STATIC_MAX_VALUES 262144
int netmax_read_columns_static(netmax_ctx* ctx, const int64_t* host_cols, int64_t n_cols, float* host_out);

/*
 * Peers drawn in rounds [first_round, first_round + n): host_out[(r - first_round) * M + i]
 * is the peer of worker i in round r (an absolute round number, >= netmax_config.first_round).
 * Only the last trace_rounds rounds are kept; NETMAX_TRACE_RANGE otherwise.  Synchronises.
 */
int netmax_peer_trace(netmax_ctx* ctx, int64_t first_round, int64_t n, int32_t* host_out);

/*
 * Telemetry of rounds [first_round, first_round + n), measured on each round's START state:
 * consensus[r] = (1/M) sum_i ||x_i - mean_j x_j||^2 and loss[r] = (1/M) sum_i 1/2 ||x_i - c_i||^2
 * (the two parts of the consensus objective, Eq. 1, that the simulator observes).  Either
 * output may be NULL.  Same ring rule as netmax_peer_trace.  Synchronises.
 */
int netmax_telemetry(netmax_ctx* ctx, int64_t first_round, int64_t n, double* host_consensus, double* host_loss);

/*
 * Telemetry of the CURRENT replicas, on demand: the same two quantities as netmax_telemetry
 * (consensus distance and mean loss, the observable parts of Eq. 1), computed by one
 * read-only kernel.  Either output may be NULL.  Synchronises.
 */
int netmax_measure(netmax_ctx* ctx, double* consensus, double* loss);

/*
 * Asynchronous timeline: the paper's own process (Section II-B and Eq. 17), in which workers
 * run on their own clocks and exactly ONE worker updates at every global step.
 *
 * Worker i's local iteration n draws its peer m from P[i,:] (Algorithm 2; the peer stream at
 * counter (worker i, iteration n)), lasts t_im = max{C_i, N_im} (t_ii for a self-draw) and is
 * followed at once by iteration n + 1.  Global step k belongs to the worker whose iteration
 * finishes next (ties: the lowest index); it applies Eq. 15 and Eq. 16 to x_i IN PLACE with the
 * peer's replica as it is at that moment (x_m^k in Eq. 17), then folds the iteration time into
 * its moving average T_i[m] <- beta T_i[m] + (1 - beta) t_im (Algorithm 2, UpdateTimeVector;
 * T starts at 0).  A policy set with netmax_set_policy, and the iteration times that come
 * with new link speeds, apply to iterations that START afterwards (Algorithm 2: "if received
 * new policy").  The clocks and draws are host control plane; the replica updates run on the
 * GPU, consecutive steps on disjoint replicas sharing a launch.
 *
 * netmax_async_begin switches a context that has run no round to this timeline for good
 * (netmax_round is refused afterwards).  t_iter (host, M*M, t_ii on the diagonal) overrides
 * the iteration times derived from the context's link speeds; NULL keeps those.
 */
int netmax_async_begin(netmax_ctx* ctx, const double* t_iter, double beta);
/* Replaces the iteration-time matrix (host, M*M) for iterations that start afterwards. */
int netmax_async_set_times(netmax_ctx* ctx, const double* t_iter);
/* Runs the next n_steps global steps, asynchronously on the context's stream. */
int netmax_async_steps(netmax_ctx* ctx, int64_t n_steps);
/*
 * Network Monitor (Algorithm 1) on the simulated clock: every period_s simulated seconds,
 * before the first global step at or after the boundary, the moving averages T_i[m] are
 * collected, Algorithm 3 runs on them (policy_K x policy_R grid) and the resulting P and rho are
 * installed for iterations that start afterwards.  An average with n samples is read as
 * T / (1 - beta^n) (Algorithm 2 starts T at 0); a link never sampled so far is taken at its
 * current iteration time; a grid with no feasible point leaves the policy unchanged.  A context
 * with a constant pull weight runs netmax_policy_generate_fixed_weight instead ("AD-PSGD with a
 * Network Monitor").
 * period_s = 0 switches the monitor off.  netmax_async_monitor_refreshes counts the policies
 * installed so far.
 */
int netmax_async_monitor(netmax_ctx* ctx, double period_s);
int64_t netmax_async_monitor_refreshes(const netmax_ctx* ctx);
/* Simulated time of the last global step and the number of global steps so far. */
int netmax_async_time(netmax_ctx* ctx, double* sim_time, int64_t* steps_done);
/*
 * The global steps [first_step, first_step + n): which worker acted, the peer it pulled from,
 * its local iteration number and the simulated finish time.  Host arrays of n entries, any of
 * which may be NULL.  The last max(trace_rounds * M, 1024) steps are kept.
 */
int netmax_async_trace(netmax_ctx* ctx, int64_t first_step, int64_t n, int32_t* worker, int32_t* peer,
                       int64_t* local_iter, double* finish_time);
/* The moving averages T_i[m] (host, M*M) and how many samples each has seen (may be NULL):
 * what the Network Monitor of Algorithm 1 collects. */
int netmax_async_ema(netmax_ctx* ctx, double* ema_out, int64_t* samples_out);

/*
 * Device access for callers that keep working on the GPU (for example through PyTorch):
 * *x is the buffer holding the current replicas, row i at x + i * ld, ld >= d floats,
 * valid until the next netmax_round / netmax_set_* / netmax_read_replicas call; nothing is
 * synchronised.  In a bfloat16 context the buffer holds bfloat16 values: cast the pointer;
 * ld then counts bfloat16 elements.
 */
int netmax_replicas_device(netmax_ctx* ctx, const float** x, int64_t* ld);

/*
 * Peer draws alone (the sampler of Algorithm 2), for n_rounds rounds starting at
 * first_round, written to device_out (device, n_rounds*M int32), asynchronously on the
 * context's stream; does not advance the context's round counter.
 */
int netmax_sample_peers(netmax_ctx* ctx, int64_t first_round, int64_t n_rounds, int32_t* device_out);

/*
 * Host control plane.  Iteration-time model (Section II-B: t_im = max{C_i, N_im}):
 * N_im = 32 d / (s_im 1e9) s, C_i = min N / 4, t_ii = C_i.  t_out (M*M) and adj_out (M*M,
 * 0/1) are host arrays.
 */
int netmax_iteration_times(int32_t M, int64_t d, const double* link_speed_gbps, double* t_out, uint8_t* adj_out);

/*
 * Algorithm 3 (communication policy generation): searches K values of rho and, for each,
 * R values of the average iteration time t_bar; at every grid point solves the row-wise LP
 * (Eq. 14 under Eq. 10-13), forms Y_P = E[D^T D] (Eq. 22), and keeps the point minimising
 * t_bar ln(eps) / ln(lambda_2).  All arrays are host memory; prob_out is M*M.  info_out,
 * if not NULL, receives {lambda_2, t_bar, t_convergence (eps = 1e-3), k, r}.
 */
int netmax_policy_generate(int32_t M, const double* t_iter, const uint8_t* adj, double lr, int32_t K, int32_t R,
                           double* prob_out, double* rho_out, double* info_out /* 5 doubles */);

/*
 * The same with the upper end of the rho grid given explicitly: rho_k = k rho_upper / K.
 * rho_upper <= 0 is the default (the grid ends where the Eq. 11 floors alone fill a row).
 * 0.5 / lr is the U_rho Algorithm 3 prints; most of that grid is infeasible for M > 2, so a
 * coarse K then selects a smaller rho and a P that favours fast links more strongly.
 */
int netmax_policy_generate_ex(int32_t M, const double* t_iter, const uint8_t* adj, double lr, int32_t K, int32_t R,
                              double rho_upper, double* prob_out, double* rho_out, double* info_out);

/*
 * Algorithm 3 for a pull rule with a CONSTANT weight w (netmax_config.pull_weight): the paper's
 * section on extending existing decentralised PSGD approaches (gossip / AD-PSGD style averaging,
 * x_i <- (1 - w)(x_i - alpha g_i) + w x_m) asks for two steps.  First, Eq. 11 is replaced by the
 * condition that every entry y_im of E[D^T D] on a link is positive; with a constant weight
 * y_im = (w - w^2)(p_i p_im + p_m p_mi), so the condition is p_im + p_mi > 0, taken here as a floor
 * phi on both directions of every link.  Second, the optimisation problem (Eq. 8-13) is solved
 * again: phi takes rho's place in the outer loop (phi_k = k floor_upper / K; floor_upper <= 0: the
 * value at which the floors alone fill a row), t_bar is searched in the inner loop (the midpoints of R
 * cells between the least and the largest mean time the floors allow), and the grid
 * point minimising t_bar ln(eps) / ln(lambda_2) is kept.  Y_P is doubly stochastic only if, besides
 * Eq. 10, the columns of P sum to 1, which couples the rows; among the feasible P with p_ii = 0 the
 * one of maximum entropy above the floors is returned (rows, columns and mean iteration times are
 * met to 1e-9).  The link graph must be symmetric.  Host arrays; info_out as in
 * netmax_policy_generate; *floor_out receives the selected phi.
 */
int netmax_policy_generate_fixed_weight(int32_t M, const double* t_iter, const uint8_t* adj, double pull_weight, int32_t K,
                                        int32_t R, double floor_upper, double* prob_out, double* floor_out,
                                        double* info_out /* 5 doubles or NULL */);

/* One grid point of the search above: the maximum-entropy P with p_im >= floor on every link, zero
 * diagonal, rows and columns summing to 1 and a mean iteration time of M t_bar in every row (Eq. 10);
 * NETMAX_INFEASIBLE if there is none.  Host arrays; prob_out is M*M. */
int netmax_policy_fixed_weight_at(int32_t M, const double* t_iter, const uint8_t* adj, double floor, double t_bar,
                                  double* prob_out);

/*
 * Algorithm 3 on the GPU, for large M (thousands of workers, links redrawn often): the same
 * grids, the same row-wise LP optimum and the same selection as netmax_policy_generate, with
 * one CTA per row of P, Y_P (Eq. 22) kept in device memory and lambda_2 by Lanczos on the
 * device.  Host arrays in and out as for netmax_policy_generate; allocates its own device
 * buffers (about 4 M*M doubles) on `device` and works on `stream` (a cudaStream_t, may be
 * NULL); synchronises before returning.  Results agree with the host generator to rounding.
 */
int netmax_policy_generate_device(int32_t M, const double* t_iter, const uint8_t* adj, double lr, int32_t K, int32_t R,
                                  double rho_upper /* as in netmax_policy_generate_ex */, int32_t device, void* stream, double* prob_out, double* rho_out,
                                  double* info_out /* 5 doubles or NULL */);

/*
 * Test hook for the bounded waits of multi-round launches (short vectors, netmax_round(n >= 2)):
 * the NEXT such launch also waits, at its grid-wide barrier, for n CTAs that do not exist, so
 * every wait runs out (about two seconds), the kernel returns after its first round and the
 * next synchronising call reports NETMAX_CUDA_ERROR; the replicas are then not valid and should
 * be set again.  Nothing faults or hangs, and the context stays usable.  n = 0 cancels.
 */
int netmax_debug_absent_ctas(netmax_ctx* ctx, int32_t n);

/* Counters for benchmarks: kernels launched by this context so far. */
int64_t netmax_kernel_launches(const netmax_ctx* ctx);

/* Message of the last failure on this context ("" if none); ctx == NULL: the last failure
 * of a call that had no context (creation).  The string is owned by the library. */
const char* netmax_last_error(const netmax_ctx* ctx);

#ifdef __cplusplus
}
#endif
#endif /* NETMAX_H_ */
