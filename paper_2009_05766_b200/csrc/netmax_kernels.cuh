// CUDA kernels of the NetMax round simulator (sm_100a).
//
//   sample_peers_kernel   Algorithm 2, peer selection: one Philox draw per (round, worker)
//                         searched in that worker's row of 32-bit cumulative thresholds.
//   round_kernel          Eq. 15 (local SGD step with inline Gaussian gradient noise) fused
//                         with Eq. 16 (pull from the round-start snapshot of the peer) and
//                         with the round's telemetry; reads one buffer, writes the other.
//   fused_rounds_kernel   the same for up to four rounds per launch on tiles that stay in a
//                         CTA's shared memory (long vectors, up to 36 workers).
//   cluster_rounds_kernel the same with the rows of a tile split over the CTAs of a thread-block
//                         cluster, pulls through distributed shared memory (up to 144 workers).
//   resident_rounds_kernel, multi_round_kernel   short vectors: all rounds of a call in one launch.
//   step_kernel           the asynchronous timeline: one worker per global step (Eq. 17).
//   init_normal_kernel    x(0) and c from the seed.
//   gather_columns_kernel sampled read-back.
//
// State precision.  The replicas and centres are stored as fp32 (kHalves == 1) or, as an option
// the paper does not have, as bfloat16 (kHalves == 2).  Either way a thread moves 16-byte column
// groups -- 4 fp32 or 8 bfloat16 values, i.e. kHalves Philox blocks of four normals -- and all
// arithmetic is fp32: bfloat16 values are widened exactly on load, and each new parameter is
// rounded once, to the nearest bfloat16 (ties to even), at the store.
#pragma once
#include <cstdint>
#include <type_traits>
#include <cuda_runtime.h>

#include "netmax_rng.cuh"

namespace netmax {

// ------------------------------------------------------------------------- sampler
struct SampleParams {
  const uint32_t* thresholds;  // [M][M] non-decreasing per row
  const int32_t* last_nz;      // [M] last index with p > 0
  int32_t* out;                // slot s of round r is out + ((slot0 + r) % ring) * M
  float* w_out;                // same indexing: pull weight of the draw (0 on a self-draw); may be NULL
  const float* wtab;           // [M][M] pull weights (read when w_out is given)
  int64_t slot0, ring;
  uint64_t first_round;
  int64_t n_rounds;
  int32_t M;
  PhiloxKeys keys;
};

// m = min(#{j : T[j] <= u}, last_nz): the count is found by bisection (T is sorted).
__global__ void __launch_bounds__(256) sample_peers_kernel(const SampleParams p) {
  const int64_t total = p.n_rounds * (int64_t)p.M;
  for (int64_t idx = blockIdx.x * (int64_t)blockDim.x + threadIdx.x; idx < total;
       idx += (int64_t)gridDim.x * blockDim.x) {
    const int64_t r = idx / p.M;
    const int32_t i = (int32_t)(idx - r * p.M);
    const uint64_t round = p.first_round + (uint64_t)r;
    const uint32_t u = philox4x32_10(0u, (uint32_t)i, (uint32_t)round, philox_ctr3(kTagPeer, round), p.keys).x;
    const uint32_t* __restrict__ row = p.thresholds + (size_t)i * p.M;
    int32_t lo = 0, hi = p.M;
    while (lo < hi) {
      const int32_t mid = (lo + hi) >> 1;
      if (__ldg(row + mid) <= u) lo = mid + 1; else hi = mid;
    }
    const int32_t m = min(lo, __ldg(p.last_nz + i));
    const int64_t at = ((p.slot0 + r) % p.ring) * p.M + i;
    p.out[at] = m;
    if (p.w_out) p.w_out[at] = (m == i) ? 0.0f : __ldg(p.wtab + (size_t)i * p.M + m);
  }
}

// ------------------------------------------------------------------------- round
struct RoundParams {
  const float4* x_cur;   // [M][ldq] round-start replicas (16-byte column groups: 4 fp32 or 8 bfloat16)
  float4* x_nxt;         // [M][ldq] next replicas
  const float4* c;       // [M][ldq] centres
  const int32_t* peers;  // [M] this round's draws
  const float* wtab;     // [M][M] pull weights w_im (fp32)
  double* partials;      // [gridDim.x][2] per-CTA telemetry sums
  unsigned int* ticket;  // last-CTA-done counter (0 between launches)
  double* tel_out;       // [2] this round's (consensus, loss)
  int64_t ldq;           // row stride, in column groups
  uint32_t row_bytes;    // row stride, in bytes (< 2^32)
  int64_t nq;            // column groups per row = ceil(d / (4 kHalves))
  int64_t n_tiles;       // ceil(nq / cg)
  int32_t M;
  int32_t tail;          // d % (4 kHalves): live lanes of the last column group (0 = all of them)
  int32_t cg;            // column groups per tile   (cg * rl == blockDim.x, both powers of two)
  int32_t rl;            // row lanes per tile
  int32_t rg;            // row groups: tile t covers column tile t / rg, rows of group t % rg
  int32_t rows_per_group;  // ceil(M / rg)
  float4* colpart;       // rg > 1: per tile, per column group, per half: (sum, sum of squares) partials
  unsigned int* coltick; // rg > 1: arrivals per column tile (0 between launches)
  float alpha, sigma;    // sigma: the noise scale sigma sqrt(2 ln 2) (see update_core_rnd)
  float inv_M;
  uint32_t round_lo, ctr3;
  uint32_t q_offset;     // Philox block index (element / 4) of the context's first element in the global vector
  PhiloxKeys keys;
};

// Per-thread telemetry accumulators.  ColAcc: four columns as two fp32 pairs, sum (x - pivot)
// and sum (x - pivot)^2 over the rows the thread has seen.  LossAcc: sum (x - c)^2 over all of
// the thread's elements.
struct ColAcc {
  pair_t s1a = 0ull, s1b = 0ull, s2a = 0ull, s2b = 0ull;  // +0.0f pairs
};
struct LossAcc {
  pair_t la = 0ull, lb = 0ull;
};

// Four bfloat16 values in a 64-bit word (element 0 in the lowest 16 bits) <-> two fp32 pairs.
// Widening is exact; narrowing rounds to nearest, ties to even.
__device__ __forceinline__ ulonglong2 widen_bf16x4(unsigned long long v) {
  const uint32_t lo = (uint32_t)v, hi = (uint32_t)(v >> 32);
  return make_ulonglong2(pack2(__uint_as_float(lo << 16), __uint_as_float(lo & 0xFFFF0000u)),
                         pack2(__uint_as_float(hi << 16), __uint_as_float(hi & 0xFFFF0000u)));
}
__device__ __forceinline__ unsigned long long narrow_bf16x4(ulonglong2 v) {
  float e0, e1, e2, e3;
  unpack2(v.x, e0, e1);
  unpack2(v.y, e2, e3);
  uint32_t lo, hi;
  asm("cvt.rn.bf16x2.f32 %0, %1, %2;" : "=r"(lo) : "f"(e1), "f"(e0));  // first operand -> upper half
  asm("cvt.rn.bf16x2.f32 %0, %1, %2;" : "=r"(hi) : "f"(e3), "f"(e2));
  return ((unsigned long long)hi << 32) | lo;
}
// Half h (four elements, as two fp32 pairs) of a 16-byte column group.
template <int kHalves>
__device__ __forceinline__ ulonglong2 group_half(ulonglong2 raw, int h) {
  if (kHalves == 1) return raw;
  return widen_bf16x4(h == 0 ? raw.x : raw.y);
}
// Live lanes of half h of a column group: 4 everywhere but in a row's last, ragged group.
__device__ __forceinline__ int live_lanes(bool ragged, int tail, int h) {
  return ragged ? min(4, max(0, tail - 4 * h)) : 4;
}

// Per-lane noise scale of one column group (fused_rounds_kernel): sigma_s on real elements, 0 on the padding lanes of a
// row's last, ragged group.  Padding lanes hold x = c = 0 in every row; with no noise Eq. 15-16
// keep them at exactly +0 (every product and sum below is +0 or -0 + +0), so nothing has to be
// masked after the update.
struct NoiseLanes {
  pair_t a, b;
};
__device__ __forceinline__ NoiseLanes noise_lanes(float sigma_s, int live) {
  NoiseLanes n;
  n.a = pack2(live > 0 ? sigma_s : 0.0f, live > 1 ? sigma_s : 0.0f);
  n.b = pack2(live > 2 ? sigma_s : 0.0f, live > 3 ? sigma_s : 0.0f);
  return n;
}

// Eq. 15 and Eq. 16 on one column group of one worker, on packed fp32 pairs:
//   g = (x - c) + sigma z,  h = x - alpha g                                       (Eq. 15)
//   x' = h - w (h - x_m),   w = alpha rho gamma_im  (w = 0 on a self-draw)          (Eq. 16)
// rnd is the Philox block of the four elements (counter: global index of the block, worker,
// round or -- on the asynchronous timeline -- the worker's local iteration); ns holds, per lane,
// sigma sqrt(2 ln 2), the noise scale with the constant factor of the Box-Muller radius folded in
// (fast path; the accurate path takes it out again), or 0 on padding lanes; nw2 is (-w, -w).
// ta, tb return x - c for the caller's loss statistic.
template <int kObjective, bool kFastNoise>
__device__ __forceinline__ ulonglong2 update_core_rnd(float alpha, const NoiseLanes& ns, uint4 rnd, ulonglong2 xv, ulonglong2 cv,
                                                      ulonglong2 xm, pair_t nw2, pair_t& ta, pair_t& tb) {
  const pair_t neg1 = pack2(-1.0f, -1.0f);
  ta = fma2(cv.x, neg1, xv.x);  // x - c
  tb = fma2(cv.y, neg1, xv.y);
  pair_t ha = xv.x, hb = xv.y;
  if (kObjective == 1) {
    const pair_t nalpha2 = pack2(-alpha, -alpha);
    pair_t za, zb, sa = ns.a, sb = ns.b;
    if (kFastNoise) {
      za = normal_pair_fast_unscaled(rnd.x, rnd.y);
      zb = normal_pair_fast_unscaled(rnd.z, rnd.w);
    } else {
      const pair_t inv = pack2((float)(1.0 / kNormalScale), (float)(1.0 / kNormalScale));
      sa = mul2(sa, inv);
      sb = mul2(sb, inv);
      const float4 z = normals4<false>(rnd);
      za = pack2(z.x, z.y);
      zb = pack2(z.z, z.w);
    }
    ha = fma2(nalpha2, fma2(sa, za, ta), xv.x);
    hb = fma2(nalpha2, fma2(sb, zb, tb), xv.y);
  }
  const pair_t oa = fma2(nw2, fma2(xm.x, neg1, ha), ha);
  const pair_t ob = fma2(nw2, fma2(xm.y, neg1, hb), hb);
  return make_ulonglong2(oa, ob);
}

// The Philox block of the noise of one column group of one worker (only drawn when there is noise).
template <int kObjective>
__device__ __forceinline__ uint4 noise_block(const PhiloxKeys& keys, uint32_t iter_lo, uint32_t ctr3, uint32_t q32, uint32_t worker) {
  if (kObjective != 1) return make_uint4(0u, 0u, 0u, 0u);
  return philox4x32_10(q32, worker, iter_lo, ctr3, keys);
}

// The same update with the Philox block drawn inside, for the kernels that stream rows through
// registers (round_kernel, step_kernel) or walk them one at a time (resident_rounds_kernel).  One
// noise scale serves all four lanes and the padding lanes of a ragged group (`live` < 4 real
// elements) are cleared after the update: the streaming kernel runs at its register limit, and
// this form -- one scale pair instead of NoiseLanes' two, the masking behind a branch that is
// almost never taken -- measured 191 us per round against 223 on 8 x 11.2 M elements.  Real lanes
// see exactly the arithmetic of update_core_rnd, so all kernels agree bit for bit.
template <int kObjective, bool kFastNoise>
__device__ __forceinline__ ulonglong2 update_core(float alpha, float sigma_s, const PhiloxKeys& keys,
                                                  uint32_t iter_lo, uint32_t ctr3, uint32_t q32, uint32_t worker,
                                                  ulonglong2 xv, ulonglong2 cv, ulonglong2 xm, float w, int live,
                                                  pair_t& ta, pair_t& tb) {
  const pair_t neg1 = pack2(-1.0f, -1.0f);
  const pair_t nw2 = pack2(-w, -w);
  ta = fma2(cv.x, neg1, xv.x);  // x - c
  tb = fma2(cv.y, neg1, xv.y);
  pair_t ha = xv.x, hb = xv.y;
  if (kObjective == 1) {
    pair_t sig2 = pack2(sigma_s, sigma_s);
    const pair_t nalpha2 = pack2(-alpha, -alpha);
    const uint4 rnd = philox4x32_10(q32, worker, iter_lo, ctr3, keys);
    pair_t za, zb;
    if (kFastNoise) {
      za = normal_pair_fast_unscaled(rnd.x, rnd.y);
      zb = normal_pair_fast_unscaled(rnd.z, rnd.w);
    } else {
      sig2 = mul2(sig2, pack2((float)(1.0 / kNormalScale), (float)(1.0 / kNormalScale)));
      const float4 z = normals4<false>(rnd);
      za = pack2(z.x, z.y);
      zb = pack2(z.z, z.w);
    }
    ha = fma2(nalpha2, fma2(sig2, za, ta), xv.x);
    hb = fma2(nalpha2, fma2(sig2, zb, tb), xv.y);
  }
  pair_t oa = fma2(nw2, fma2(xm.x, neg1, ha), ha);
  pair_t ob = fma2(nw2, fma2(xm.y, neg1, hb), hb);
  if (live < 4) {  // keep the padding lanes of the last group at zero
    float o0, o1, o2, o3;
    unpack2(oa, o0, o1);
    unpack2(ob, o2, o3);
    if (live < 1) o0 = 0.f;
    if (live < 2) o1 = 0.f;
    if (live < 3) o2 = 0.f;
    oa = pack2(o0, o1);
    ob = pack2(o2, 0.f);
  }
  return make_ulonglong2(oa, ob);
}

// update_core plus the telemetry sums of the round-start values.  kObjective == 2 measures only.
template <int kObjective, bool kFastNoise>
__device__ __forceinline__ ulonglong2 row_update_rnd(float alpha, const NoiseLanes& ns, uint4 rnd, ulonglong2 xv, ulonglong2 cv,
                                                     ulonglong2 xm, ulonglong2 pivot, pair_t nw2, ColAcc& acc, LossAcc& lacc) {
  const pair_t neg1 = pack2(-1.0f, -1.0f);
  pair_t ta, tb;
  ulonglong2 o = xv;
  if (kObjective == 2) {
    ta = fma2(cv.x, neg1, xv.x);
    tb = fma2(cv.y, neg1, xv.y);
  } else {
    o = update_core_rnd<kObjective, kFastNoise>(alpha, ns, rnd, xv, cv, xm, nw2, ta, tb);
  }
  const pair_t da = fma2(pivot.x, neg1, xv.x), db = fma2(pivot.y, neg1, xv.y);  // x - pivot
  acc.s1a = add2(acc.s1a, da);
  acc.s1b = add2(acc.s1b, db);
  acc.s2a = fma2(da, da, acc.s2a);
  acc.s2b = fma2(db, db, acc.s2b);
  lacc.la = fma2(ta, ta, lacc.la);
  lacc.lb = fma2(tb, tb, lacc.lb);
  return o;
}

template <int kObjective, bool kFastNoise>
__device__ __forceinline__ ulonglong2 row_update(float alpha, float sigma_s, const PhiloxKeys& keys, uint32_t round_lo,
                                                 uint32_t ctr3, uint32_t q32, uint32_t worker, ulonglong2 xv, ulonglong2 cv,
                                                 ulonglong2 xm, ulonglong2 pivot, float w, int live, ColAcc& acc,
                                                 LossAcc& lacc) {
  const pair_t neg1 = pack2(-1.0f, -1.0f);
  pair_t ta, tb;
  ulonglong2 o = xv;
  if (kObjective == 2) {
    ta = fma2(cv.x, neg1, xv.x);
    tb = fma2(cv.y, neg1, xv.y);
  } else {
    o = update_core<kObjective, kFastNoise>(alpha, sigma_s, keys, round_lo, ctr3, q32, worker, xv, cv, xm, w, live, ta, tb);
  }
  const pair_t da = fma2(pivot.x, neg1, xv.x), db = fma2(pivot.y, neg1, xv.y);  // x - pivot
  acc.s1a = add2(acc.s1a, da);
  acc.s1b = add2(acc.s1b, db);
  acc.s2a = fma2(da, da, acc.s2a);
  acc.s2b = fma2(db, db, acc.s2b);
  lacc.la = fma2(ta, ta, lacc.la);
  lacc.lb = fma2(tb, tb, lacc.lb);
  return o;
}

// Block reduction of a CTA's two telemetry sums into partials[2 * blockIdx.x ..].
// s_red: 64 doubles of shared memory.  Every thread of the CTA must call this.
__device__ __forceinline__ void block_partials(double* partials, double acc_cons, double acc_loss, double* s_red) {
  const int tid = threadIdx.x;
  acc_loss *= 0.5;
  for (int off = 16; off > 0; off >>= 1) {
    acc_cons += __shfl_down_sync(0xffffffffu, acc_cons, off);
    acc_loss += __shfl_down_sync(0xffffffffu, acc_loss, off);
  }
  const int warp = tid >> 5, lane = tid & 31, nwarps = blockDim.x >> 5;
  __syncthreads();  // s_red may still be read by an earlier call
  if (lane == 0) {
    s_red[warp] = acc_cons;
    s_red[32 + warp] = acc_loss;
  }
  __syncthreads();
  if (tid == 0) {
    double a = 0.0, b = 0.0;
    for (int wi = 0; wi < nwarps; ++wi) {
      a += s_red[wi];
      b += s_red[32 + wi];
    }
    partials[2 * (size_t)blockIdx.x] = a;
    partials[2 * (size_t)blockIdx.x + 1] = b;
  }
}

// Adds all CTA partials in index order (deterministic) and writes the round's telemetry.
// Every thread of the (one) calling CTA must call this.
__device__ __forceinline__ void sum_partials(const double* partials, double inv_M, double* tel_out, double* s_red) {
  const int tid = threadIdx.x;
  const int warp = tid >> 5, lane = tid & 31, nwarps = blockDim.x >> 5;
  double a = 0.0, b = 0.0;
  for (unsigned int j = tid; j < gridDim.x; j += blockDim.x) {
    a += __ldcg(partials + 2 * (size_t)j);
    b += __ldcg(partials + 2 * (size_t)j + 1);
  }
  for (int off = 16; off > 0; off >>= 1) {
    a += __shfl_down_sync(0xffffffffu, a, off);
    b += __shfl_down_sync(0xffffffffu, b, off);
  }
  __syncthreads();
  if (lane == 0) {
    s_red[warp] = a;
    s_red[32 + warp] = b;
  }
  __syncthreads();
  if (tid == 0) {
    a = 0.0;
    b = 0.0;
    for (int wi = 0; wi < nwarps; ++wi) {
      a += s_red[wi];
      b += s_red[32 + wi];
    }
    tel_out[0] = a * inv_M;
    tel_out[1] = b * inv_M;
  }
}

// One launch per round: the last CTA of the grid to publish its partials sums them.
__device__ __forceinline__ void finalize_telemetry(const RoundParams& p, double acc_cons, double acc_loss, double* s_red) {
  block_partials(p.partials, acc_cons, acc_loss, s_red);
  __shared__ bool s_last;
  if (threadIdx.x == 0) {
    __threadfence();
    const unsigned int t = atomicAdd(p.ticket, 1u);
    s_last = (t == gridDim.x - 1);
  }
  __syncthreads();
  if (s_last) {
    __threadfence();
    sum_partials(p.partials, (double)p.inv_M, p.tel_out, s_red);
    if (threadIdx.x == 0) *p.ticket = 0u;
  }
}

// Direct-load round kernel (any M).  One tile = all M rows (or, for short vectors with many
// workers, one of rg row groups) x cg column groups.  Thread (cgi, rli) owns column group cgi
// of the tile and the rows rli, rli + rl, ... of its row group; tiles are taken round-robin by
// the resident CTAs.  All accesses are plain cacheable 128-bit loads and
// stores: the peer read (a row this tile reads anyway) then hits L1/L2, and streaming hints on
// c and on the output measured slower.
// Dynamic shared memory: (peer, weight) int2[M], then (rl > 1) 2 * kHalves * blockDim float4 of
// column-sum scratch, then 64 doubles for the block reduction.
#ifndef NETMAX_ROUND_MIN_CTAS
#define NETMAX_ROUND_MIN_CTAS 4  // CTAs per SM the register allocation leaves room for
#endif
#ifndef NETMAX_ROUND_MIN_CTAS_BF16
#define NETMAX_ROUND_MIN_CTAS_BF16 2  // bfloat16 state: eight elements per thread; measured 152 us (2), 161 (3), 157 (4) per cfg2 round
#endif

// kRowsInFlight = 1 (64 registers, 4 CTAs/SM) is the streaming shape for long vectors, where
// occupancy hides the HBM latency; kRowsInFlight = 4 (2 CTAs/SM) serves short, L2-resident
// problems, where a thread's chain of dependent row loads is what takes the time.
// this round's (peer, weight) of workers [r0, r1) into shared memory
__device__ __forceinline__ void load_draws(const RoundParams& p, const int32_t* peers, int2* s_pw, int r0, int r1) {
  for (int i = r0 + threadIdx.x; i < r1; i += blockDim.x) {
    const int32_t m = __ldg(peers + i);
    s_pw[i] = make_int2(m, __float_as_int((m == i) ? 0.0f : __ldg(p.wtab + (size_t)i * p.M + m)));
  }
}

// 16 bytes from global to shared memory without passing through registers or L1 (data that no other
// thread of the SM will ask for); completion is awaited by the same thread with cp_async_wait_all.
__device__ __forceinline__ void cp_async_16_stream(void* smem_dst, const void* gmem_src) {
  const uint32_t dst = (uint32_t)__cvta_generic_to_shared(smem_dst);
  asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(dst), "l"(gmem_src) : "memory");
}
// The same for 8 bytes (four bfloat16 values; copies below 16 bytes go through L1).
__device__ __forceinline__ void cp_async_8(void* smem_dst, const void* gmem_src) {
  const uint32_t dst = (uint32_t)__cvta_generic_to_shared(smem_dst);
  asm volatile("cp.async.ca.shared.global [%0], [%1], 8;" ::"r"(dst), "l"(gmem_src) : "memory");
}
__device__ __forceinline__ void cp_async_wait_all() { asm volatile("cp.async.wait_all;" ::: "memory"); }

// Loads of replica data.  Inside one launch per round the round-start buffer is read-only
// (non-coherent path); a launch that runs several rounds reads what other SMs wrote a round
// earlier and must bypass L1.
template <bool kCoherent>
__device__ __forceinline__ ulonglong2 ld_x(const char* ptr) {
  return kCoherent ? __ldcg(reinterpret_cast<const ulonglong2*>(ptr)) : __ldg(reinterpret_cast<const ulonglong2*>(ptr));
}

// All tiles of this CTA for one round.  Every thread of the CTA must call this.
template <int kObjective, bool kFastNoise, int kRowsInFlight, bool kCoherent, int kHalves>
__device__ __forceinline__ void round_tiles(const RoundParams& p, const float4* x_cur, float4* x_nxt, const int32_t* peers,
                                            uint32_t round_lo, uint32_t ctr3, int2* s_pw, float4* s_col,
                                            double& acc_cons, double& acc_loss) {
  constexpr int kStats = 2 * kHalves;  // float4 column statistics per thread: (sum, sum of squares) per half
  const int tid = threadIdx.x;
  const int G = p.rg;
  __shared__ bool s_lastcol;
  const int cgi = tid & (p.cg - 1);
  const int rli = tid / p.cg;
  const int M = p.M;
  const int step = p.rl;
  if (G == 1 && kObjective != 2) {
    __syncthreads();  // readers of the previous round's draws are done
    load_draws(p, peers, s_pw, 0, M);
    __syncthreads();
  }

  for (int64_t tile = blockIdx.x; tile < p.n_tiles; tile += gridDim.x) {
    const int64_t ct = G == 1 ? tile : tile / G;      // column tile
    const int grp = G == 1 ? 0 : (int)(tile - ct * G);  // row group
    const int r0 = grp * p.rows_per_group, r1 = min(M, r0 + p.rows_per_group);
    if (G > 1 && kObjective != 2) {
      __syncthreads();  // the previous tile's readers of s_pw are done
      load_draws(p, peers, s_pw, r0, r1);
      __syncthreads();
    }
    const int64_t q = ct * p.cg + cgi;
    const bool live = q < p.nq;
    const bool ragged = (p.tail != 0) && (q == p.nq - 1);
    float4 st[kStats];  // st[2h] = sum (x - pivot), st[2h + 1] = sum (x - pivot)^2 of half h's columns
#pragma unroll
    for (int a = 0; a < kStats; ++a) st[a] = make_float4(0.f, 0.f, 0.f, 0.f);
    float loss = 0.f;
    if (live) {
      // byte pointers to this thread's column group in row 0; row i is i * row_bytes further
      const char* xq = reinterpret_cast<const char*>(x_cur + q);
      const char* cq = reinterpret_cast<const char*>(p.c + q);
      char* oq = reinterpret_cast<char*>(x_nxt + q);
      const uint32_t q32 = (uint32_t)q * kHalves + p.q_offset;
      const ulonglong2 pivot = ld_x<kCoherent>(xq);  // row 0: pivot of the one-pass variance
      ColAcc acc[kHalves];
      LossAcc lacc;
      for (int i0 = r0 + rli; i0 < r1; i0 += step * kRowsInFlight) {
        ulonglong2 xv[kRowsInFlight], xm[kRowsInFlight], cv[kRowsInFlight];
        int2 pw[kRowsInFlight];
#pragma unroll
        for (int u = 0; u < kRowsInFlight; ++u) {  // issue the loads of kRowsInFlight rows
          const int i = i0 + u * step;
          if (kRowsInFlight == 1 || i < r1) {
            const uint64_t row = (uint64_t)(uint32_t)i * p.row_bytes;
            xv[u] = ld_x<kCoherent>(xq + row);
            if (kObjective == 2) {  // measuring: no peers involved
              pw[u] = make_int2(i, 0);
              xm[u] = xv[u];
            } else {
              pw[u] = s_pw[i];
              xm[u] = ld_x<kCoherent>(xq + (uint64_t)(uint32_t)pw[u].x * p.row_bytes);
            }
            cv[u] = __ldg(reinterpret_cast<const ulonglong2*>(cq + row));
          }
        }
#pragma unroll
        for (int u = 0; u < kRowsInFlight; ++u) {
          const int i = i0 + u * step;
          if (kRowsInFlight == 1 || i < r1) {
            ulonglong2 o;
#pragma unroll
            for (int h = 0; h < kHalves; ++h) {
              const ulonglong2 oh = row_update<kObjective, kFastNoise>(
                  p.alpha, p.sigma, p.keys, round_lo, ctr3, q32 + h, (uint32_t)i, group_half<kHalves>(xv[u], h), group_half<kHalves>(cv[u], h),
                  group_half<kHalves>(xm[u], h), group_half<kHalves>(pivot, h), __int_as_float(pw[u].y),
                  live_lanes(ragged, p.tail, h), acc[h], lacc);
              if (kHalves == 1) o = oh;
              else if (h == 0) o.x = narrow_bf16x4(oh);
              else o.y = narrow_bf16x4(oh);
            }
            if (kObjective != 2) *reinterpret_cast<ulonglong2*>(oq + (uint64_t)(uint32_t)i * p.row_bytes) = o;
          }
        }
      }
#pragma unroll
      for (int h = 0; h < kHalves; ++h) {
        unpack2(acc[h].s1a, st[2 * h].x, st[2 * h].y);
        unpack2(acc[h].s1b, st[2 * h].z, st[2 * h].w);
        unpack2(acc[h].s2a, st[2 * h + 1].x, st[2 * h + 1].y);
        unpack2(acc[h].s2b, st[2 * h + 1].z, st[2 * h + 1].w);
      }
      float l0, l1, l2, l3;
      unpack2(lacc.la, l0, l1);
      unpack2(lacc.lb, l2, l3);
      loss = (l0 + l1) + (l2 + l3);
    }
    if (p.rl > 1) {  // sum the column statistics over the row lanes (stride cg in tid)
#pragma unroll
      for (int a = 0; a < kStats; ++a) s_col[a * blockDim.x + tid] = st[a];
      __syncthreads();
      for (int s = blockDim.x >> 1; s >= p.cg; s >>= 1) {
        if (tid < s) {
#pragma unroll
          for (int a = 0; a < kStats; ++a) {
            float4 v = s_col[a * blockDim.x + tid];
            const float4 b = s_col[a * blockDim.x + tid + s];
            v.x += b.x; v.y += b.y; v.z += b.z; v.w += b.w;
            s_col[a * blockDim.x + tid] = v;
          }
        }
        __syncthreads();
      }
#pragma unroll
      for (int a = 0; a < kStats; ++a) st[a] = s_col[a * blockDim.x + cgi];
      __syncthreads();
    }
    bool owner = true;  // does this CTA hold the complete column sums of the tile?
    if (G > 1) {
      // rows are split over rg CTAs: publish this CTA's column partials; the last of the rg
      // CTAs of a column tile to arrive adds them up in group order (deterministic)
      if (rli == 0) {
#pragma unroll
        for (int a = 0; a < kStats; ++a) p.colpart[((size_t)tile * p.cg + cgi) * kStats + a] = st[a];
      }
      __threadfence();
      __syncthreads();
      if (tid == 0) {
        const unsigned int t = atomicAdd(p.coltick + ct, 1u);
        s_lastcol = (t == (unsigned int)G - 1);
        if (s_lastcol) p.coltick[ct] = 0u;
      }
      __syncthreads();
      owner = s_lastcol;
      if (owner && rli == 0) {
        __threadfence();
#pragma unroll
        for (int a = 0; a < kStats; ++a) st[a] = make_float4(0.f, 0.f, 0.f, 0.f);
        for (int gg = 0; gg < G; ++gg) {
#pragma unroll
          for (int a = 0; a < kStats; ++a) {
            const float4 b = __ldcg(p.colpart + (((size_t)ct * G + gg) * p.cg + cgi) * kStats + a);
            st[a].x += b.x; st[a].y += b.y; st[a].z += b.z; st[a].w += b.w;
          }
        }
      }
    }
    if (rli == 0 && owner) {
      // sum_i (x_i - xbar)^2 = sum_i (x_i - a)^2 - (sum_i (x_i - a))^2 / M   per column
#pragma unroll
      for (int h = 0; h < kHalves; ++h) {
        const float4 s1 = st[2 * h], s2 = st[2 * h + 1];
        const float cons = (s2.x - s1.x * s1.x * p.inv_M) + (s2.y - s1.y * s1.y * p.inv_M) +
                           (s2.z - s1.z * s1.z * p.inv_M) + (s2.w - s1.w * s1.w * p.inv_M);
        acc_cons += (double)cons;
      }
    }
    acc_loss += (double)loss;
  }
}

// kRowsInFlight = 1 (64 registers, 4 CTAs/SM) is the streaming shape for long vectors, where
// occupancy hides the HBM latency; kRowsInFlight = 4 (2 CTAs/SM) serves short, L2-resident
// problems, where a thread's chain of dependent row loads is what takes the time.
template <int kObjective, bool kFastNoise, int kRowsInFlight, int kHalves>
__global__ void __launch_bounds__(256, kRowsInFlight != 1 ? 2 : kHalves == 1 ? NETMAX_ROUND_MIN_CTAS : NETMAX_ROUND_MIN_CTAS_BF16)
    round_kernel(const RoundParams p) {
  extern __shared__ __align__(128) unsigned char smem_raw[];
  int2* s_pw = reinterpret_cast<int2*>(smem_raw);  // (peer, bits of the pull weight) per worker
  const size_t head = (((size_t)p.M * 8) + 15) & ~(size_t)15;
  float4* s_col = reinterpret_cast<float4*>(smem_raw + head);
  double* s_red = reinterpret_cast<double*>(smem_raw + head + (p.rl > 1 ? (size_t)blockDim.x * 32 * kHalves : 0));
  double acc_cons = 0.0, acc_loss = 0.0;
  round_tiles<kObjective, kFastNoise, kRowsInFlight, false, kHalves>(p, p.x_cur, p.x_nxt, p.peers, p.round_lo, p.ctr3, s_pw,
                                                                     s_col, acc_cons, acc_loss);
  finalize_telemetry(p, acc_cons, acc_loss, s_red);
}

// ---- several rounds in one launch (short, L2-resident problems) ------------------------------
// For problems of a few microseconds per round the launch and the chain of dependent global
// round trips are what take the time.  This kernel is launched cooperatively (all CTAs
// resident), runs n_rounds rounds back to back and separates them with a grid-wide barrier: an
// arrival counter in global memory that every CTA polls a bounded number of times.  A CTA
// whose wait runs out raises *error and leaves; the others then run out as well.
struct MultiRoundParams {
  RoundParams r;          // x_cur / x_nxt: the buffers of the first round; peers, tel_out, round_lo, ctr3 unused
  const int32_t* trace;   // peer-trace ring [ring][M], filled for these rounds by sample_peers_kernel
  double* tel;            // telemetry ring [ring][2]
  double* partials2;      // [2][gridDim.x][2]: CTA partials, alternating by round
  unsigned int* barrier;  // arrival counter, 0 at launch
  unsigned int* error;    // raised when a barrier wait gave up
  int64_t slot0, ring;    // ring slot of the first round
  uint64_t first_round;
  int32_t n_rounds;
  uint32_t absent_ctas;   // test hook: the barrier also waits for this many CTAs that do not exist
};

constexpr uint32_t kBarrierSpinLimit = 1u << 21;

// Grid-wide barrier number `epoch` (1, 2, ...).  Returns false if the wait gave up.
__device__ __forceinline__ bool grid_barrier(unsigned int* counter, unsigned int epoch, unsigned int* error,
                                             unsigned int absent_ctas) {
  __shared__ int s_ok;
  __syncthreads();
  if (threadIdx.x == 0) {
    __threadfence();  // this CTA's writes of the round are visible before it is counted
    atomicAdd(counter, 1u);
    const unsigned int target = epoch * (gridDim.x + absent_ctas);
    int ok = 0;
    for (uint32_t it = 0; it < kBarrierSpinLimit; ++it) {
      if (*reinterpret_cast<volatile unsigned int*>(counter) >= target) {
        ok = 1;
        break;
      }
      __nanosleep(32);
    }
    if (!ok) atomicExch(error, 1u);
    __threadfence();
    s_ok = ok;
  }
  __syncthreads();
  return s_ok != 0;
}

template <int kObjective, bool kFastNoise, int kHalves>
__global__ void __launch_bounds__(256, 2) multi_round_kernel(const MultiRoundParams mp) {
  extern __shared__ __align__(128) unsigned char smem_raw[];
  const RoundParams& p = mp.r;
  int2* s_pw = reinterpret_cast<int2*>(smem_raw);
  const size_t head = (((size_t)p.M * 8) + 15) & ~(size_t)15;
  float4* s_col = reinterpret_cast<float4*>(smem_raw + head);
  double* s_red = reinterpret_cast<double*>(smem_raw + head + (p.rl > 1 ? (size_t)blockDim.x * 32 * kHalves : 0));
  const float4* x_cur = p.x_cur;
  float4* x_nxt = p.x_nxt;
  for (int k = 0; k < mp.n_rounds; ++k) {
    const uint64_t round = mp.first_round + (uint64_t)k;
    const int64_t slot = (mp.slot0 + k) % mp.ring;
    double* partials = mp.partials2 + (size_t)(k & 1) * 2 * gridDim.x;
    double acc_cons = 0.0, acc_loss = 0.0;
    round_tiles<kObjective, kFastNoise, 4, true, kHalves>(p, x_cur, x_nxt, mp.trace + slot * p.M, (uint32_t)round,
                                                          philox_ctr3(kTagNoise, round), s_pw, s_col, acc_cons, acc_loss);
    block_partials(partials, acc_cons, acc_loss, s_red);
    if (!grid_barrier(mp.barrier, (unsigned int)(k + 1), mp.error, mp.absent_ctas)) return;
    // round k is complete everywhere: one CTA publishes its telemetry while the rest move on
    // (partials alternate, so round k+1 cannot overwrite what is being summed here)
    if (blockIdx.x == 0) sum_partials(partials, (double)p.inv_M, mp.tel + 2 * slot, s_red);
    const float4* t = x_cur;
    x_cur = x_nxt;
    x_nxt = const_cast<float4*>(t);
  }
}

// ---- several rounds over one resident tile (long vectors, few workers) -----------------------
// Given the peer draws, every column of the M x d state evolves on its own (Eq. 16 is
// elementwise), so a tile that holds ALL M rows of a column range can be advanced several
// rounds without touching global memory in between: the HBM traffic per element drops from
// 12 bytes per round (x and c read, x' written; the peer read is a cache hit) to 12 bytes per
// kFusedMaxRounds rounds, and the kernel becomes bound by its arithmetic instead.
//
// A thread owns one 16-byte column group for all M rows.  Its slab of shared memory
// ([2][M] replica values, double-buffered by round, and [M] centres, each entry 16 bytes,
// laid out [row][thread] so that a warp's accesses are conflict-free) is private to the thread:
// the peer's value of the same column group was written by this very thread a round earlier,
// so the rounds need no barrier.  Per-element arithmetic is row_update's, hence the replicas
// are bit-identical to one launch per round; telemetry sums only differ in the order of their
// double-precision accumulation.  The slabs always hold fp32; with bfloat16 state (kBf16) a
// thread's column group is four bfloat16 values (8 bytes of global memory), widened on the way
// in, and every round's result is rounded to bfloat16 before it is written to the slab, exactly
// as a store to and a load from the bfloat16 state would.
#ifndef NETMAX_FUSED_MAX_ROUNDS
#define NETMAX_FUSED_MAX_ROUNDS 8
#endif
#ifndef NETMAX_CLUSTER_MAX_ROUNDS
#define NETMAX_CLUSTER_MAX_ROUNDS 4
#endif
#ifndef NETMAX_FUSED_UNROLL
#define NETMAX_FUSED_UNROLL 2
#endif
#ifndef NETMAX_FUSED_PREFETCH
#define NETMAX_FUSED_PREFETCH 1  // fetch the next tile under the last round of the current one (fp32 state)
#endif
constexpr int kFusedMaxRounds = NETMAX_FUSED_MAX_ROUNDS;      // rounds per launch of fused_rounds_kernel, at most
constexpr int kClusterMaxRounds = NETMAX_CLUSTER_MAX_ROUNDS;  // of cluster_rounds_kernel (16 accumulator registers per four rounds: it has none to spare)
constexpr int kFusedUnroll = NETMAX_FUSED_UNROLL;  // rows of a round in flight per thread

struct FusedParams {
  const float4* x_cur;   // [M][ldq] replicas at the start of the first round
  float4* x_nxt;         // [M][ldq] replicas after the last round
  const float4* c;       // [M][ldq]
  const int32_t* trace;  // peer-trace ring [ring][M], filled for these rounds
  const float* wtab;     // [M][M]
  double* tel;           // telemetry ring [ring][2]
  double* partials;      // [kFusedMaxRounds][gridDim.x][2]
  unsigned int* ticket;  // last-CTA-done counter (0 between launches)
  int64_t slot0, ring;   // ring slot of the first round
  uint64_t first_round;
  int32_t n_rounds;      // 1 .. slots
  int32_t slots;         // rounds the table of draws at the head of the shared memory has room for (<= kFusedMaxRounds)
  int64_t nq, n_tiles;   // column groups of FOUR elements per row (whatever the storage), tiles of blockDim of them
  uint32_t row_bytes;
  int32_t M, tail;       // tail = d % 4
  float alpha, sigma, inv_M;
  uint32_t q_offset;
  PhiloxKeys keys;
};

// Dynamic shared memory: (peer row offset, -, -weight, -weight) int4[slots][M], then the slabs
// float4[3][M][blockDim] (replicas of even rounds, of odd rounds, centres), then 64 doubles.
// Any block size that is a multiple of 32 up to 256 works.
// kRounds: rounds a launch runs at most (4 or kFusedMaxRounds); a thread keeps two double accumulators per round,
// and a launch of up to four rounds runs 4 % faster on the instance that holds eight instead of sixteen of them.
template <int kObjective, bool kFastNoise, bool kBf16, int kRounds>
__global__ void __launch_bounds__(256, 2) fused_rounds_kernel(const FusedParams p) {
  constexpr uint32_t kGroupBytes = kBf16 ? 8u : 16u;  // four elements in global memory
  extern __shared__ __align__(128) unsigned char smem_raw[];
  const int tid = threadIdx.x, T = blockDim.x, M = p.M;
  int4* s_pw = reinterpret_cast<int4*>(smem_raw);  // (byte offset of the peer's row in a slab, unused, -w, -w)
  const uint32_t head = ((uint32_t)(p.slots * M * 16) + 127u) & ~127u;
  const uint32_t stride = (uint32_t)T * 16u;     // bytes between consecutive rows of a slab
  const uint32_t plane = (uint32_t)M * stride;   // bytes of one [M][T] slab
  unsigned char* slab = smem_raw + head + (uint32_t)tid * 16u;  // this thread's column: slabs 0, 1 (replicas), 2 (centres)
  double* s_red = reinterpret_cast<double*>(smem_raw + head + 3u * plane);

  for (int k = 0; k < p.n_rounds; ++k) {
    const int32_t* peers = p.trace + ((p.slot0 + k) % p.ring) * M;
    for (int i = tid; i < M; i += T) {
      const int32_t m = __ldg(peers + i);
      const int nw = __float_as_int((m == i) ? -0.0f : -__ldg(p.wtab + (size_t)i * M + m));
      s_pw[k * M + i] = make_int4((int)((uint32_t)m * stride), 0, nw, nw);
    }
  }
  __syncthreads();

  double acc_cons[kRounds], acc_loss[kRounds];
#pragma unroll
  for (int k = 0; k < kRounds; ++k) acc_cons[k] = acc_loss[k] = 0.0;

  // Slab `base` (0 or 1) holds the tile's values at the start of the first round; round k reads
  // slab (base + k) & 1 and writes the other one.  The LAST round of a tile writes its results
  // straight to global memory, which leaves its would-be output slab idle for that whole round:
  // the next tile's replicas are fetched into it (cp.async, fp32 state), and the next tile's centre
  // of a row replaces the current one as soon as that row has been updated for the last time.  The
  // global loads of a tile thus run under the last round of its predecessor.  Every slab slot is
  // read and written by its own thread only, so cp.async.wait_all is all the synchronisation needed.
  // bfloat16 state arrives as the 8 stored bytes in the low half of a 16-byte slot and is widened in
  // place when the tile starts.
  constexpr bool kPrefetch = NETMAX_FUSED_PREFETCH != 0;
  uint32_t base = 0;
  bool fetched = false;  // has this tile been fetched by the previous one?
  for (int64_t tile = blockIdx.x; tile < p.n_tiles; tile += gridDim.x) {
    const int64_t q = tile * T + tid;
    if (q >= p.nq) continue;  // no barrier below: threads are independent (and later tiles only have larger q)
    const NoiseLanes ns = noise_lanes(p.sigma, live_lanes((p.tail != 0) && (q == p.nq - 1), p.tail, 0));
    const uint32_t q32 = (uint32_t)q + p.q_offset;
    const int64_t q_next = q + (int64_t)gridDim.x * T;
    const bool have_next = kPrefetch && tile + gridDim.x < p.n_tiles && q_next < p.nq;
    if (fetched) {
      cp_async_wait_all();
      if (kBf16) {
        unsigned char* sx = slab + base * plane;
        unsigned char* sc = slab + 2u * plane;
#pragma unroll 4
        for (int i = 0; i < M; ++i) {
          *reinterpret_cast<ulonglong2*>(sx) = widen_bf16x4(*reinterpret_cast<const unsigned long long*>(sx));
          *reinterpret_cast<ulonglong2*>(sc) = widen_bf16x4(*reinterpret_cast<const unsigned long long*>(sc));
          sx += stride;
          sc += stride;
        }
      }
    } else {  // all rows of this column group into the thread's slabs
      const char* xq = reinterpret_cast<const char*>(p.x_cur) + (uint64_t)q * kGroupBytes;
      const char* cq = reinterpret_cast<const char*>(p.c) + (uint64_t)q * kGroupBytes;
      unsigned char* sx = slab + base * plane;
      unsigned char* sc = slab + 2u * plane;
#pragma unroll 4
      for (int i = 0; i < M; ++i) {
        if (kBf16) {
          *reinterpret_cast<ulonglong2*>(sx) = widen_bf16x4(__ldg(reinterpret_cast<const unsigned long long*>(xq)));
          *reinterpret_cast<ulonglong2*>(sc) = widen_bf16x4(__ldg(reinterpret_cast<const unsigned long long*>(cq)));
        } else {
          *reinterpret_cast<ulonglong2*>(sx) = __ldg(reinterpret_cast<const ulonglong2*>(xq));
          *reinterpret_cast<ulonglong2*>(sc) = __ldg(reinterpret_cast<const ulonglong2*>(cq));
        }
        xq += p.row_bytes;
        cq += p.row_bytes;
        sx += stride;
        sc += stride;
      }
    }
    unsigned char* const cen = slab + 2u * plane;
    char* const oq = reinterpret_cast<char*>(p.x_nxt) + (uint64_t)q * kGroupBytes;
    const char* const cq_next = reinterpret_cast<const char*>(p.c) + (uint64_t)q_next * kGroupBytes;

    // one round over the thread's column group; kLast: the tile's last round (see above)
    auto run_round = [&](int k, auto last_tag) {
      constexpr bool kLast = decltype(last_tag)::value;
      const uint64_t round = p.first_round + (uint64_t)k;
      const uint32_t round_lo = (uint32_t)round, ctr3 = philox_ctr3(kTagNoise, round);
      const unsigned char* cur = slab + ((base + (uint32_t)k) & 1u) * plane;
      unsigned char* nxt = slab + ((base + (uint32_t)k + 1u) & 1u) * plane;
      if (kLast && have_next) {
        const char* xq = reinterpret_cast<const char*>(p.x_cur) + (uint64_t)q_next * kGroupBytes;
        unsigned char* sx = nxt;
#pragma unroll 4
        for (int i = 0; i < M; ++i) {
          if (kBf16) cp_async_8(sx, xq);
          else cp_async_16_stream(sx, xq);
          xq += p.row_bytes;
          sx += stride;
        }
      }
      const int4* pw = s_pw + k * M;
      const ulonglong2 pivot = *reinterpret_cast<const ulonglong2*>(cur);
      ColAcc acc;
      LossAcc lacc;
      uint32_t off = 0;
      uint64_t goff = 0;
      auto do_row = [&](int i, uint4 rnd) {
        const int4 d = pw[i];
        const pair_t nw2 = ((pair_t)(uint32_t)d.w << 32) | (uint32_t)d.z;
        const ulonglong2 o = row_update_rnd<kObjective, kFastNoise>(
            p.alpha, ns, rnd, *reinterpret_cast<const ulonglong2*>(cur + off),
            *reinterpret_cast<const ulonglong2*>(cen + off), *reinterpret_cast<const ulonglong2*>(cur + (uint32_t)d.x), pivot,
            nw2, acc, lacc);
        if (kLast) {
          if (kBf16) *reinterpret_cast<unsigned long long*>(oq + goff) = narrow_bf16x4(o);
          else *reinterpret_cast<ulonglong2*>(oq + goff) = o;
          if (have_next) {  // this row's centre is not read again in this tile
            if (kBf16) cp_async_8(cen + off, cq_next + goff);
            else cp_async_16_stream(cen + off, cq_next + goff);
          }
          goff += p.row_bytes;
        } else {
          *reinterpret_cast<ulonglong2*>(nxt + off) = kBf16 ? widen_bf16x4(narrow_bf16x4(o)) : o;
        }
        off += stride;
      };
      // the Philox block of row i + 1 is drawn while row i goes through Box-Muller and Eq. 15-16:
      // the two are independent, so the integer multiplies of the one fill the latencies of the other
      uint4 rnd = noise_block<kObjective>(p.keys, round_lo, ctr3, q32, 0u);
#pragma unroll kFusedUnroll
      for (int i = 0; i + 1 < M; ++i) {
        const uint4 rnd_next = noise_block<kObjective>(p.keys, round_lo, ctr3, q32, (uint32_t)(i + 1));
        do_row(i, rnd);
        rnd = rnd_next;
      }
      do_row(M - 1, rnd);
      float4 s1, s2;
      unpack2(acc.s1a, s1.x, s1.y);
      unpack2(acc.s1b, s1.z, s1.w);
      unpack2(acc.s2a, s2.x, s2.y);
      unpack2(acc.s2b, s2.z, s2.w);
      float l0, l1, l2, l3;
      unpack2(lacc.la, l0, l1);
      unpack2(lacc.lb, l2, l3);
      const double cons = (double)((s2.x - s1.x * s1.x * p.inv_M) + (s2.y - s1.y * s1.y * p.inv_M) +
                                   (s2.z - s1.z * s1.z * p.inv_M) + (s2.w - s1.w * s1.w * p.inv_M));
      const double loss = (double)((l0 + l1) + (l2 + l3));
#pragma unroll
      for (int kk = 0; kk < kRounds; ++kk) {  // acc[k] with k known only at run time: predicated adds keep it in registers
        if (kk == k) {
          acc_cons[kk] += cons;
          acc_loss[kk] += loss;
        }
      }
    };
    for (int k = 0; k + 1 < p.n_rounds; ++k) run_round(k, std::false_type());
    run_round(p.n_rounds - 1, std::true_type());
    base = (base + (uint32_t)p.n_rounds) & 1u;
    fetched = have_next;
  }

  // telemetry: per round, CTA partials; the last CTA to finish sums them in index order
#pragma unroll
  for (int k = 0; k < kRounds; ++k)
    if (k < p.n_rounds) block_partials(p.partials + (size_t)k * 2 * gridDim.x, acc_cons[k], acc_loss[k], s_red);
  __shared__ bool s_last;
  if (tid == 0) {
    __threadfence();
    const unsigned int t = atomicAdd(p.ticket, 1u);
    s_last = (t == gridDim.x - 1);
  }
  __syncthreads();
  if (s_last) {
    __threadfence();
    for (int k = 0; k < p.n_rounds; ++k)
      sum_partials(p.partials + (size_t)k * 2 * gridDim.x, (double)p.inv_M, p.tel + 2 * ((p.slot0 + k) % p.ring), s_red);
    if (tid == 0) *p.ticket = 0u;
  }
}

// ---- several rounds over a tile that is resident across a thread-block cluster ----------------
// More workers than a thread's slab can hold (48 M bytes per column group: M = 64 would leave two
// warps per SM): the rows of a tile are split over the CTAs of a cluster.  CTA `rank` keeps rows
// [rank * rpc, rank * rpc + rpc) of T column groups in its shared memory exactly as
// fused_rounds_kernel keeps all of them, a thread still owns one column group, and the peer's
// value -- the same column group of a row that may live in another CTA of the cluster -- is read
// through distributed shared memory (mapa + ld.shared::cluster: plain loads, no multicast).  All
// CTAs of a cluster advance round by round: a cluster barrier (the hardware's
// barrier.cluster, not a spin) ends every round, which orders this round's remote reads of a slab
// before the next round's writes to it and keeps a CTA's shared memory alive while others read it.
// The consensus statistic needs the column sums over ALL rows: every CTA measures its rows against
// the common pivot (row 0 of the tile, read from rank 0), sum (x - a)^2 adds up CTA by CTA like
// the loss does, and the per-column sums of (x - a) go to a small double-buffered exchange area
// that rank 0 collects after the barrier.  Prefetch, direct store of the last round and the
// arithmetic are fused_rounds_kernel's, so replicas agree with every other launch shape bit for bit.
struct ClusterParams {
  FusedParams f;       // n_tiles: tiles of blockDim column groups
  int32_t rpc;         // rows per CTA = ceil(M / cluster size)
};

__device__ __forceinline__ uint32_t cluster_ctarank() {
  uint32_t r;
  asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
  return r;
}
__device__ __forceinline__ uint32_t cluster_nctarank() {
  uint32_t r;
  asm volatile("mov.u32 %0, %%cluster_nctarank;" : "=r"(r));
  return r;
}
// All threads of all CTAs of the cluster; release / acquire order shared-memory accesses across it.
__device__ __forceinline__ void cluster_barrier() {
  asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory");
  asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory");
}
// 16 bytes at the same shared-memory offset in CTA `rank` of the cluster.
__device__ __forceinline__ ulonglong2 ld_cluster_16(uint32_t smem_addr, uint32_t rank) {
  uint32_t remote;
  asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(remote) : "r"(smem_addr), "r"(rank));
  ulonglong2 v;
  asm volatile("ld.shared::cluster.v2.u64 {%0, %1}, [%2];" : "=l"(v.x), "=l"(v.y) : "r"(remote) : "memory");
  return v;
}

// Dynamic shared memory: (peer's local row offset, peer's CTA, -weight, -weight) int4[kClusterMaxRounds][rpc],
// then the slabs float4[3][rpc][blockDim], then the exchange area float4[2][blockDim], then 64 doubles.
template <int kObjective, bool kFastNoise>
__global__ void __launch_bounds__(256, 2) cluster_rounds_kernel(const ClusterParams cp) {
  const FusedParams& p = cp.f;
  extern __shared__ __align__(128) unsigned char smem_raw[];
  const int tid = threadIdx.x, T = blockDim.x, M = p.M, rpc = cp.rpc;
  const uint32_t rank = cluster_ctarank(), C = cluster_nctarank();
  const int r0 = min(M, (int)rank * rpc), rows = min(M, r0 + rpc) - r0;  // this CTA's rows [r0, r0 + rows)
  int4* s_pw = reinterpret_cast<int4*>(smem_raw);
  const uint32_t head = ((uint32_t)(kClusterMaxRounds * rpc * 16) + 127u) & ~127u;
  const uint32_t stride = (uint32_t)T * 16u;
  const uint32_t plane = (uint32_t)rpc * stride;
  unsigned char* slab = smem_raw + head + (uint32_t)tid * 16u;
  float4* s_xchg = reinterpret_cast<float4*>(smem_raw + head + 3u * plane);  // [2][T] column sums of (x - pivot) over this CTA's rows
  double* s_red = reinterpret_cast<double*>(smem_raw + head + 3u * plane + 2u * stride);
  const uint32_t slab_addr = (uint32_t)__cvta_generic_to_shared(slab);
  const uint32_t xchg_addr = (uint32_t)__cvta_generic_to_shared(s_xchg + tid);

  for (int k = 0; k < p.n_rounds; ++k) {
    const int32_t* peers = p.trace + ((p.slot0 + k) % p.ring) * M;
    for (int j = tid; j < rows; j += T) {
      const int i = r0 + j;
      const int32_t m = __ldg(peers + i);
      const int nw = __float_as_int((m == i) ? -0.0f : -__ldg(p.wtab + (size_t)i * M + m));
      const int pm = m / rpc;
      s_pw[k * rpc + j] = make_int4((int)((uint32_t)(m - pm * rpc) * stride), pm, nw, nw);
    }
  }
  __syncthreads();

  double acc_cons[kClusterMaxRounds], acc_loss[kClusterMaxRounds];
#pragma unroll
  for (int k = 0; k < kClusterMaxRounds; ++k) acc_cons[k] = acc_loss[k] = 0.0;

  const int64_t n_clusters = gridDim.x / C, cluster_id = blockIdx.x / C;
  const uint64_t row0_bytes = (uint64_t)(uint32_t)r0 * p.row_bytes;
  uint32_t base = 0;
  bool fetched = false;
  uint32_t epoch = 0;  // rounds done by this cluster: parity selects the exchange buffer
  // every CTA of a cluster runs the same tiles and rounds, so all of them meet at every barrier
  for (int64_t tile = cluster_id; tile < p.n_tiles; tile += n_clusters) {
    const int64_t q = tile * T + tid;
    const bool live = q < p.nq;
    const NoiseLanes ns = noise_lanes(p.sigma, live_lanes((p.tail != 0) && (q == p.nq - 1), p.tail, 0));
    const uint32_t q32 = (uint32_t)q + p.q_offset;
    const int64_t q_next = q + n_clusters * T;
    const bool tile_has_next = NETMAX_FUSED_PREFETCH != 0 && tile + n_clusters < p.n_tiles;  // the same in every CTA of the cluster
    const bool have_next = tile_has_next && q_next < p.nq;
    if (!fetched && live) {
      const char* xq = reinterpret_cast<const char*>(p.x_cur) + row0_bytes + (uint64_t)q * 16u;
      const char* cq = reinterpret_cast<const char*>(p.c) + row0_bytes + (uint64_t)q * 16u;
      unsigned char* sx = slab + base * plane;
      unsigned char* sc = slab + 2u * plane;
#pragma unroll 4
      for (int j = 0; j < rows; ++j) {
        *reinterpret_cast<ulonglong2*>(sx) = __ldg(reinterpret_cast<const ulonglong2*>(xq));
        *reinterpret_cast<ulonglong2*>(sc) = __ldg(reinterpret_cast<const ulonglong2*>(cq));
        xq += p.row_bytes;
        cq += p.row_bytes;
        sx += stride;
        sc += stride;
      }
    }
    // every CTA's rows of the tile are in place before anyone pulls from them (a fetched tile was
    // published by the barrier that ended its predecessor's last round)
    if (!fetched) cluster_barrier();
    unsigned char* const cen = slab + 2u * plane;
    char* const oq = reinterpret_cast<char*>(p.x_nxt) + row0_bytes + (uint64_t)q * 16u;
    const char* const cq_next = reinterpret_cast<const char*>(p.c) + row0_bytes + (uint64_t)q_next * 16u;

    auto run_round = [&](int k, auto last_tag) {
      constexpr bool kLast = decltype(last_tag)::value;
      const uint64_t round = p.first_round + (uint64_t)k;
      const uint32_t round_lo = (uint32_t)round, ctr3 = philox_ctr3(kTagNoise, round);
      const uint32_t cur_off = ((base + (uint32_t)k) & 1u) * plane;
      const unsigned char* cur = slab + cur_off;
      unsigned char* nxt = slab + ((base + (uint32_t)k + 1u) & 1u) * plane;
      if (kLast && have_next) {
        const char* xq = reinterpret_cast<const char*>(p.x_cur) + row0_bytes + (uint64_t)q_next * 16u;
        unsigned char* sx = nxt;
#pragma unroll 4
        for (int j = 0; j < rows; ++j) {
          cp_async_16_stream(sx, xq);
          xq += p.row_bytes;
          sx += stride;
        }
      }
      ColAcc acc;
      LossAcc lacc;
      if (live) {
        const int4* pw = s_pw + k * rpc;
        const ulonglong2 pivot = ld_cluster_16(slab_addr + cur_off, 0u);  // row 0 of the tile lives in CTA 0
        uint32_t off = 0;
        uint64_t goff = 0;
        auto pull = [&](int j) {  // the peer's value for local row j, from whichever CTA holds that row
          const int4 d = pw[j];
          return ld_cluster_16(slab_addr + cur_off + (uint32_t)d.x, (uint32_t)d.y);
        };
        auto do_row = [&](int j, uint4 rnd, ulonglong2 xm) {
          const int4 d = pw[j];
          const pair_t nw2 = ((pair_t)(uint32_t)d.w << 32) | (uint32_t)d.z;
          const ulonglong2 o = row_update_rnd<kObjective, kFastNoise>(p.alpha, ns, rnd, *reinterpret_cast<const ulonglong2*>(cur + off),
                                                                      *reinterpret_cast<const ulonglong2*>(cen + off), xm, pivot, nw2, acc,
                                                                      lacc);
          if (kLast) {
            *reinterpret_cast<ulonglong2*>(oq + goff) = o;
            if (have_next) cp_async_16_stream(cen + off, cq_next + goff);
            goff += p.row_bytes;
          } else {
            *reinterpret_cast<ulonglong2*>(nxt + off) = o;
          }
          off += stride;
        };
        if (rows > 0) {
          // one row ahead: the next row's Philox block (integer work that fills this row's latencies) and
          // its pull, whose trip through the cluster's shared-memory network takes several hundred cycles
          // (two rows ahead measured slower: 1.43 against 1.39 ms per round of 64 x 11.2 M elements)
          uint4 rnd = noise_block<kObjective>(p.keys, round_lo, ctr3, q32, (uint32_t)r0);
          ulonglong2 xm = pull(0);
#pragma unroll kFusedUnroll
          for (int j = 0; j + 1 < rows; ++j) {
            const ulonglong2 xm_next = pull(j + 1);
            const uint4 rnd_next = noise_block<kObjective>(p.keys, round_lo, ctr3, q32, (uint32_t)(r0 + j + 1));
            do_row(j, rnd, xm);
            rnd = rnd_next;
            xm = xm_next;
          }
          do_row(rows - 1, rnd, xm);
        }
      }
      float4 s1, s2;
      unpack2(acc.s1a, s1.x, s1.y);
      unpack2(acc.s1b, s1.z, s1.w);
      unpack2(acc.s2a, s2.x, s2.y);
      unpack2(acc.s2b, s2.z, s2.w);
      float l0, l1, l2, l3;
      unpack2(lacc.la, l0, l1);
      unpack2(lacc.lb, l2, l3);
      const uint32_t buf = epoch & 1u;
      s_xchg[buf * T + tid] = s1;
      if (kLast) cp_async_wait_all();  // the next tile's rows have landed: the barrier below publishes them too
      cluster_barrier();  // the round is complete everywhere; the column sums of all CTAs are published
      ++epoch;
      double cons = (double)((s2.x + s2.y) + (s2.z + s2.w));  // this CTA's share of sum (x - a)^2
      if (rank == 0) {
        // sum_i (x_i - xbar)^2 = sum_i (x_i - a)^2 - (sum_i (x_i - a))^2 / M per column: rank 0 subtracts the second term
        float4 tot = s1;
        for (uint32_t r = 1; r < C; ++r) {
          const ulonglong2 v = ld_cluster_16(xchg_addr + buf * stride, r);
          float a, b, c2, d2;
          unpack2(v.x, a, b);
          unpack2(v.y, c2, d2);
          tot.x += a;
          tot.y += b;
          tot.z += c2;
          tot.w += d2;
        }
        cons -= (double)((tot.x * tot.x + tot.y * tot.y + tot.z * tot.z + tot.w * tot.w) * p.inv_M);
      }
      const double loss = (double)((l0 + l1) + (l2 + l3));
#pragma unroll
      for (int kk = 0; kk < kClusterMaxRounds; ++kk) {
        if (kk == k) {
          acc_cons[kk] += cons;
          acc_loss[kk] += loss;
        }
      }
    };
    for (int k = 0; k + 1 < p.n_rounds; ++k) run_round(k, std::false_type());
    run_round(p.n_rounds - 1, std::true_type());
    base = (base + (uint32_t)p.n_rounds) & 1u;
    fetched = tile_has_next;
  }
  cluster_barrier();  // no CTA leaves while another may still read its exchange area

#pragma unroll
  for (int k = 0; k < kClusterMaxRounds; ++k)
    if (k < p.n_rounds) block_partials(p.partials + (size_t)k * 2 * gridDim.x, acc_cons[k], acc_loss[k], s_red);
  __shared__ bool s_last;
  if (tid == 0) {
    __threadfence();
    const unsigned int t = atomicAdd(p.ticket, 1u);
    s_last = (t == gridDim.x - 1);
  }
  __syncthreads();
  if (s_last) {
    __threadfence();
    for (int k = 0; k < p.n_rounds; ++k)
      sum_partials(p.partials + (size_t)k * 2 * gridDim.x, (double)p.inv_M, p.tel + 2 * ((p.slot0 + k) % p.ring), s_red);
    if (tid == 0) *p.ticket = 0u;
  }
}

// ---- all rounds of a call over resident columns (short vectors) -------------------------------
// The same independence of columns serves the opposite shape: when the whole problem is a few
// megabytes, a round takes microseconds and what costs time is every launch and every grid-wide
// exchange.  Here a CTA keeps ALL M rows of G column groups (four elements each) in shared
// memory, fp32, double-buffered by round, together with their centres, and runs every round of
// the call on them; CTAs never talk to each other.  Two thread mappings:
//   G == blockDim  a thread owns a column group and walks all M rows (small M): no barrier is
//                  needed for the data, only the per-round telemetry reduction synchronises
//                  (and not even that in a CTA of a single warp);
//   G <= 32        thread (g, r) owns the rows r, r + blockDim / G, ... of group g (large M):
//                  a peer's row belongs to another thread, so rounds are separated by ONE barrier
//                  (a warp-level one in a single-warp CTA); the column sums of the round are
//                  added over the lanes of each warp before it and over the warps after it, by
//                  one warp that changes from round to round while the others carry on.
// Per round every CTA writes its two telemetry sums to partials[round][tile]; a second small
// kernel adds the tiles of each round in index order.  Arithmetic per element is row_update's,
// so replicas are bit-identical to the other launch shapes.
struct ResidentParams {
  const char* x_cur;      // replicas at the start of the first round, row stride row_bytes
  char* x_nxt;            // replicas after the last round
  const char* c;
  const int32_t* trace;   // peer-trace ring [ring][M]
  const float* wring;     // pull weight of every draw, same ring
  double* partials;       // [n_rounds][n_tiles][2]
  int64_t slot0, ring;
  uint64_t first_round;
  int32_t n_rounds;
  int64_t nq, n_tiles;    // column groups of four elements per row; tiles of G of them
  uint32_t row_bytes;
  int32_t M, tail;        // tail = d % 4
  int32_t G, log2G;       // column groups per tile (a power of two)
  int32_t draw_chunk;     // > 0: the (peer, weight) pairs of this many rounds at a time are staged in shared
                          // memory; 0 (large M): every thread loads the draws of its own rows, a round ahead
  float alpha, sigma, inv_M;
  uint32_t q_offset;
  PhiloxKeys keys;
};

// Dynamic shared memory: slabs float4[3][M][G]; then (G < blockDim) two reduction scratch
// buffers float[warps][G][9] (padded to 16 bytes); then 2 x 64 floats; then int2[draw_chunk][M].
constexpr int kDrawRegs = 8;  // large M: draws of a thread's first rows that are fetched a round ahead
#ifndef NETMAX_RESIDENT_UNROLL
#define NETMAX_RESIDENT_UNROLL 2
#endif
constexpr int kResidentUnroll = NETMAX_RESIDENT_UNROLL;  // rows of a round in flight per thread
__host__ __device__ inline uint32_t resident_scratch_floats(int threads, int G) {
  return G < threads ? (uint32_t)(((threads >> 5) * G * 9 + 3) & ~3) : 0u;
}
template <int kObjective, bool kFastNoise, bool kBf16>
__global__ void __launch_bounds__(512) resident_rounds_kernel(const ResidentParams p) {
  constexpr uint32_t kGroupBytes = kBf16 ? 8u : 16u;
  extern __shared__ __align__(128) unsigned char smem_raw[];
  const int tid = threadIdx.x, T = blockDim.x, M = p.M, G = p.G;
  const int g = tid & (G - 1), r = tid >> p.log2G, RL = T >> p.log2G;
  const int lane = tid & 31, warp = tid >> 5, nwarps = T >> 5;
  const uint32_t stride = (uint32_t)G * 16u;    // bytes between consecutive rows of a slab
  const uint32_t plane = (uint32_t)M * stride;
  unsigned char* slab = smem_raw + (uint32_t)g * 16u;
  float* s_scratch = reinterpret_cast<float*>(smem_raw + 3u * plane);
  const uint32_t scratch_floats = resident_scratch_floats(T, G);
  float* s_red = s_scratch + 2 * scratch_floats;  // 2 x 64 floats
  int2* s_pw = reinterpret_cast<int2*>(s_red + 128);

  for (int64_t tile = blockIdx.x; tile < p.n_tiles; tile += gridDim.x) {
    const int64_t q = tile * G + g;
    const bool live = q < p.nq;
    const int live_lo = live_lanes((p.tail != 0) && (q == p.nq - 1), p.tail, 0);
    const uint32_t q32 = (uint32_t)q + p.q_offset;
    __syncthreads();  // the previous tile is stored
    for (int i = r; i < M; i += RL) {
      ulonglong2 xv = make_ulonglong2(0ull, 0ull), cv = xv;
      if (live) {
        const char* xq = p.x_cur + (uint64_t)(uint32_t)i * p.row_bytes + (uint64_t)q * kGroupBytes;
        const char* cq = p.c + (uint64_t)(uint32_t)i * p.row_bytes + (uint64_t)q * kGroupBytes;
        if (kBf16) {
          xv = widen_bf16x4(__ldg(reinterpret_cast<const unsigned long long*>(xq)));
          cv = widen_bf16x4(__ldg(reinterpret_cast<const unsigned long long*>(cq)));
        } else {
          xv = __ldg(reinterpret_cast<const ulonglong2*>(xq));
          cv = __ldg(reinterpret_cast<const ulonglong2*>(cq));
        }
      }
      *reinterpret_cast<ulonglong2*>(slab + (uint32_t)i * stride) = xv;
      *reinterpret_cast<ulonglong2*>(slab + 2u * plane + (uint32_t)i * stride) = cv;
    }
    int64_t slot = p.slot0 % p.ring;  // ring slot of round k, stepped along with k
    const int KC = p.draw_chunk;      // rounds whose draws are staged in shared memory at a time (0: none)
    int2 dreg[kDrawRegs];             // KC == 0: the draws of this thread's first rows, loaded a round ahead
    if (KC == 0 && live) {
#pragma unroll
      for (int j = 0; j < kDrawRegs; ++j) {
        const int i = r + j * RL;
        if (i < M) dreg[j] = make_int2(__ldg(p.trace + slot * M + i), __float_as_int(__ldg(p.wring + slot * M + i)));
      }
    }
    __syncthreads();

    for (int k = 0; k < p.n_rounds; ++k) {
      const uint64_t round = p.first_round + (uint64_t)k;
      const uint32_t round_lo = (uint32_t)round, ctr3 = philox_ctr3(kTagNoise, round);
      const int kc = KC > 0 ? k % KC : 0;
      if (KC > 0 && kc == 0) {
        // stage the draws of the next KC rounds (the previous round's barrier has retired their predecessors)
        const int n = min(KC, p.n_rounds - k) * M;
#pragma unroll 4
        for (int idx = tid; idx < n; idx += T) {
          const int ahead = idx / M;  // rounds ahead of round k
          int64_t s2 = slot + ahead;
          if (s2 >= p.ring) s2 -= p.ring;  // (a chunk is never longer than the ring)
          const int64_t src = s2 * M + (idx - ahead * M);
          s_pw[idx] = make_int2(__ldg(p.trace + src), __float_as_int(__ldg(p.wring + src)));
        }
        __syncthreads();
      }
      const int64_t at = slot * M;
      slot = slot + 1 == p.ring ? 0 : slot + 1;
      const unsigned char* cur = slab + (uint32_t)(k & 1) * plane;
      unsigned char* nxt = slab + (uint32_t)((k & 1) ^ 1) * plane;
      const unsigned char* cen = slab + 2u * plane;
      ColAcc acc;
      LossAcc lacc;
      if (live) {
        const ulonglong2 pivot = *reinterpret_cast<const ulonglong2*>(cur);
        auto do_row = [&](int i, int2 d) {
          const uint32_t off = (uint32_t)i * stride;
          ulonglong2 o = row_update<kObjective, kFastNoise>(
              p.alpha, p.sigma, p.keys, round_lo, ctr3, q32, (uint32_t)i, *reinterpret_cast<const ulonglong2*>(cur + off),
              *reinterpret_cast<const ulonglong2*>(cen + off), *reinterpret_cast<const ulonglong2*>(cur + (uint32_t)d.x * stride),
              pivot, __int_as_float(d.y), live_lo, acc, lacc);
          if (kBf16) o = widen_bf16x4(narrow_bf16x4(o));
          *reinterpret_cast<ulonglong2*>(nxt + off) = o;
        };
        if (KC > 0) {
          const int2* pw = s_pw + kc * M;
#pragma unroll kResidentUnroll
          for (int i = r; i < M; i += RL) do_row(i, pw[i]);
        } else {
#pragma unroll
          for (int j = 0; j < kDrawRegs; ++j) {
            const int i = r + j * RL;
            if (i < M) do_row(i, dreg[j]);
          }
          for (int i = r + kDrawRegs * RL; i < M; i += RL)
            do_row(i, make_int2(__ldg(p.trace + at + i), __float_as_int(__ldg(p.wring + at + i))));
          if (k + 1 < p.n_rounds) {  // next round's draws: in flight during the reduction below
#pragma unroll
            for (int j = 0; j < kDrawRegs; ++j) {
              const int i = r + j * RL;
              if (i < M) dreg[j] = make_int2(__ldg(p.trace + slot * M + i), __float_as_int(__ldg(p.wring + slot * M + i)));
            }
          }
        }
      }
      // ---- telemetry of the round: column sums over the row lanes, then over the tile
      float v[9];
      unpack2(acc.s1a, v[0], v[1]);
      unpack2(acc.s1b, v[2], v[3]);
      unpack2(acc.s2a, v[4], v[5]);
      unpack2(acc.s2b, v[6], v[7]);
      {
        float l0, l1, l2, l3;
        unpack2(lacc.la, l0, l1);
        unpack2(lacc.lb, l2, l3);
        v[8] = (l0 + l1) + (l2 + l3);
      }
      double* out = p.partials + ((size_t)k * p.n_tiles + tile) * 2;
      if (RL > 1) {
        // the rows of a column group are spread over row lanes: first over those of this warp ...
        for (int off = 16; off >= G; off >>= 1) {
#pragma unroll
          for (int a = 0; a < 9; ++a) v[a] += __shfl_xor_sync(0xffffffffu, v[a], off);
        }
        if (nwarps > 1) {
          float* scratch = s_scratch + (k & 1) * scratch_floats;
          if (lane < G) {
#pragma unroll
            for (int a = 0; a < 9; ++a) scratch[(warp * G + lane) * 9 + a] = v[a];
          }
          __syncthreads();  // the round's one barrier: every row is written before the next round reads it, every warp's sums are out
          // ... then over the warps, by ONE warp (a different one every round) while the others go on with
          // the next round: its buffer is not written again before the barrier after next.  (With a second
          // barrier and one thread adding the warps' sums, a round of 4096 x 4 elements spent 2,900 of its
          // 9,800 cycles here.)
          if (warp == k % nwarps) {
#pragma unroll
            for (int a = 0; a < 9; ++a) v[a] = 0.f;
            for (int e = lane; e < nwarps * G; e += 32) {  // entry e = (warp, group e % G); G divides 32
#pragma unroll
              for (int a = 0; a < 9; ++a) v[a] += scratch[e * 9 + a];
            }
            for (int off = 16; off >= G; off >>= 1) {
#pragma unroll
              for (int a = 0; a < 9; ++a) v[a] += __shfl_xor_sync(0xffffffffu, v[a], off);
            }
          }
        } else {
          __syncwarp();  // a single warp: its lanes are all the threads that exchange rows
        }
        if (nwarps == 1 || warp == k % nwarps) {  // lanes 0 .. G-1 hold the sums of their groups
          float cons = 0.f, loss = 0.f;
          if (lane < G) {
            cons = (v[4] - v[0] * v[0] * p.inv_M) + (v[5] - v[1] * v[1] * p.inv_M) + (v[6] - v[2] * v[2] * p.inv_M) +
                   (v[7] - v[3] * v[3] * p.inv_M);
            loss = v[8];
          }
          for (int off = 16; off > 0; off >>= 1) {
            cons += __shfl_down_sync(0xffffffffu, cons, off);
            loss += __shfl_down_sync(0xffffffffu, loss, off);
          }
          if (lane == 0) {
            out[0] = (double)cons;
            out[1] = 0.5 * (double)loss;
          }
        }
      } else {
        // a thread holds the complete sums of its column group; no thread reads another's rows
        float cons = (v[4] - v[0] * v[0] * p.inv_M) + (v[5] - v[1] * v[1] * p.inv_M) + (v[6] - v[2] * v[2] * p.inv_M) +
                     (v[7] - v[3] * v[3] * p.inv_M);
        float loss = v[8];
        for (int off = 16; off > 0; off >>= 1) {
          cons += __shfl_down_sync(0xffffffffu, cons, off);
          loss += __shfl_down_sync(0xffffffffu, loss, off);
        }
        if (nwarps == 1) {
          if (lane == 0) {
            out[0] = (double)cons;
            out[1] = 0.5 * (double)loss;
          }
          __syncwarp();  // (the staged draws are overwritten by whichever lane gets there first)
        } else {
          float* red = s_red + (k & 1) * 64;
          if (lane == 0) {
            red[warp] = cons;
            red[32 + warp] = loss;
          }
          __syncthreads();
          if (tid == 0) {
            double a = 0.0, b = 0.0;
            for (int w = 0; w < nwarps; ++w) {
              a += (double)red[w];
              b += (double)red[32 + w];
            }
            out[0] = a;
            out[1] = 0.5 * b;
          }
        }
      }
    }

    if (live) {
      const unsigned char* fin = slab + (uint32_t)(p.n_rounds & 1) * plane;
      for (int i = r; i < M; i += RL) {
        char* oq = p.x_nxt + (uint64_t)(uint32_t)i * p.row_bytes + (uint64_t)q * kGroupBytes;
        const ulonglong2 o = *reinterpret_cast<const ulonglong2*>(fin + (uint32_t)i * stride);
        if (kBf16) *reinterpret_cast<unsigned long long*>(oq) = narrow_bf16x4(o);
        else *reinterpret_cast<ulonglong2*>(oq) = o;
      }
    }
  }
}

// tel[slot of round k] = (sum over tiles of partials[k][tile]) / M, one warp per round, tiles in a fixed order.
__global__ void __launch_bounds__(256) sum_tile_partials_kernel(const double* partials, int64_t n_tiles, int32_t n_rounds,
                                                                double inv_M, double* tel, int64_t slot0, int64_t ring) {
  const int lane = threadIdx.x & 31;
  const int k = (int)((blockIdx.x * (int64_t)blockDim.x + threadIdx.x) >> 5);
  if (k >= n_rounds) return;
  double a = 0.0, b = 0.0;
  for (int64_t t = lane; t < n_tiles; t += 32) {
    a += partials[((size_t)k * n_tiles + t) * 2];
    b += partials[((size_t)k * n_tiles + t) * 2 + 1];
  }
  for (int off = 16; off > 0; off >>= 1) {
    a += __shfl_down_sync(0xffffffffu, a, off);
    b += __shfl_down_sync(0xffffffffu, b, off);
  }
  if (lane == 0) {
    double* out = tel + 2 * ((slot0 + k) % ring);
    out[0] = a * inv_M;
    out[1] = b * inv_M;
  }
}

// tel[slot of round k] = sum over chunks of chunk_tel[chunk][slot], chunks in order (a pipelined host
// round trip runs the rounds chunk of columns by chunk; both statistics are sums over columns).
__global__ void __launch_bounds__(256) sum_chunk_telemetry_kernel(const double* chunk_tel, int32_t n_chunks, int64_t ring,
                                                                  int64_t slot0, int64_t n_rounds, double* tel) {
  const int64_t k = blockIdx.x * (int64_t)blockDim.x + threadIdx.x;
  if (k >= n_rounds) return;
  const int64_t slot = (slot0 + k) % ring;
  double a = 0.0, b = 0.0;
  for (int c = 0; c < n_chunks; ++c) {
    a += chunk_tel[((size_t)c * ring + slot) * 2];
    b += chunk_tel[((size_t)c * ring + slot) * 2 + 1];
  }
  tel[2 * slot] = a;
  tel[2 * slot + 1] = b;
}

// ------------------------------------------------------------------------- asynchronous steps
// The paper's own process (Eq. 17): at a global step ONE worker i applies Eq. 15-16 to its
// replica, in place, with the peer's current replica; every other replica is unchanged.  A
// launch carries up to kMaxStepEvents consecutive global steps that touch disjoint replicas
// (no step writes a row another step of the launch reads or writes), so their order inside
// the launch does not matter.  16 bytes of HBM traffic per element: nothing is shared.
constexpr int kMaxStepEvents = 32;

struct StepEvent {
  int32_t worker, peer;
  uint32_t iter_lo, ctr3;  // the worker's local iteration, as Philox counter words of the noise stream
  float w;                 // pull weight w_im (0 on a self-draw)
};

struct StepParams {
  float4* x;        // [M][ldq] replicas (16-byte column groups), updated in place
  const float4* c;  // [M][ldq]
  int64_t nq;
  uint32_t row_bytes;
  int32_t tail;     // d % (4 kHalves)
  float alpha, sigma;
  uint32_t q_offset;
  int32_t n_events;
  StepEvent ev[kMaxStepEvents];
  PhiloxKeys keys;
};

template <int kObjective, bool kFastNoise, int kHalves>
__global__ void __launch_bounds__(256) step_kernel(const StepParams p) {
  const StepEvent& e = p.ev[blockIdx.y];
  const uint64_t row_i = (uint64_t)(uint32_t)e.worker * p.row_bytes;
  const uint64_t row_m = (uint64_t)(uint32_t)e.peer * p.row_bytes;
  char* xb = reinterpret_cast<char*>(p.x);
  const char* cb = reinterpret_cast<const char*>(p.c);
  for (int64_t q = blockIdx.x * (int64_t)blockDim.x + threadIdx.x; q < p.nq; q += (int64_t)gridDim.x * blockDim.x) {
    const uint64_t off = (uint64_t)q * 16;
    const ulonglong2 xv = *reinterpret_cast<const ulonglong2*>(xb + row_i + off);
    const ulonglong2 xm = *reinterpret_cast<const ulonglong2*>(xb + row_m + off);
    ulonglong2 cv = make_ulonglong2(0ull, 0ull);
    if (kObjective == 1) cv = __ldg(reinterpret_cast<const ulonglong2*>(cb + row_i + off));
    const bool ragged = (p.tail != 0) && (q == p.nq - 1);
    ulonglong2 o;
#pragma unroll
    for (int h = 0; h < kHalves; ++h) {
      pair_t ta, tb;
      const ulonglong2 oh = update_core<kObjective, kFastNoise>(
          p.alpha, p.sigma, p.keys, e.iter_lo, e.ctr3, (uint32_t)q * kHalves + h + p.q_offset, (uint32_t)e.worker,
          group_half<kHalves>(xv, h), group_half<kHalves>(cv, h), group_half<kHalves>(xm, h), e.w,
          live_lanes(ragged, p.tail, h), ta, tb);
      if (kHalves == 1) o = oh;
      else if (h == 0) o.x = narrow_bf16x4(oh);
      else o.y = narrow_bf16x4(oh);
    }
    *reinterpret_cast<ulonglong2*>(xb + row_i + off) = o;
  }
}

// ------------------------------------------------------------------------- init / IO
struct InitParams {
  float4* dst;  // [M][ldq] column groups
  int64_t ldq, nq;
  int32_t M, tail;  // tail = d % (4 kHalves)
  float stddev;
  uint32_t tag;
  uint32_t q_offset;
  PhiloxKeys keys;
};

template <int kHalves>
__global__ void __launch_bounds__(256) init_normal_kernel(const InitParams p) {
  const int64_t total = (int64_t)p.M * p.nq;
  for (int64_t idx = blockIdx.x * (int64_t)blockDim.x + threadIdx.x; idx < total;
       idx += (int64_t)gridDim.x * blockDim.x) {
    const int64_t i = idx / p.nq, q = idx - i * p.nq;
    const bool ragged = p.tail != 0 && q == p.nq - 1;
    ulonglong2 o;
#pragma unroll
    for (int h = 0; h < kHalves; ++h) {
      float4 z = normals4<false>(philox4x32_10((uint32_t)q * kHalves + h + p.q_offset, (uint32_t)i, 0u, p.tag, p.keys));
      z.x *= p.stddev; z.y *= p.stddev; z.z *= p.stddev; z.w *= p.stddev;
      const int live = live_lanes(ragged, p.tail, h);
      if (live < 1) z.x = 0.f;
      if (live < 2) z.y = 0.f;
      if (live < 3) z.z = 0.f;
      if (live < 4) z.w = 0.f;
      const ulonglong2 v = make_ulonglong2(pack2(z.x, z.y), pack2(z.z, z.w));
      if (kHalves == 1) o = v;
      else if (h == 0) o.x = narrow_bf16x4(v);
      else o.y = narrow_bf16x4(v);
    }
    *reinterpret_cast<ulonglong2*>(p.dst + (size_t)i * p.ldq + q) = o;
  }
}

// One stored element as fp32 (bfloat16 widens exactly).
__device__ __forceinline__ float load_element(const void* plane, size_t index, bool bf16) {
  if (bf16) return __uint_as_float((uint32_t)reinterpret_cast<const unsigned short*>(plane)[index] << 16);
  return reinterpret_cast<const float*>(plane)[index];
}

__global__ void __launch_bounds__(256) gather_columns_kernel(const void* x, bool bf16, int64_t ld, int32_t M,
                                                             const int64_t* cols, int64_t n_cols, float* out) {
  const int64_t total = (int64_t)M * n_cols;
  for (int64_t idx = blockIdx.x * (int64_t)blockDim.x + threadIdx.x; idx < total;
       idx += (int64_t)gridDim.x * blockDim.x) {
    const int64_t i = idx / n_cols, k = idx - i * n_cols;
    out[idx] = load_element(x, (size_t)i * ld + cols[k], bf16);
  }
}

// bfloat16 state <-> dense fp32 rows (host transfers of a bfloat16 context are staged in fp32
// on the device): `rows` rows of d elements; the bfloat16 side has row stride ld.
__global__ void __launch_bounds__(256) narrow_rows_kernel(const float* src, unsigned short* dst, int64_t rows, int64_t d,
                                                          int64_t ld) {
  const int64_t total = rows * d;
  for (int64_t idx = blockIdx.x * (int64_t)blockDim.x + threadIdx.x; idx < total;
       idx += (int64_t)gridDim.x * blockDim.x) {
    const int64_t i = idx / d, e = idx - i * d;
    unsigned short v;
    asm("cvt.rn.bf16.f32 %0, %1;" : "=h"(v) : "f"(src[idx]));
    dst[(size_t)i * ld + e] = v;
  }
}

__global__ void __launch_bounds__(256) widen_rows_kernel(const unsigned short* src, float* dst, int64_t rows, int64_t d,
                                                         int64_t ld) {
  const int64_t total = rows * d;
  for (int64_t idx = blockIdx.x * (int64_t)blockDim.x + threadIdx.x; idx < total;
       idx += (int64_t)gridDim.x * blockDim.x) {
    const int64_t i = idx / d, e = idx - i * d;
    dst[idx] = __uint_as_float((uint32_t)src[(size_t)i * ld + e] << 16);
  }
}

}  // namespace netmax
