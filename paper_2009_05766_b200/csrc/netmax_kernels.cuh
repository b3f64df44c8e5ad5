// CUDA kernels of the NetMax round simulator (sm_100a).
//
//   sample_peers_kernel   Algorithm 2, peer selection: one Philox draw per (round, worker)
//                         searched in that worker's row of 32-bit cumulative thresholds.
//   round_kernel          Eq. 15 (local SGD step with inline Gaussian gradient noise) fused
//                         with Eq. 16 (pull from the round-start snapshot of the peer) and
//                         with the round's telemetry; reads one buffer, writes the other.
//   init_normal_kernel    x(0) and c from the seed.
//   gather_columns_kernel sampled read-back.
#pragma once
#include <cstdint>
#include <cuda_runtime.h>

#include "netmax_rng.cuh"

namespace netmax {

// ------------------------------------------------------------------------- sampler
struct SampleParams {
  const uint32_t* thresholds;  // [M][M] non-decreasing per row
  const int32_t* last_nz;      // [M] last index with p > 0
  int32_t* out;                // slot s of round r is out + ((slot0 + r) % ring) * M
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
    p.out[((p.slot0 + r) % p.ring) * p.M + i] = m;
  }
}

// ------------------------------------------------------------------------- round
struct RoundParams {
  const float4* x_cur;   // [M][ldq] round-start replicas
  float4* x_nxt;         // [M][ldq] next replicas
  const float4* c;       // [M][ldq] centres
  const int32_t* peers;  // [M] this round's draws
  const float* wtab;     // [M][M] pull weights w_im (fp32)
  double* partials;      // [gridDim.x][2] per-CTA telemetry sums
  unsigned int* ticket;  // last-CTA-done counter (0 between launches)
  double* tel_out;       // [2] this round's (consensus, loss)
  int64_t ldq;           // row stride, in float4
  int64_t nq;            // column groups per row = ceil(d / 4)
  int64_t n_tiles;       // ceil(nq / cg)
  int32_t M;
  int32_t tail;          // d % 4: live lanes of the last column group (0 = all four)
  int32_t cg;            // column groups per tile   (cg * rl == blockDim.x, both powers of two)
  int32_t rl;            // row lanes per tile
  float alpha, sigma;
  float inv_M;
  uint32_t round_lo, ctr3;
  uint32_t q_offset;     // column-group index of the context's first element in the global vector
  PhiloxKeys keys;
};

__device__ __forceinline__ float4 ld_stream(const float4* p) { return __ldcs(p); }
__device__ __forceinline__ void st_stream(float4* p, float4 v) { __stcs(p, v); }

template <int kObjective, bool kFastNoise>
__device__ __forceinline__ float4 update_group(const RoundParams& p, uint32_t q, uint32_t worker, float4 x, float4 c,
                                               float4 xm, float w) {
  float4 h = x;
  if (kObjective == 1) {
    const float4 z = normals4<kFastNoise>(philox4x32_10(q, worker, p.round_lo, p.ctr3, p.keys));
    // g = (x - c) + sigma z ;  h = x - alpha g                                    (Eq. 15)
    h.x = fmaf(-p.alpha, fmaf(p.sigma, z.x, x.x - c.x), x.x);
    h.y = fmaf(-p.alpha, fmaf(p.sigma, z.y, x.y - c.y), x.y);
    h.z = fmaf(-p.alpha, fmaf(p.sigma, z.z, x.z - c.z), x.z);
    h.w = fmaf(-p.alpha, fmaf(p.sigma, z.w, x.w - c.w), x.w);
  }
  // x' = h - w (h - x_m)  with w = alpha rho gamma_im; w = 0 on a self-draw          (Eq. 16)
  float4 o;
  o.x = fmaf(-w, h.x - xm.x, h.x);
  o.y = fmaf(-w, h.y - xm.y, h.y);
  o.z = fmaf(-w, h.z - xm.z, h.z);
  o.w = fmaf(-w, h.w - xm.w, h.w);
  return o;
}

// One tile = all M rows x cg column groups.  Thread (cgi, rli) owns column group cgi of the
// tile and the rows rli, rli + rl, ...; tiles are taken round-robin by the resident CTAs.
// Dynamic shared memory: int32 peer[M], float w[M], then (rl > 1) 2 * blockDim float4 of
// column-sum scratch, then 2 * 32 doubles for the block reduction.
// Tuning constants of round_kernel: rows whose loads are in flight together per thread, and
// the CTAs per SM the register allocation must leave room for.
#ifndef NETMAX_ROUND_UNROLL
#define NETMAX_ROUND_UNROLL 1
#endif
#ifndef NETMAX_ROUND_MIN_CTAS
#define NETMAX_ROUND_MIN_CTAS 4
#endif

template <int kObjective, bool kFastNoise, int kUnroll>
__global__ void __launch_bounds__(256, NETMAX_ROUND_MIN_CTAS) round_kernel(const RoundParams p) {
  extern __shared__ __align__(16) unsigned char smem_raw[];
  int32_t* s_peer = reinterpret_cast<int32_t*>(smem_raw);
  float* s_w = reinterpret_cast<float*>(s_peer + p.M);
  const size_t head = (((size_t)p.M * 8) + 15) & ~(size_t)15;
  float4* s_col = reinterpret_cast<float4*>(smem_raw + head);
  double* s_red = reinterpret_cast<double*>(smem_raw + head + (p.rl > 1 ? (size_t)blockDim.x * 32 : 0));

  const int tid = threadIdx.x;
  for (int i = tid; i < p.M; i += blockDim.x) {
    const int32_t m = __ldg(p.peers + i);
    s_peer[i] = m;
    s_w[i] = (m == i) ? 0.0f : __ldg(p.wtab + (size_t)i * p.M + m);
  }
  __syncthreads();

  const int cgi = tid & (p.cg - 1);
  const int rli = tid / p.cg;
  const int M = p.M;
  const int step = p.rl;
  double acc_cons = 0.0, acc_loss = 0.0;

  for (int64_t tile = blockIdx.x; tile < p.n_tiles; tile += gridDim.x) {
    const int64_t q = tile * p.cg + cgi;
    const bool live = q < p.nq;
    const bool ragged = (p.tail != 0) && (q == p.nq - 1);
    float4 s1 = make_float4(0.f, 0.f, 0.f, 0.f), s2 = s1;
    float loss = 0.f;
    if (live) {
      const float4 pivot = __ldg(p.x_cur + q);  // row 0: pivot of the one-pass variance
      for (int i0 = rli; i0 < M; i0 += step * kUnroll) {
        float4 xv[kUnroll], cv[kUnroll], xm[kUnroll];
        float wv[kUnroll];
#pragma unroll
        for (int u = 0; u < kUnroll; ++u) {
          const int i = i0 + u * step;
          if (i < M) {
            const int m = s_peer[i];
            wv[u] = s_w[i];
            xv[u] = __ldg(p.x_cur + (size_t)i * p.ldq + q);
            xm[u] = __ldg(p.x_cur + (size_t)m * p.ldq + q);
            cv[u] = ld_stream(p.c + (size_t)i * p.ldq + q);
          }
        }
#pragma unroll
        for (int u = 0; u < kUnroll; ++u) {
          const int i = i0 + u * step;
          if (i < M) {
            float4 o = update_group<kObjective, kFastNoise>(p, (uint32_t)q + p.q_offset, (uint32_t)i, xv[u], cv[u], xm[u], wv[u]);
            if (ragged) {  // keep the padding lanes of the last group at zero
              if (p.tail < 2) o.y = 0.f;
              if (p.tail < 3) o.z = 0.f;
              o.w = 0.f;
            }
            st_stream(p.x_nxt + (size_t)i * p.ldq + q, o);
            const float dx = xv[u].x - pivot.x, dy = xv[u].y - pivot.y, dz = xv[u].z - pivot.z, dw = xv[u].w - pivot.w;
            s1.x += dx; s1.y += dy; s1.z += dz; s1.w += dw;
            s2.x = fmaf(dx, dx, s2.x); s2.y = fmaf(dy, dy, s2.y); s2.z = fmaf(dz, dz, s2.z); s2.w = fmaf(dw, dw, s2.w);
            const float ex = xv[u].x - cv[u].x, ey = xv[u].y - cv[u].y, ez = xv[u].z - cv[u].z, ew = xv[u].w - cv[u].w;
            loss = fmaf(ex, ex, fmaf(ey, ey, fmaf(ez, ez, fmaf(ew, ew, loss))));
          }
        }
      }
    }
    if (p.rl > 1) {  // sum the column statistics over the row lanes (stride cg in tid)
      s_col[tid] = s1;
      s_col[blockDim.x + tid] = s2;
      __syncthreads();
      for (int s = blockDim.x >> 1; s >= p.cg; s >>= 1) {
        if (tid < s) {
          float4 a = s_col[tid], b = s_col[tid + s];
          a.x += b.x; a.y += b.y; a.z += b.z; a.w += b.w;
          s_col[tid] = a;
          a = s_col[blockDim.x + tid]; b = s_col[blockDim.x + tid + s];
          a.x += b.x; a.y += b.y; a.z += b.z; a.w += b.w;
          s_col[blockDim.x + tid] = a;
        }
        __syncthreads();
      }
      s1 = s_col[cgi];
      s2 = s_col[blockDim.x + cgi];
      __syncthreads();
    }
    if (rli == 0) {
      // sum_i (x_i - xbar)^2 = sum_i (x_i - a)^2 - (sum_i (x_i - a))^2 / M   per column
      const float cons = (s2.x - s1.x * s1.x * p.inv_M) + (s2.y - s1.y * s1.y * p.inv_M) +
                         (s2.z - s1.z * s1.z * p.inv_M) + (s2.w - s1.w * s1.w * p.inv_M);
      acc_cons += (double)cons;
    }
    acc_loss += (double)loss;
  }

  // block reduction of the two doubles, then the last CTA to finish sums all partials in
  // index order (deterministic) and publishes the round's telemetry.
  acc_loss *= 0.5;
  for (int off = 16; off > 0; off >>= 1) {
    acc_cons += __shfl_down_sync(0xffffffffu, acc_cons, off);
    acc_loss += __shfl_down_sync(0xffffffffu, acc_loss, off);
  }
  const int warp = tid >> 5, lane = tid & 31, nwarps = blockDim.x >> 5;
  if (lane == 0) {
    s_red[warp] = acc_cons;
    s_red[32 + warp] = acc_loss;
  }
  __syncthreads();
  __shared__ bool s_last;
  if (tid == 0) {
    double a = 0.0, b = 0.0;
    for (int wi = 0; wi < nwarps; ++wi) {
      a += s_red[wi];
      b += s_red[32 + wi];
    }
    p.partials[2 * (size_t)blockIdx.x] = a;
    p.partials[2 * (size_t)blockIdx.x + 1] = b;
    __threadfence();
    const unsigned int t = atomicAdd(p.ticket, 1u);
    s_last = (t == gridDim.x - 1);
  }
  __syncthreads();
  if (s_last) {
    __threadfence();
    double a = 0.0, b = 0.0;
    for (unsigned int j = tid; j < gridDim.x; j += blockDim.x) {
      a += __ldcg(p.partials + 2 * (size_t)j);
      b += __ldcg(p.partials + 2 * (size_t)j + 1);
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
      p.tel_out[0] = a * (double)p.inv_M;
      p.tel_out[1] = b * (double)p.inv_M;
      *p.ticket = 0u;
    }
  }
}

// ------------------------------------------------------------------------- init / IO
struct InitParams {
  float4* dst;  // [M][ldq]
  int64_t ldq, nq;
  int32_t M, tail;
  float stddev;
  uint32_t tag;
  uint32_t q_offset;
  PhiloxKeys keys;
};

__global__ void __launch_bounds__(256) init_normal_kernel(const InitParams p) {
  const int64_t total = (int64_t)p.M * p.nq;
  for (int64_t idx = blockIdx.x * (int64_t)blockDim.x + threadIdx.x; idx < total;
       idx += (int64_t)gridDim.x * blockDim.x) {
    const int64_t i = idx / p.nq, q = idx - i * p.nq;
    float4 z = normals4<false>(philox4x32_10((uint32_t)q + p.q_offset, (uint32_t)i, 0u, p.tag, p.keys));
    z.x *= p.stddev; z.y *= p.stddev; z.z *= p.stddev; z.w *= p.stddev;
    if (p.tail != 0 && q == p.nq - 1) {
      if (p.tail < 2) z.y = 0.f;
      if (p.tail < 3) z.z = 0.f;
      z.w = 0.f;
    }
    p.dst[(size_t)i * p.ldq + q] = z;
  }
}

__global__ void __launch_bounds__(256) gather_columns_kernel(const float* x, int64_t ld, int32_t M, const int64_t* cols,
                                                             int64_t n_cols, float* out) {
  const int64_t total = (int64_t)M * n_cols;
  for (int64_t idx = blockIdx.x * (int64_t)blockDim.x + threadIdx.x; idx < total;
       idx += (int64_t)gridDim.x * blockDim.x) {
    const int64_t i = idx / n_cols, k = idx - i * n_cols;
    out[idx] = x[(size_t)i * ld + cols[k]];
  }
}

}  // namespace netmax
