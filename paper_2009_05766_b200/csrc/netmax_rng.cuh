// Device-side random numbers of the NetMax round simulator: Philox4x32-10 (Salmon, Moraes,
// Dror, Shaw, SC'11) and a Box-Muller transform on fixed-point uniforms.
//
// The paper only assumes additive gradient noise with zero mean and bounded variance
// (Assumption 1); the generator, the counter layout and the uniform-to-normal map are this
// library's choice and are documented in the C header's conventions.
#pragma once
#include <cstdint>
#include <cuda_runtime.h>

namespace netmax {

constexpr uint32_t kPhiloxMul0 = 0xD2511F53u;
constexpr uint32_t kPhiloxMul1 = 0xCD9E8D57u;
constexpr uint32_t kPhiloxWeyl0 = 0x9E3779B9u;
constexpr uint32_t kPhiloxWeyl1 = 0xBB67AE85u;

// Streams (fourth counter word, low byte).
constexpr uint32_t kTagPeer = 1, kTagNoise = 2, kTagX0 = 3, kTagC = 4;

// The ten round keys of one seed, expanded once on the host (the key schedule does not
// depend on the counter, so every thread shares it).
struct PhiloxKeys {
  uint32_t k0[10];
  uint32_t k1[10];
};

inline PhiloxKeys make_philox_keys(uint64_t seed) {
  PhiloxKeys k;
  uint32_t a = (uint32_t)seed, b = (uint32_t)(seed >> 32);
  for (int r = 0; r < 10; ++r) {
    k.k0[r] = a;
    k.k1[r] = b;
    a += kPhiloxWeyl0;
    b += kPhiloxWeyl1;
  }
  return k;
}

// Counter layout: (column group e/4, worker, round low word, tag | round high bits << 8).
__host__ __device__ __forceinline__ uint32_t philox_ctr3(uint32_t tag, uint64_t round) {
  return tag | ((uint32_t)(round >> 32) << 8);
}

__device__ __forceinline__ uint4 philox4x32_10(uint32_t c0, uint32_t c1, uint32_t c2, uint32_t c3,
                                               const PhiloxKeys& keys) {
#pragma unroll
  for (int r = 0; r < 10; ++r) {
    const uint64_t p0 = (uint64_t)kPhiloxMul0 * c0;  // one 32x32->64 multiply each
    const uint64_t p1 = (uint64_t)kPhiloxMul1 * c2;
    const uint32_t n0 = (uint32_t)(p1 >> 32) ^ c1 ^ keys.k0[r];
    const uint32_t n2 = (uint32_t)(p0 >> 32) ^ c3 ^ keys.k1[r];
    c0 = n0;
    c1 = (uint32_t)p1;
    c2 = n2;
    c3 = (uint32_t)p0;
  }
  return make_uint4(c0, c1, c2, c3);
}

// u1 = (top23(a) + 1/2) / 2^23 in (0,1), exactly representable in fp32:
// bits 0x3F800000 | top23 are the float 1 + top23 / 2^23; subtracting 1 - 2^-24 is exact.
__device__ __forceinline__ float radius_uniform(uint32_t a) {
  return __uint_as_float(0x3F800000u | (a >> 9)) - 0.99999994039535522461f;
}

// Hardware log2 of a normal number (u1 >= 2^-24 here, so flushing subnormals changes nothing
// and saves the subnormal-input handling around the instruction).
__device__ __forceinline__ float log2_fast(float v) {
#ifdef NETMAX_LG2_NO_FTZ
  return __log2f(v);
#else
  float r;
  asm("lg2.approx.ftz.f32 %0, %1;" : "=f"(r) : "f"(v));
  return r;
#endif
}

// Accurate pair (library logf / sincospif / sqrtf): used where speed does not matter.
__device__ __forceinline__ void normal_pair_accurate(uint32_t a, uint32_t b, float& z0, float& z1) {
  const float u1 = radius_uniform(a);
  const float turns2 = (float)((int32_t)b >> 8) * 1.1920928955078125e-07f;  // 2 u2 in [-1, 1)
  const float rad = sqrtf(-2.0f * logf(u1));
  float s, c;
  sincospif(turns2, &s, &c);
  z0 = rad * c;
  z1 = rad * s;
}

// ---- packed fp32x2 arithmetic (sm_100: two IEEE fp32 operations per instruction) ----------
typedef unsigned long long pair_t;  // two floats in one 64-bit register: (low lane, high lane)

__device__ __forceinline__ pair_t pack2(float lo, float hi) {
  pair_t r;
  asm("mov.b64 %0, {%1, %2};" : "=l"(r) : "f"(lo), "f"(hi));
  return r;
}
__device__ __forceinline__ void unpack2(pair_t v, float& lo, float& hi) {
  asm("mov.b64 {%0, %1}, %2;" : "=f"(lo), "=f"(hi) : "l"(v));
}
__device__ __forceinline__ pair_t fma2(pair_t a, pair_t b, pair_t c) {
  pair_t d;
  asm("fma.rn.f32x2 %0, %1, %2, %3;" : "=l"(d) : "l"(a), "l"(b), "l"(c));
  return d;
}
__device__ __forceinline__ pair_t mul2(pair_t a, pair_t b) {
  pair_t d;
  asm("mul.rn.f32x2 %0, %1, %2;" : "=l"(d) : "l"(a), "l"(b));
  return d;
}
__device__ __forceinline__ pair_t add2(pair_t a, pair_t b) {
  pair_t d;
  asm("add.rn.f32x2 %0, %1, %2;" : "=l"(d) : "l"(a), "l"(b));
  return d;
}

// The two normals of one Box-Muller pair, packed, fast path, WITHOUT the constant factor of the
// radius: returns sqrt(-log2 u1) (cos 2 pi u2, sin 2 pi u2), i.e. the pair of normals divided by
// kNormalScale = sqrt(2 ln 2); the caller folds that constant into its noise scale.
// u1 < 1, so log2 u1 < 0; the hardware logarithm has an absolute error of about 2^-22 and may
// return +0 or a tiny positive value for u1 next to 1, hence |.| (an operand modifier, not an
// instruction) instead of a negation under the square root.
constexpr double kNormalScale = 1.17741002251547469101;  // sqrt(2 ln 2)
__device__ __forceinline__ pair_t normal_pair_fast_unscaled(uint32_t a, uint32_t b) {
  const float u1 = radius_uniform(a);
  const float ang = (float)((int32_t)b >> 8) * 3.74507028e-07f;  // 2 pi / 2^24
  float rad;
  asm("sqrt.approx.ftz.f32 %0, %1;" : "=f"(rad) : "f"(fabsf(log2_fast(u1))));
  float s, c;
  __sincosf(ang, &s, &c);
  return mul2(pack2(rad, rad), pack2(c, s));
}

template <bool kFast>
__device__ __forceinline__ float4 normals4(uint4 r) {
  float4 z;
  if (kFast) {  // (the update kernels use normal_pair_fast_unscaled directly and fold the constant into their noise scale)
    unpack2(normal_pair_fast_unscaled(r.x, r.y), z.x, z.y);
    unpack2(normal_pair_fast_unscaled(r.z, r.w), z.z, z.w);
    z.x *= (float)kNormalScale; z.y *= (float)kNormalScale; z.z *= (float)kNormalScale; z.w *= (float)kNormalScale;
  } else {
    normal_pair_accurate(r.x, r.y, z.x, z.y);
    normal_pair_accurate(r.z, r.w, z.z, z.w);
  }
  return z;
}

}  // namespace netmax
