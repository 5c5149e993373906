// Device-side generator of the projection P (Algorithm 1 lines 1-2, Algorithm 3
// lines 6-7, Section 3.3): Philox4x32-10 keyed by the 64-bit layer seed with
// counter (column group, row, layer_id, epoch), followed by Box-Muller.
// Entry (i, j) of P is a pure function of (seed, layer_id, epoch, i, j).
#pragma once
#include <cuda_bf16.h>
#include <stdint.h>

namespace compact {

struct PhiloxKey {
  // Round keys are the same for every call of one launch; precomputed on the host.
  uint32_t k0[10];
  uint32_t k1[10];
};

__host__ __device__ inline PhiloxKey make_philox_key(uint64_t seed) {
  PhiloxKey k;
  uint32_t a = (uint32_t)seed, b = (uint32_t)(seed >> 32);
  for (int i = 0; i < 10; ++i) {
    k.k0[i] = a;
    k.k1[i] = b;
    a += 0x9E3779B9u;
    b += 0xBB67AE85u;
  }
  return k;
}

__device__ __forceinline__ uint4 philox4x32_10(uint32_t c0, uint32_t c1, uint32_t c2, uint32_t c3,
                                               const PhiloxKey& key) {
#pragma unroll
  for (int i = 0; i < 10; ++i) {
    const uint32_t hi0 = __umulhi(0xD2511F53u, c0), lo0 = 0xD2511F53u * c0;
    const uint32_t hi1 = __umulhi(0xCD9E8D57u, c2), lo1 = 0xCD9E8D57u * c2;
    c0 = hi1 ^ c1 ^ key.k0[i];
    c1 = lo1;
    c2 = hi0 ^ c3 ^ key.k1[i];
    c3 = lo0;
  }
  return make_uint4(c0, c1, c2, c3);
}

// Four consecutive entries P[i, 4q .. 4q+3] before the 1/sqrt(r) scale.
// Words (0,1) make the (cos, sin) pair of columns 4q, 4q+1; words (2,3) that of 4q+2, 4q+3.
__device__ __forceinline__ float4 gaussian4(uint4 x) {
  const float u1a = ((float)(x.x >> 9) + 0.5f) * 1.1920928955078125e-07f;   // 2^-23, in (0,1)
  const float u2a = (float)(x.y >> 8) * 5.9604644775390625e-08f;            // 2^-24, in [0,1)
  const float u1b = ((float)(x.z >> 9) + 0.5f) * 1.1920928955078125e-07f;
  const float u2b = (float)(x.w >> 8) * 5.9604644775390625e-08f;
  const float ra = sqrtf(-2.0f * logf(u1a));
  const float rb = sqrtf(-2.0f * logf(u1b));
  float sa, ca, sb, cb;
  sincospif(2.0f * u2a, &sa, &ca);
  sincospif(2.0f * u2b, &sb, &cb);
  return make_float4(ra * ca, ra * sa, rb * cb, rb * sb);
}

struct ProjectionParams {
  PhiloxKey key;
  uint32_t layer_id;
  uint32_t epoch;
  int32_t n;
  int32_t r;
  float inv_sqrt_r;
};

// P[i, 4q .. 4q+3] in fp32; columns >= r are zero, rows >= n are zero.
__device__ __forceinline__ float4 projection4(const ProjectionParams& pp, int i, int q) {
  if (i >= pp.n || 4 * q >= pp.r) return make_float4(0.f, 0.f, 0.f, 0.f);
  float4 g = gaussian4(philox4x32_10((uint32_t)q, (uint32_t)i, pp.layer_id, pp.epoch, pp.key));
  g.x *= pp.inv_sqrt_r;
  g.y = (4 * q + 1 < pp.r) ? g.y * pp.inv_sqrt_r : 0.f;
  g.z = (4 * q + 2 < pp.r) ? g.z * pp.inv_sqrt_r : 0.f;
  g.w = (4 * q + 3 < pp.r) ? g.w * pp.inv_sqrt_r : 0.f;
  return g;
}

__device__ __forceinline__ float projection1(const ProjectionParams& pp, int i, int j) {
  const float4 g = projection4(pp, i, j >> 2);
  const int l = j & 3;
  return l == 0 ? g.x : (l == 1 ? g.y : (l == 2 ? g.z : g.w));
}

}  // namespace compact
