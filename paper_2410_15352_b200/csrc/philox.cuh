// Device-side generator of the projection P (Algorithm 1 lines 1-2, Algorithm 3
// lines 6-7, Section 3.3): Philox4x32-10 keyed by the 64-bit layer seed with
// counter (column group j >> 3, row, layer_id, epoch), followed by Box-Muller with
// 16 bits per uniform: one call yields the eight entries P[i, 8q .. 8q+7].
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

// Ten rounds starting from the state after `first` rounds.
template <int kFirst>
__device__ __forceinline__ uint4 philox_rounds(uint32_t c0, uint32_t c1, uint32_t c2, uint32_t c3, const PhiloxKey& key) {
#pragma unroll
  for (int i = kFirst; i < 10; ++i) {
    const uint64_t p0 = (uint64_t)0xD2511F53u * c0;   // one wide multiply each
    const uint64_t p1 = (uint64_t)0xCD9E8D57u * c2;
    c0 = (uint32_t)(p1 >> 32) ^ c1 ^ key.k0[i];
    c1 = (uint32_t)p1;
    c2 = (uint32_t)(p0 >> 32) ^ c3 ^ key.k1[i];
    c3 = (uint32_t)p0;
  }
  return make_uint4(c0, c1, c2, c3);
}

__device__ __forceinline__ uint4 philox4x32_10(uint32_t c0, uint32_t c1, uint32_t c2, uint32_t c3,
                                               const PhiloxKey& key) {
  return philox_rounds<0>(c0, c1, c2, c3, key);
}

// Same function for the projection's counter (q, i, layer_id, epoch): the third counter word is
// the same for every entry of a layer, so its first-round product 0xCD9E8D57 * layer_id is
// computed once on the host (hi, lo) and the first round needs one wide multiply instead of two.
__device__ __forceinline__ uint4 philox4x32_10_layer(uint32_t q, uint32_t i, uint32_t epoch, uint32_t layer_hi,
                                                     uint32_t layer_lo, const PhiloxKey& key) {
  const uint64_t p0 = (uint64_t)0xD2511F53u * q;
  const uint32_t c0 = layer_hi ^ i ^ key.k0[0];
  const uint32_t c1 = layer_lo;
  const uint32_t c2 = (uint32_t)(p0 >> 32) ^ epoch ^ key.k1[0];
  const uint32_t c3 = (uint32_t)p0;
  return philox_rounds<1>(c0, c1, c2, c3, key);
}

// One word makes a pair of standard normals: its low half is the radius' uniform u1 = ((x & 0xffff) + 0.5) 2^-16 in
// (0,1), its high half the angle's u2 = (x >> 16) 2^-16 in [0,1); the pair is (rad cos(2 pi u2), rad sin(2 pi u2)).
// Word w of the call for column group q makes columns 8q + 2w and 8q + 2w + 1.
__device__ __forceinline__ void box_muller(uint32_t x, float& c, float& s) {
  const float u1 = ((float)(x & 0xFFFFu) + 0.5f) * 1.52587890625e-05f;     // 2^-16
  const float u2 = (float)(x >> 16) * 1.52587890625e-05f;
  const float rad = sqrtf(-2.0f * logf(u1));
  float sn, cs;
  sincospif(2.0f * u2, &sn, &cs);
  c = rad * cs;
  s = rad * sn;
}

// The same pair already scaled by 1/sqrt(r), built from the hardware
// approximations (lg2/sqrt/sin/cos) and bit tricks instead of int->float
// conversions.  Used where P is rounded to bf16 anyway.
//   u1 = float(1.m) - 1 with mantissa m = (x & 0xffff) << 7 | 0x40      (exact)
//   2 pi u2 = pi*[x>>31] + pi * ((x>>16) & 0x7fff) 2^-15: the top bit of u2
//   adds pi to the angle, which flips the sign of both cos and sin.
// neg2ln2_over_r = -2 ln(2) / r, so sqrt(lg2(u1) * neg2ln2_over_r) = sqrt(-2 ln u1) / sqrt(r).
__device__ __forceinline__ float sqrt_approx(float x) {
  float y;
  asm("sqrt.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}
// Flush-to-zero forms: every argument here is a normal number or zero, and they spare the
// instructions that rescale denormal arguments.
__device__ __forceinline__ float lg2_approx(float x) {
  float y;
  asm("lg2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}
__device__ __forceinline__ float sin_approx(float x) {
  float y;
  asm("sin.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}
__device__ __forceinline__ float cos_approx(float x) {
  float y;
  asm("cos.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}
__device__ __forceinline__ void box_muller_fast(uint32_t x, float neg2ln2_over_r, float& c, float& s) {
  const float u1 = __uint_as_float(((x << 7) & 0x007FFF80u) | 0x3F800040u) - 1.0f;     // at most 1 - 2^-17: lg2 < 0
  const float rad = sqrt_approx(lg2_approx(u1) * neg2ln2_over_r);
  const float th = (__uint_as_float(((x >> 8) & 0x007FFF00u) | 0x3F800000u) - 1.0f) * 3.14159265358979f;
  const float rs = __uint_as_float(__float_as_uint(rad) ^ (x & 0x80000000u));
  c = rs * cos_approx(th);
  s = rs * sin_approx(th);
}

struct ProjectionParams {
  PhiloxKey key;
  uint32_t layer_id;
  uint32_t layer_hi, layer_lo;   // 0xCD9E8D57 * layer_id, high and low words
  uint32_t epoch;
  int32_t n;
  int32_t r;
  float inv_sqrt_r;
  float neg2ln2_over_r;
  int32_t sparse_s;              // > 0: sparse Johnson-Lindenstrauss projection with this many terms per row
  float inv_sqrt_s;
};

// Sparse Johnson-Lindenstrauss projection (the paper's ablation study; the construction it cites hashes every
// input coordinate s times into the r outputs with random signs, scaled by 1/sqrt(s); colliding terms add).
// Terms 4q .. 4q+3 of row i are the words of the Philox call with counter (0x80000000 | q, i, layer_id, epoch):
// the top bit of a word is the sign, its low 31 bits pick the column as ((word & 0x7fffffff) * r) >> 31.
__device__ __forceinline__ uint4 sparse_words4(uint32_t q, uint32_t i, uint32_t epoch, uint32_t layer_hi, uint32_t layer_lo,
                                               const PhiloxKey& key) {
  return philox4x32_10_layer(0x80000000u | q, i, epoch, layer_hi, layer_lo, key);
}
__device__ __forceinline__ int sparse_col(uint32_t word, int r) { return (int)__umulhi(word << 1, (uint32_t)r); }
__device__ __forceinline__ float sparse_sign(uint32_t word) { return (word >> 31) ? -1.0f : 1.0f; }

// Entry (i, j) of the sparse projection as its integer count (the sum of the signs of the terms of row i that
// hash to column j); the caller scales by 1/sqrt(s).
__device__ __forceinline__ float sparse_count(const ProjectionParams& pp, int i, int j) {
  float k = 0.f;
  for (int q = 0; 4 * q < pp.sparse_s; ++q) {
    const uint4 x = sparse_words4((uint32_t)q, (uint32_t)i, pp.epoch, pp.layer_hi, pp.layer_lo, pp.key);
    const uint32_t w[4] = {x.x, x.y, x.z, x.w};
#pragma unroll
    for (int l = 0; l < 4; ++l)
      if (4 * q + l < pp.sparse_s && sparse_col(w[l], pp.r) == j) k += sparse_sign(w[l]);
  }
  return k;
}

// Entry (i, j) of P in fp32; zero outside n x r.
// kFast selects the approximate Box-Muller (bf16 layers); fp32 layers use the accurate one.
template <bool kFast>
__device__ __forceinline__ float projection1(const ProjectionParams& pp, int i, int j) {
  if (i >= pp.n || j >= pp.r) return 0.f;
  if (pp.sparse_s > 0) return sparse_count(pp, i, j) * pp.inv_sqrt_s;
  const uint4 x = philox4x32_10_layer((uint32_t)(j >> 3), (uint32_t)i, pp.epoch, pp.layer_hi, pp.layer_lo, pp.key);
  const int w = (j >> 1) & 3;
  const uint32_t word = w == 0 ? x.x : (w == 1 ? x.y : (w == 2 ? x.z : x.w));
  float c, s;
  if (kFast) {
    box_muller_fast(word, pp.neg2ln2_over_r, c, s);
  } else {
    box_muller(word, c, s);
    c *= pp.inv_sqrt_r;
    s *= pp.inv_sqrt_r;
  }
  return (j & 1) ? s : c;
}

}  // namespace compact
