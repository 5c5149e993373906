// Plain FFMA kernels for the CompAct layer.  They serve the fp32 configuration
// (tensor-core tf32 cannot reach 1e-5) and shapes the tensor-core kernels do not
// take, and they are the on-device cross-check of the tcgen05 kernels.
// One generic tiled GEMM whose operands are read through small functors, so the
// same loop covers Y = X W, Z = X P (P generated), dX = dY W^T, Gc = Z^T dY and
// W -= scale * P N.
#pragma once
#include <cuda_bf16.h>
#include <stdint.h>

#include "philox.cuh"

namespace compact {
namespace simt {

__device__ __forceinline__ float to_f32(float v) { return v; }
__device__ __forceinline__ float to_f32(__nv_bfloat16 v) { return __bfloat162float(v); }
template <typename T> __device__ __forceinline__ T from_f32(float v);
template <> __device__ __forceinline__ float from_f32<float>(float v) { return v; }
template <> __device__ __forceinline__ __nv_bfloat16 from_f32<__nv_bfloat16>(float v) { return __float2bfloat16_rn(v); }

// element (row, k) of a row-major matrix
template <typename T> struct RowMajor {
  const T* p; int64_t ld;
  __device__ __forceinline__ float operator()(int row, int k) const { return to_f32(p[(int64_t)row * ld + k]); }
};
// element (row, k) of the transpose of a row-major matrix
template <typename T> struct Transposed {
  const T* p; int64_t ld;
  __device__ __forceinline__ float operator()(int row, int k) const { return to_f32(p[(int64_t)k * ld + row]); }
};
// P[i, j] generated; as the B operand of Z = X P it is indexed (k = i, col = j),
// as the A operand of P N it is indexed (row = i, k = j).
template <bool kRoundBf16, bool kAsB> struct GeneratedP {
  ProjectionParams pp;
  __device__ __forceinline__ float operator()(int a, int b) const {
    const int i = kAsB ? b : a, j = kAsB ? a : b;
    float v = projection1<kRoundBf16>(pp, i, j);
    // Gaussian entries are stored as bf16 in bf16 layers; the sparse projection's multiples of 1/sqrt(s) are not rounded
    if (kRoundBf16 && pp.sparse_s == 0) v = __bfloat162float(__float2bfloat16_rn(v));
    return v;
  }
};

template <typename T> struct StoreAs {
  T* p; int64_t ld;
  __device__ __forceinline__ void operator()(int row, int col, float acc) const { p[(int64_t)row * ld + col] = from_f32<T>(acc); }
};
struct StoreF32 {
  float* p; int64_t ld; int accumulate;
  __device__ __forceinline__ void operator()(int row, int col, float acc) const {
    float* q = p + (int64_t)row * ld + col;
    *q = accumulate ? *q + acc : acc;
  }
};
// Algorithm 3 line 9: W <- W - eta * alpha * (P N), one rounding of the result.
template <typename T> struct ApplyUpdate {
  T* W; int64_t ld; float scale;
  __device__ __forceinline__ void operator()(int row, int col, float acc) const {
    T* q = W + (int64_t)row * ld + col;
    *q = from_f32<T>(fmaf(-scale, acc, to_f32(*q)));
  }
};

// C[M x N] = sum_k A(row, k) * B(col, k).  64x64 tile, 256 threads, 4x4 per thread.
template <class AF, class BF, class EP>
__global__ void __launch_bounds__(256) gemm_kernel(int M, int N, int K, AF a, BF b, EP ep) {
  constexpr int BM = 64, BN = 64, BK = 16;
  __shared__ float sA[BK][BM + 1];
  __shared__ float sB[BK][BN + 1];
  const int tid = threadIdx.x;
  const int row0 = blockIdx.y * BM, col0 = blockIdx.x * BN;
  const int ty = tid / 16, tx = tid % 16;
  float acc[4][4] = {};
  for (int k0 = 0; k0 < K; k0 += BK) {
#pragma unroll
    for (int s = 0; s < 4; ++s) {
      const int idx = tid + s * 256;
      const int k = idx % BK, rr = idx / BK;
      const int gk = k0 + k;
      sA[k][rr] = (row0 + rr < M && gk < K) ? a(row0 + rr, gk) : 0.f;
      sB[k][rr] = (col0 + rr < N && gk < K) ? b(col0 + rr, gk) : 0.f;
    }
    __syncthreads();
#pragma unroll
    for (int k = 0; k < BK; ++k) {
      float av[4], bv[4];
#pragma unroll
      for (int i = 0; i < 4; ++i) av[i] = sA[k][ty * 4 + i];
#pragma unroll
      for (int j = 0; j < 4; ++j) bv[j] = sB[k][tx * 4 + j];
#pragma unroll
      for (int i = 0; i < 4; ++i)
#pragma unroll
        for (int j = 0; j < 4; ++j) acc[i][j] = fmaf(av[i], bv[j], acc[i][j]);
    }
    __syncthreads();
  }
#pragma unroll
  for (int i = 0; i < 4; ++i)
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      const int rr = row0 + ty * 4 + i, cc = col0 + tx * 4 + j;
      if (rr < M && cc < N) ep(rr, cc, acc[i][j]);
    }
}

// Zero the pad columns r .. ldz-1 of Z.
template <typename T>
__global__ void zero_pad_columns(T* Z, int64_t ldz, int64_t tokens, int r, int ldz_cols) {
  const int pad = ldz_cols - r;
  const int64_t idx = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (pad <= 0 || idx >= tokens * pad) return;
  const int64_t t = idx / pad;
  const int c = r + (int)(idx % pad);
  Z[t * ldz + c] = from_f32<T>(0.f);
}

struct AdamScalars {
  float beta1, beta2, one_minus_beta1, one_minus_beta2;
  float inv_bias1, inv_bias2;   // 1 / (1 - beta^t)
  float eps;
};

// Algorithm 3 lines 1-5 on an r x m grid: moments in place, N written to scratch.
template <bool kRoundBf16>
__global__ void adam_moments_kernel(const float* __restrict__ Gc, int64_t ldg, float* __restrict__ Mo,
                                    float* __restrict__ Vo, float* __restrict__ Nout, int64_t ldn,
                                    int r, int m, AdamScalars s) {
  const int64_t idx = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (idx >= (int64_t)r * m) return;
  const int j = (int)(idx / m), c = (int)(idx % m);
  const float g = Gc[(int64_t)j * ldg + c];
  const float mm = fmaf(s.beta1, Mo[(int64_t)j * ldg + c], s.one_minus_beta1 * g);
  const float vv = fmaf(s.beta2, Vo[(int64_t)j * ldg + c], s.one_minus_beta2 * g * g);
  Mo[(int64_t)j * ldg + c] = mm;
  Vo[(int64_t)j * ldg + c] = vv;
  float nn = (mm * s.inv_bias1) / (sqrtf(vv * s.inv_bias2) + s.eps);
  if (kRoundBf16) nn = __bfloat162float(__float2bfloat16_rn(nn));
  Nout[(int64_t)j * ldn + c] = nn;
}

}  // namespace simt

// Debug kernels: make the generator observable.
__global__ void debug_philox_words_kernel(PhiloxKey key, uint32_t layer_id, uint32_t epoch, int n, int groups,
                                          uint32_t* out) {
  const int64_t idx = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (idx >= (int64_t)n * groups) return;
  const int i = (int)(idx / groups), q = (int)(idx % groups);
  const uint4 x = philox4x32_10((uint32_t)q, (uint32_t)i, layer_id, epoch, key);
  reinterpret_cast<uint4*>(out)[idx] = x;
}

// The same words through the form the GEMM kernels' generators call: the first round's product with the
// layer word comes precomputed from the host.
__global__ void debug_philox_layer_words_kernel(PhiloxKey key, uint32_t layer_hi, uint32_t layer_lo, uint32_t epoch, int n,
                                                int groups, uint32_t* out) {
  const int64_t idx = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (idx >= (int64_t)n * groups) return;
  const int i = (int)(idx / groups), q = (int)(idx % groups);
  const uint4 x = philox4x32_10_layer((uint32_t)q, (uint32_t)i, epoch, layer_hi, layer_lo, key);
  reinterpret_cast<uint4*>(out)[idx] = x;
}

// The terms of the sparse projection: out[i * s + t] = column | sign bit << 31.
__global__ void debug_sparse_terms_kernel(ProjectionParams pp, uint32_t* out) {
  const int64_t idx = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (idx >= (int64_t)pp.n * pp.sparse_s) return;
  const int i = (int)(idx / pp.sparse_s), t = (int)(idx % pp.sparse_s);
  const uint4 x = sparse_words4((uint32_t)(t >> 2), (uint32_t)i, pp.epoch, pp.layer_hi, pp.layer_lo, pp.key);
  const uint32_t w = (t & 3) == 0 ? x.x : ((t & 3) == 1 ? x.y : ((t & 3) == 2 ? x.z : x.w));
  out[idx] = (uint32_t)sparse_col(w, pp.r) | (w & 0x80000000u);
}

template <typename T>
__global__ void debug_projection_kernel(ProjectionParams pp, T* P) {
  const int64_t idx = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (idx >= (int64_t)pp.n * pp.r) return;
  const int i = (int)(idx / pp.r), j = (int)(idx % pp.r);
  P[idx] = simt::from_f32<T>(projection1<sizeof(T) == 2>(pp, i, j));
}

}  // namespace compact
