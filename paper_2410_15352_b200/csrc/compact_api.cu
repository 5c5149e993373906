// C ABI of the CompAct compressed linear layer (see include/compact.h).
// Host-side bookkeeping, argument validation and kernel dispatch.
#include <cuda_runtime.h>
#include <math.h>
#include <stdint.h>
#include <string.h>

#include <atomic>
#include <mutex>
#include <new>
#include <vector>

#include "../../include/compact.h"
#include "philox.cuh"
#include "simt_kernels.cuh"
#include "tc_kernels.cuh"
#include "gemm2_kernel.cuh"

using namespace compact;

struct compact_layer {
  compact_layer_config_t cfg;
  uint32_t epoch;
  uint64_t step;
  uint64_t last_refresh_step;
  int status_slot;
  int device_checked;   // -1: unsupported, 0: not yet, 1: ok
};

namespace {

std::atomic<uint64_t> g_launches{0};
#ifndef CFG_CS
#define CFG_CS 2   // CTAs of a cluster that share each generated tile of P
#endif
std::atomic<int> g_family{0};

// One status word per live layer: kernels OR error bits into it, compact_layer_status reads and clears it.
// Slots come from a free list and go back on destroy; when none is left, compact_layer_create fails.
constexpr int kStatusSlots = 4096;
__device__ unsigned int g_status_words[kStatusSlots];
// Four words per tensor-core launch for its dynamic schedulers (next item, finished CTAs, ...), taken from a
// ring by launch sequence number, so that launches that overlap on the GPU (other layers, other streams)
// never share them.  Zero at load; the last CTA of a launch leaves them zero again.  The ring is far
// longer than the number of launches that can be in flight at once.
constexpr int kSchedRing = 4096;
__device__ unsigned int g_sched_words[kSchedRing][4];
std::atomic<uint64_t> g_sched_seq{0};

std::mutex g_slot_mutex;
std::vector<int> g_free_slots;
int g_slots_handed_out = 0;

int take_status_slot() {
  std::lock_guard<std::mutex> lock(g_slot_mutex);
  if (!g_free_slots.empty()) {
    const int s = g_free_slots.back();
    g_free_slots.pop_back();
    return s;
  }
  if (g_slots_handed_out < kStatusSlots) return g_slots_handed_out++;
  return -1;
}
void give_back_status_slot(int s) {
  std::lock_guard<std::mutex> lock(g_slot_mutex);
  g_free_slots.push_back(s);
}

// Device addresses of the two arrays, asked once per device (with that device current).
constexpr int kMaxDevices = 64;
std::atomic<unsigned int*> g_status_base[kMaxDevices];
std::atomic<unsigned int*> g_sched_base[kMaxDevices];

template <class Sym>
unsigned int* symbol_base(std::atomic<unsigned int*>* cache, const Sym& sym) {
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) { cudaGetLastError(); return nullptr; }
  unsigned int* p = cache[dev].load(std::memory_order_acquire);
  if (!p) {
    if (cudaGetSymbolAddress((void**)&p, sym) != cudaSuccess || !p) { cudaGetLastError(); return nullptr; }
    cache[dev].store(p, std::memory_order_release);
  }
  return p;
}

inline size_t elem_size(int dtype) { return dtype == COMPACT_BF16 ? 2 : 4; }
inline int64_t round_up(int64_t a, int64_t b) { return (a + b - 1) / b * b; }
inline bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

compact_status_t check_device(compact_layer_t* L, void* stream) {
  if (L->device_checked == 1) return COMPACT_OK;
  if (L->device_checked == -1) return COMPACT_ERR_UNSUPPORTED_ARCH;
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess) { cudaGetLastError(); return COMPACT_ERR_CUDA; }
  int major = 0;
  if (cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, dev) != cudaSuccess) {
    cudaGetLastError();
    return COMPACT_ERR_CUDA;
  }
  if (major != 10) { L->device_checked = -1; return COMPACT_ERR_UNSUPPORTED_ARCH; }
  // the slot may have belonged to a layer that was destroyed without its status having been read
  unsigned int* w = symbol_base(g_status_base, g_status_words);
  if (!w || cudaMemsetAsync(w + L->status_slot, 0, sizeof(unsigned int), (cudaStream_t)stream) != cudaSuccess) {
    cudaGetLastError();
    return COMPACT_ERR_CUDA;
  }
  L->device_checked = 1;
  return COMPACT_OK;
}

unsigned int* status_word(const compact_layer_t* L) {
  unsigned int* base = symbol_base(g_status_base, g_status_words);
  return base ? base + L->status_slot : nullptr;
}

// The scheduler words of the next tensor-core launch.
unsigned int* sched_words(const compact_layer_t*) {
  unsigned int* base = symbol_base(g_sched_base, g_sched_words);
  return base ? base + 4 * (g_sched_seq.fetch_add(1) % kSchedRing) : nullptr;
}

// What every route of the update can work with: N as fp32 r x m (the tensor-core routes keep it in bf16).
size_t update_min_bytes(const compact_layer_t* L) { return (size_t)round_up((int64_t)L->cfg.r * L->cfg.m * (int64_t)sizeof(float), 256); }

ProjectionParams make_pp(const compact_layer_t* L, uint32_t epoch) {
  ProjectionParams pp;
  pp.key = make_philox_key(L->cfg.seed);
  pp.layer_id = L->cfg.layer_id;
  {
    const uint64_t pl = (uint64_t)0xCD9E8D57u * (uint64_t)L->cfg.layer_id;
    pp.layer_hi = (uint32_t)(pl >> 32);
    pp.layer_lo = (uint32_t)pl;
  }
  pp.epoch = epoch;
  pp.n = L->cfg.n;
  pp.r = L->cfg.r;
  pp.inv_sqrt_r = (float)(1.0 / sqrt((double)L->cfg.r));
  pp.neg2ln2_over_r = (float)(-2.0 * 0.6931471805599453 / (double)L->cfg.r);
  pp.sparse_s = L->cfg.sparse_s;
  pp.inv_sqrt_s = L->cfg.sparse_s > 0 ? (float)(1.0 / sqrt((double)L->cfg.sparse_s)) : 1.0f;
  return pp;
}

compact_status_t launch_result() {
  return cudaGetLastError() == cudaSuccess ? COMPACT_OK : COMPACT_ERR_CUDA;
}

template <class AF, class BF, class EP>
void simt_gemm(int M, int N, int K, AF a, BF b, EP ep, cudaStream_t st) {
  dim3 grid((N + 63) / 64, (M + 63) / 64);
  simt::gemm_kernel<AF, BF, EP><<<grid, 256, 0, st>>>(M, N, K, a, b, ep);
  g_launches++;
}

inline bool pitch_ok(int64_t ld, int64_t min_cols, size_t es) { return ld >= min_cols && (ld * (int64_t)es) % 16 == 0; }

// ---- forward ---------------------------------------------------------------------------
// dst[rows x cols] += src[rows x cols] (element type T, one rounding)
template <typename T>
__global__ void add_rows_kernel(T* dst, int64_t ldd, const T* src, int64_t lds, int64_t rows, int cols) {
  const int64_t idx = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (idx >= rows * cols) return;
  const int64_t r = idx / cols;
  const int c = (int)(idx % cols);
  dst[r * ldd + c] = simt::from_f32<T>(simt::to_f32(dst[r * ldd + c]) + simt::to_f32(src[r * lds + c]));
}
template <typename T>
compact_status_t add_rows(T* dst, int64_t ldd, const T* src, int64_t lds, int64_t rows, int cols, cudaStream_t st) {
  const int64_t cnt = rows * cols;
  add_rows_kernel<T><<<(unsigned)((cnt + 255) / 256), 256, 0, st>>>(dst, ldd, src, lds, rows, cols);
  g_launches++;
  return launch_result();
}

template <typename T>
compact_status_t fwd_simt(compact_layer_t* L, int64_t tokens, const T* X, int64_t ldx, const T* W, int64_t ldw,
                          T* Y, int64_t ldy, T* Z, int64_t ldz, cudaStream_t st) {
  constexpr bool kBf16 = sizeof(T) == 2;
  const int n = L->cfg.n, m = L->cfg.m, r = L->cfg.r;
  if (Y) simt_gemm((int)tokens, m, n, simt::RowMajor<T>{X, ldx}, simt::Transposed<T>{W, ldw}, simt::StoreAs<T>{Y, ldy}, st);
  if (!Z) return launch_result();
  simt::GeneratedP<kBf16, true> gp{make_pp(L, L->epoch)};
  simt_gemm((int)tokens, r, n, simt::RowMajor<T>{X, ldx}, gp, simt::StoreAs<T>{Z, ldz}, st);
  const int zc = (int)compact_z_ld(L);
  if (zc > r) {
    const int64_t cnt = tokens * (zc - r);
    simt::zero_pad_columns<T><<<(unsigned)((cnt + 255) / 256), 256, 0, st>>>(Z, ldz, tokens, r, zc);
    g_launches++;
  }
  return launch_result();
}

template <typename T>
compact_status_t bwd_simt(compact_layer_t* L, int64_t tokens, const T* dY, int64_t lddy, const T* Z, int64_t ldz,
                          const T* W, int64_t ldw, T* dX, int64_t lddx, float* Gc, int64_t ldg, int accumulate,
                          cudaStream_t st) {
  const int n = L->cfg.n, m = L->cfg.m, r = L->cfg.r;
  simt_gemm(r, m, (int)tokens, simt::Transposed<T>{Z, ldz}, simt::Transposed<T>{dY, lddy},
            simt::StoreF32{Gc, ldg, accumulate}, st);
  if (dX)
    simt_gemm((int)tokens, n, m, simt::RowMajor<T>{dY, lddy}, simt::RowMajor<T>{W, ldw}, simt::StoreAs<T>{dX, lddx}, st);
  return launch_result();
}

simt::AdamScalars adam_scalars(const compact_layer_t* L, uint64_t t) {
  simt::AdamScalars s;
  const double b1 = (double)L->cfg.beta1, b2 = (double)L->cfg.beta2;
  s.beta1 = L->cfg.beta1;
  s.beta2 = L->cfg.beta2;
  s.one_minus_beta1 = (float)(1.0 - b1);
  s.one_minus_beta2 = (float)(1.0 - b2);
  s.inv_bias1 = (float)(1.0 / (1.0 - pow(b1, (double)t)));
  s.inv_bias2 = (float)(1.0 / (1.0 - pow(b2, (double)t)));
  s.eps = L->cfg.eps;
  return s;
}

template <typename T>
compact_status_t update_simt(compact_layer_t* L, T* W, int64_t ldw, const float* Gc, int64_t ldg, float* M, float* V,
                             float lr, float* Nbuf, cudaStream_t st) {
  constexpr bool kBf16 = sizeof(T) == 2;
  const int n = L->cfg.n, m = L->cfg.m, r = L->cfg.r;
  const simt::AdamScalars s = adam_scalars(L, L->step + 1);
  const int64_t cnt = (int64_t)r * m;
  simt::adam_moments_kernel<kBf16><<<(unsigned)((cnt + 255) / 256), 256, 0, st>>>(Gc, ldg, M, V, Nbuf, m, r, m, s);
  g_launches++;
  simt::GeneratedP<kBf16, false> gp{make_pp(L, L->epoch)};
  simt_gemm(n, m, r, gp, simt::Transposed<float>{Nbuf, m}, simt::ApplyUpdate<T>{W, ldw, lr * L->cfg.alpha}, st);
  return launch_result();
}

}  // namespace

// =========================================================================================
extern "C" {

compact_status_t compact_layer_create(const compact_layer_config_t* cfg, compact_layer_t** out) {
  if (!cfg || !out) return COMPACT_ERR_INVALID_ARG;
  *out = nullptr;
  if (cfg->dtype != COMPACT_F32 && cfg->dtype != COMPACT_BF16) return COMPACT_ERR_DTYPE;
  const int mult = cfg->dtype == COMPACT_BF16 ? 8 : 4;
  if (cfg->n < 1 || cfg->m < 1 || cfg->r < 1 || cfg->r > cfg->n) return COMPACT_ERR_SHAPE;
  if (cfg->n % mult || cfg->m % mult) return COMPACT_ERR_SHAPE;
  if (!(cfg->beta1 >= 0.f && cfg->beta1 < 1.f) || !(cfg->beta2 >= 0.f && cfg->beta2 < 1.f)) return COMPACT_ERR_INVALID_ARG;
  if (!(cfg->eps >= 0.f) || isnan(cfg->lr) || isnan(cfg->alpha)) return COMPACT_ERR_INVALID_ARG;
  if (cfg->sparse_s < 0 || cfg->sparse_s > 64) return COMPACT_ERR_INVALID_ARG;
  compact_layer_t* L = new (std::nothrow) compact_layer_t;
  if (!L) return COMPACT_ERR_INVALID_ARG;
  L->cfg = *cfg;
  L->epoch = 0;
  L->step = 0;
  L->last_refresh_step = 0;
  L->status_slot = take_status_slot();
  if (L->status_slot < 0) { delete L; return COMPACT_ERR_TOO_MANY_LAYERS; }
  L->device_checked = 0;
  *out = L;
  return COMPACT_OK;
}

compact_status_t compact_layer_destroy(compact_layer_t* layer) {
  if (!layer) return COMPACT_ERR_INVALID_ARG;
  give_back_status_slot(layer->status_slot);
  delete layer;
  return COMPACT_OK;
}

int64_t compact_z_ld(const compact_layer_t* layer) { return layer ? round_up(layer->cfg.r, 16) : -1; }

size_t compact_workspace_bytes(const compact_layer_t* layer, int64_t tokens) {
  if (!layer || tokens < 0) return 0;
  const int m = layer->cfg.m, r = layer->cfg.r;
  // update: N as fp32 r x m (SIMT) or bf16 (tensor-core kernels); backward: split-K partials.
  size_t upd = (size_t)r * m * sizeof(float);
  size_t bwd = tc::gc_workspace_bytes(tokens, r, m);
  size_t need = upd > bwd ? upd : bwd;
  const size_t fwd = compact_fwd_workspace_bytes(layer);
  need = fwd > need ? fwd : need;
  // the update's fastest route: N and the expanded P side by side
  if (layer->cfg.dtype == COMPACT_BF16) {
    const size_t u2 = g2::g2_update_scratch_bytes(layer->cfg.n, m, r, (int)compact_z_ld(layer));
    need = u2 > need ? u2 : need;
  }
  return (size_t)round_up((int64_t)need, 256);
}

size_t compact_fwd_workspace_bytes(const compact_layer_t* layer) {
  if (!layer || layer->cfg.dtype != COMPACT_BF16) return 0;
  return (size_t)round_up((int64_t)g2::expanded_bytes(layer->cfg.n, (int)compact_z_ld(layer)), 256);
}

size_t compact_saved_bytes(const compact_layer_t* layer, int64_t tokens) {
  if (!layer || tokens < 0) return 0;
  return (size_t)tokens * (size_t)compact_z_ld(layer) * elem_size(layer->cfg.dtype);
}

compact_status_t compact_linear_fwd(compact_layer_t* L, int64_t tokens, const void* X, int64_t ldx, const void* W,
                                    int64_t ldw, void* Y, int64_t ldy, void* Z, int64_t ldz, uint32_t* epoch_used,
                                    void* workspace, size_t workspace_bytes, void* stream) {
  if (!L || tokens < 0 || tokens > 0x7fffffff) return COMPACT_ERR_INVALID_ARG;
  if (epoch_used) *epoch_used = L->epoch;
  if (tokens == 0) return COMPACT_OK;
  if (!X || !W || !Y) return COMPACT_ERR_INVALID_ARG;
  if (workspace && !aligned16(workspace)) return COMPACT_ERR_ALIGNMENT;
  const size_t es = elem_size(L->cfg.dtype);
  if (!aligned16(X) || !aligned16(W) || !aligned16(Y) || (Z && !aligned16(Z))) return COMPACT_ERR_ALIGNMENT;
  if (!pitch_ok(ldx, L->cfg.n, es) || !pitch_ok(ldw, L->cfg.m, es) || !pitch_ok(ldy, L->cfg.m, es) ||
      (Z && !pitch_ok(ldz, compact_z_ld(L), es)))
    return COMPACT_ERR_ALIGNMENT;
  compact_status_t s = check_device(L, stream);
  if (s != COMPACT_OK) return s;
  cudaStream_t st = (cudaStream_t)stream;
  if (L->cfg.dtype == COMPACT_BF16) {
    typedef __nv_bfloat16 T;
    if (g_family.load() != 1) {
      tc::LaunchInfo li{g_family.load() == 2 ? 1 : CFG_CS, st, status_word(L), sched_words(L), &g_launches};
      // With scratch for the expanded projection: P is written out once, then Z and Y are one product on pairs of SMs.
      if (g_family.load() == 0 && Z && workspace && workspace_bytes >= compact_fwd_workspace_bytes(L)) {
        g2::G2Layer gl;
        gl.pp = make_pp(L, L->epoch);
        gl.m = L->cfg.m; gl.zcols = (int)compact_z_ld(L);
        gl.W = (const T*)W; gl.ldw = ldw; gl.Y = (T*)Y; gl.ldy = ldy; gl.Z = (T*)Z; gl.ldz = ldz;
        s = g2::g2_forward(li, 1, &gl, tokens, L->cfg.n, (const T*)X, ldx, workspace);
        if (s != COMPACT_ERR_SHAPE) return s;
      }
      // Without it P is generated inside the kernel, tile by tile.  Two routes with the same bits.  One launch: the Z
      // items, then the Y items as 256 x 256 tiles on single SMs, which also fill the SMs the Z items leave idle.  Two
      // launches: Z alone, then Y on pairs of SMs, whose epilogues run under the next tile's MMAs (about 3 % on Y).
      // The second pays when that gain outweighs the idle tail of a launch that holds nothing but Z items.
      bool split = false;
      if (g_family.load() == 0 && Z && tokens >= 2 * tc::BN_MAX) {
        const double z_rounds = (double)((compact_z_ld(L) + tc::BM - 1) / tc::BM) * (double)((tokens + 511) / 512) / tc::NUM_SMS;
        const double y_rounds = (double)((tokens + 255) / 256) * (double)((L->cfg.m + 255) / 256) / tc::NUM_SMS;
        split = (ceil(z_rounds) - z_rounds) < 0.03 * y_rounds;
      }
      if (split) {
        s = tc::forward(li, make_pp(L, L->epoch), tokens, L->cfg.m, (const T*)X, ldx, nullptr, 0, nullptr, 0, (T*)Z, ldz, (int)compact_z_ld(L));
        if (s == COMPACT_OK) s = g2::g2_forward_y(li, tokens, L->cfg.n, L->cfg.m, (const T*)X, ldx, (const T*)W, ldw, (T*)Y, ldy);
      } else {
        s = tc::forward(li, make_pp(L, L->epoch), tokens, L->cfg.m, (const T*)X, ldx, (const T*)W, ldw, (T*)Y, ldy, (T*)Z, ldz,
                        (int)compact_z_ld(L));
      }
      if (s != COMPACT_ERR_SHAPE) return s;   // SHAPE: the tensor-core kernels do not take it
    }
    return fwd_simt<T>(L, tokens, (const T*)X, ldx, (const T*)W, ldw, (T*)Y, ldy, (T*)Z, ldz, st);
  }
  return fwd_simt<float>(L, tokens, (const float*)X, ldx, (const float*)W, ldw, (float*)Y, ldy, (float*)Z, ldz, st);
}

compact_status_t compact_linear_bwd(compact_layer_t* L, int64_t tokens, const void* dY, int64_t lddy, const void* Z,
                                    int64_t ldz, const void* W, int64_t ldw, void* dX, int64_t lddx, float* Gc,
                                    int64_t ldg, int accumulate, void* workspace, size_t workspace_bytes,
                                    void* stream) {
  if (!L || tokens < 0 || tokens > 0x7fffffff) return COMPACT_ERR_INVALID_ARG;
  if (!Gc) return COMPACT_ERR_INVALID_ARG;
  const size_t es = elem_size(L->cfg.dtype);
  if (!aligned16(Gc) || !pitch_ok(ldg, L->cfg.m, 4)) return COMPACT_ERR_ALIGNMENT;
  compact_status_t s = check_device(L, stream);
  cudaStream_t st = (cudaStream_t)stream;
  if (tokens == 0) {
    // An empty micro-batch contributes nothing: Gc is zeroed unless accumulating.
    if (accumulate) return COMPACT_OK;
    if (s != COMPACT_OK) return s;
    if (cudaMemset2DAsync(Gc, (size_t)ldg * 4, 0, (size_t)L->cfg.m * 4, (size_t)L->cfg.r, st) != cudaSuccess) {
      cudaGetLastError();
      return COMPACT_ERR_CUDA;
    }
    return COMPACT_OK;
  }
  if (!dY || !Z || !W) return COMPACT_ERR_INVALID_ARG;
  if (!aligned16(dY) || !aligned16(Z) || !aligned16(W) || (dX && !aligned16(dX))) return COMPACT_ERR_ALIGNMENT;
  if (!pitch_ok(lddy, L->cfg.m, es) || !pitch_ok(ldz, compact_z_ld(L), es) || !pitch_ok(ldw, L->cfg.m, es) ||
      (dX && !pitch_ok(lddx, L->cfg.n, es)))
    return COMPACT_ERR_ALIGNMENT;
  if (workspace_bytes < compact_workspace_bytes(L, tokens) || (!workspace && compact_workspace_bytes(L, tokens)))
    return COMPACT_ERR_WORKSPACE;
  if (workspace && !aligned16(workspace)) return COMPACT_ERR_ALIGNMENT;
  if (s != COMPACT_OK) return s;
  if (L->cfg.dtype == COMPACT_BF16) {
    typedef __nv_bfloat16 T;
    if (g_family.load() != 1) {
      tc::LaunchInfo li{g_family.load() == 2 ? 1 : CFG_CS, st, status_word(L), sched_words(L), &g_launches};
      // both products on pairs of SMs (family 2: on single SMs, the cross-check)
      if (g_family.load() == 0)
        s = g2::g2_backward(li, tokens, L->cfg.n, L->cfg.m, L->cfg.r, (int)compact_z_ld(L), (const T*)dY, lddy, (const T*)Z, ldz, (const T*)W,
                            ldw, (T*)dX, lddx, Gc, ldg, accumulate, workspace, workspace_bytes);
      else
        s = tc::backward(li, tokens, L->cfg.n, L->cfg.m, L->cfg.r, (int)compact_z_ld(L), (const T*)dY, lddy, (const T*)Z, ldz, (const T*)W,
                         ldw, (T*)dX, lddx, Gc, ldg, accumulate, workspace, workspace_bytes);
      if (s != COMPACT_ERR_SHAPE) return s;
    }
    return bwd_simt<T>(L, tokens, (const T*)dY, lddy, (const T*)Z, ldz, (const T*)W, ldw, (T*)dX, lddx, Gc, ldg,
                       accumulate, st);
  }
  return bwd_simt<float>(L, tokens, (const float*)dY, lddy, (const float*)Z, ldz, (const float*)W, ldw, (float*)dX,
                         lddx, Gc, ldg, accumulate, st);
}

// ---- groups of layers that share their input ---------------------------------------------------
namespace {
// The fused launches take bf16 layers with one input width, one seed and at most three members;
// anything else (and the SIMT family) runs layer by layer.
bool group_fusable(compact_layer_t* const* Ls, int count) {
  if (count < 1 || count > tc::MAXG || g_family.load() == 1) return false;
  for (int g = 0; g < count; ++g) {
    if (Ls[g]->cfg.dtype != COMPACT_BF16 || Ls[g]->cfg.n != Ls[0]->cfg.n || Ls[g]->cfg.seed != Ls[0]->cfg.seed) return false;
    if (Ls[g]->cfg.n % 8 || Ls[g]->cfg.m % 8) return false;
  }
  return true;
}
}  // namespace

size_t compact_group_workspace_bytes(compact_layer_t* const* layers, int count, int64_t tokens) {
  if (!layers || count < 1 || tokens < 0) return 0;
  size_t fused = 0, single = 0;
  int r[tc::MAXG], m[tc::MAXG];
  for (int g = 0; g < count; ++g) {
    if (!layers[g]) return 0;
    const size_t w = compact_workspace_bytes(layers[g], tokens);
    single = w > single ? w : single;
    if (g < tc::MAXG) { r[g] = layers[g]->cfg.r; m[g] = layers[g]->cfg.m; }
  }
  if (count <= tc::MAXG) fused = tc::group_gc_workspace_bytes(count, r, m, tokens);
  // layer-by-layer fallback: one layer's workspace plus a dX-sized buffer for the partial input gradients
  const size_t fallback = single + (size_t)round_up((int64_t)tokens * layers[0]->cfg.n * (int64_t)elem_size(layers[0]->cfg.dtype), 256);
  size_t need = fused > fallback ? fused : fallback;
  const size_t fwd = compact_group_fwd_workspace_bytes(layers, count);
  need = fwd > need ? fwd : need;
  return (size_t)round_up((int64_t)need, 256);
}

size_t compact_group_fwd_workspace_bytes(compact_layer_t* const* layers, int count) {
  if (!layers || count < 1) return 0;
  size_t sum = 0;
  for (int g = 0; g < count; ++g) {
    if (!layers[g]) return 0;
    sum += compact_fwd_workspace_bytes(layers[g]);
  }
  return sum;
}

compact_status_t compact_group_fwd(compact_layer_t* const* layers, int count, int64_t tokens, const void* X, int64_t ldx,
                                   const void* const* W, const int64_t* ldw, void* const* Y, const int64_t* ldy,
                                   void* const* Z, const int64_t* ldz, uint32_t* epochs_used, void* workspace,
                                   size_t workspace_bytes, void* stream) {
  if (!layers || count < 1 || !W || !ldw || !Y || !ldy || !Z || !ldz) return COMPACT_ERR_INVALID_ARG;
  if (workspace && !aligned16(workspace)) return COMPACT_ERR_ALIGNMENT;
  for (int g = 0; g < count; ++g)
    if (!layers[g] || layers[g]->cfg.n != layers[0]->cfg.n || layers[g]->cfg.dtype != layers[0]->cfg.dtype) return COMPACT_ERR_INVALID_ARG;
  if (!group_fusable(layers, count) || tokens <= 0) {
    for (int g = 0; g < count; ++g) {
      compact_status_t s = compact_linear_fwd(layers[g], tokens, X, ldx, W[g], ldw[g], Y[g], ldy[g], Z[g], ldz[g],
                                              epochs_used ? epochs_used + g : nullptr, workspace, workspace_bytes, stream);
      if (s != COMPACT_OK) return s;
    }
    return COMPACT_OK;
  }
  typedef __nv_bfloat16 T;
  if (tokens > 0x7fffffff || !X) return COMPACT_ERR_INVALID_ARG;
  if (!aligned16(X) || !pitch_ok(ldx, layers[0]->cfg.n, 2)) return COMPACT_ERR_ALIGNMENT;
  tc::GroupLayer gl[tc::MAXG];
  memset(gl, 0, sizeof(gl));
  for (int g = 0; g < count; ++g) {
    compact_layer_t* L = layers[g];
    if (epochs_used) epochs_used[g] = L->epoch;
    if (!W[g] || !Y[g] || !Z[g]) return COMPACT_ERR_INVALID_ARG;
    if (!aligned16(W[g]) || !aligned16(Y[g]) || !aligned16(Z[g])) return COMPACT_ERR_ALIGNMENT;
    if (!pitch_ok(ldw[g], L->cfg.m, 2) || !pitch_ok(ldy[g], L->cfg.m, 2) || !pitch_ok(ldz[g], compact_z_ld(L), 2)) return COMPACT_ERR_ALIGNMENT;
    gl[g].pp = make_pp(L, L->epoch);
    gl[g].m = L->cfg.m; gl[g].r = L->cfg.r; gl[g].zcols = (int)compact_z_ld(L);
    gl[g].W = (const T*)W[g]; gl[g].ldw = ldw[g];
    gl[g].Y = (T*)Y[g]; gl[g].ldy = ldy[g];
    gl[g].Z = (T*)Z[g]; gl[g].ldz = ldz[g];
  }
  compact_status_t s = check_device(layers[0], stream);
  if (s != COMPACT_OK) return s;
  tc::LaunchInfo li{g_family.load() == 2 ? 1 : CFG_CS, (cudaStream_t)stream, status_word(layers[0]), sched_words(layers[0]), &g_launches};
  if (g_family.load() == 0 && workspace && workspace_bytes >= compact_group_fwd_workspace_bytes(layers, count)) {
    g2::G2Layer g2l[tc::MAXG];
    for (int g = 0; g < count; ++g) {
      g2l[g].pp = gl[g].pp; g2l[g].m = gl[g].m; g2l[g].zcols = gl[g].zcols;
      g2l[g].W = gl[g].W; g2l[g].ldw = gl[g].ldw; g2l[g].Y = gl[g].Y; g2l[g].ldy = gl[g].ldy; g2l[g].Z = gl[g].Z; g2l[g].ldz = gl[g].ldz;
    }
    s = g2::g2_forward(li, count, g2l, tokens, layers[0]->cfg.n, (const T*)X, ldx, workspace);
    if (s != COMPACT_ERR_SHAPE) return s;
  }
  return tc::forward_group(li, count, gl, tokens, layers[0]->cfg.n, (const T*)X, ldx);
}

compact_status_t compact_group_bwd(compact_layer_t* const* layers, int count, int64_t tokens, const void* const* dY,
                                   const int64_t* lddy, const void* const* Z, const int64_t* ldz, const void* const* W,
                                   const int64_t* ldw, void* dX, int64_t lddx, float* const* Gc, const int64_t* ldg,
                                   int accumulate, void* workspace, size_t workspace_bytes, void* stream) {
  if (!layers || count < 1 || !dY || !lddy || !Z || !ldz || !W || !ldw || !Gc || !ldg) return COMPACT_ERR_INVALID_ARG;
  for (int g = 0; g < count; ++g)
    if (!layers[g] || layers[g]->cfg.n != layers[0]->cfg.n || layers[g]->cfg.dtype != layers[0]->cfg.dtype) return COMPACT_ERR_INVALID_ARG;
  if (workspace_bytes < compact_group_workspace_bytes(layers, count, tokens) || !workspace) return COMPACT_ERR_WORKSPACE;
  if (!aligned16(workspace)) return COMPACT_ERR_ALIGNMENT;
  const int n = layers[0]->cfg.n;
  if (!group_fusable(layers, count) || tokens <= 0) {
    // layer by layer: the first layer writes dX, the others write their share into scratch and it is added
    const size_t es = elem_size(layers[0]->cfg.dtype);
    size_t single = 0;
    for (int g = 0; g < count; ++g) {
      const size_t w = compact_workspace_bytes(layers[g], tokens);
      single = w > single ? w : single;
    }
    void* part = (char*)workspace + single;
    for (int g = 0; g < count; ++g) {
      void* dst = (dX && g > 0) ? part : dX;
      compact_status_t s = compact_linear_bwd(layers[g], tokens, dY[g], lddy[g], Z[g], ldz[g], W[g], ldw[g], dst,
                                              dst == dX ? lddx : n, Gc[g], ldg[g], accumulate, workspace, single, stream);
      if (s != COMPACT_OK) return s;
      if (dX && g > 0 && tokens > 0) {
        s = es == 2 ? add_rows<__nv_bfloat16>((__nv_bfloat16*)dX, lddx, (const __nv_bfloat16*)part, n, tokens, n, (cudaStream_t)stream)
                    : add_rows<float>((float*)dX, lddx, (const float*)part, n, tokens, n, (cudaStream_t)stream);
        if (s != COMPACT_OK) return s;
      }
    }
    return COMPACT_OK;
  }
  typedef __nv_bfloat16 T;
  if (tokens > 0x7fffffff) return COMPACT_ERR_INVALID_ARG;
  if (dX && (!aligned16(dX) || !pitch_ok(lddx, n, 2))) return COMPACT_ERR_ALIGNMENT;
  tc::GroupLayer gl[tc::MAXG];
  memset(gl, 0, sizeof(gl));
  for (int g = 0; g < count; ++g) {
    compact_layer_t* L = layers[g];
    if (!dY[g] || !Z[g] || !W[g] || !Gc[g]) return COMPACT_ERR_INVALID_ARG;
    if (!aligned16(dY[g]) || !aligned16(Z[g]) || !aligned16(W[g]) || !aligned16(Gc[g])) return COMPACT_ERR_ALIGNMENT;
    if (!pitch_ok(lddy[g], L->cfg.m, 2) || !pitch_ok(ldz[g], compact_z_ld(L), 2) || !pitch_ok(ldw[g], L->cfg.m, 2) ||
        !pitch_ok(ldg[g], L->cfg.m, 4))
      return COMPACT_ERR_ALIGNMENT;
    gl[g].m = L->cfg.m; gl[g].r = L->cfg.r; gl[g].zcols = (int)compact_z_ld(L);
    gl[g].W = (const T*)W[g]; gl[g].ldw = ldw[g];
    gl[g].Z = (T*)const_cast<void*>(Z[g]); gl[g].ldz = ldz[g];
    gl[g].dY = (const T*)dY[g]; gl[g].lddy = lddy[g];
    gl[g].Gc = Gc[g]; gl[g].ldg = ldg[g];
  }
  compact_status_t s = check_device(layers[0], stream);
  if (s != COMPACT_OK) return s;
  tc::LaunchInfo li{1, (cudaStream_t)stream, status_word(layers[0]), sched_words(layers[0]), &g_launches};
  // on pairs of SMs (family 2: on single SMs, the cross-check); same bits
  if (g_family.load() == 0) {
    s = g2::g2_backward_group(li, count, gl, tokens, n, (T*)dX, lddx, accumulate, workspace, workspace_bytes);
    if (s != COMPACT_ERR_SHAPE) return s;
  }
  return tc::backward_group(li, count, gl, tokens, n, (T*)dX, lddx, accumulate, workspace, workspace_bytes);
}

size_t compact_recompute_workspace_bytes(const compact_layer_t* layer, int64_t tokens) {
  if (!layer || tokens < 0) return 0;
  return (size_t)round_up((int64_t)compact_saved_bytes(layer, tokens), 256) + compact_workspace_bytes(layer, tokens);
}

compact_status_t compact_linear_bwd_recompute(compact_layer_t* L, int64_t tokens, const void* X, int64_t ldx,
                                              uint32_t epoch_of_fwd, const void* dY, int64_t lddy, const void* W,
                                              int64_t ldw, void* dX, int64_t lddx, float* Gc, int64_t ldg, int accumulate,
                                              void* workspace, size_t workspace_bytes, void* stream) {
  if (!L || tokens < 0 || tokens > 0x7fffffff) return COMPACT_ERR_INVALID_ARG;
  if (epoch_of_fwd != L->epoch) return COMPACT_ERR_EPOCH_MISMATCH;
  const int64_t ldz = compact_z_ld(L);
  const size_t zbytes = (size_t)round_up((int64_t)compact_saved_bytes(L, tokens), 256);
  if (tokens > 0) {
    if (!X) return COMPACT_ERR_INVALID_ARG;
    const size_t es = elem_size(L->cfg.dtype);
    if (!aligned16(X) || !pitch_ok(ldx, L->cfg.n, es)) return COMPACT_ERR_ALIGNMENT;
    if (!workspace || workspace_bytes < compact_recompute_workspace_bytes(L, tokens)) return COMPACT_ERR_WORKSPACE;
    if (!aligned16(workspace)) return COMPACT_ERR_ALIGNMENT;
    compact_status_t s = check_device(L, stream);
    if (s != COMPACT_OK) return s;
    cudaStream_t st = (cudaStream_t)stream;
    // Z = X P again, into the front of the workspace
    if (L->cfg.dtype == COMPACT_BF16) {
      typedef __nv_bfloat16 T;
      s = COMPACT_ERR_SHAPE;
      if (g_family.load() != 1) {
        tc::LaunchInfo li{g_family.load() == 2 ? 1 : CFG_CS, st, status_word(L), sched_words(L), &g_launches};
        // P goes, for the duration of this product, where the backward will put its partials afterwards
        if (g_family.load() == 0 && workspace_bytes - zbytes >= compact_fwd_workspace_bytes(L))
          s = g2::g2_project(li, make_pp(L, L->epoch), tokens, (const T*)X, ldx, (T*)workspace, ldz, (int)ldz, (char*)workspace + zbytes);
        if (s == COMPACT_ERR_SHAPE)
          s = tc::forward(li, make_pp(L, L->epoch), tokens, L->cfg.m, (const T*)X, ldx, nullptr, 0, nullptr, 0, (T*)workspace, ldz,
                          (int)ldz);
      }
      if (s == COMPACT_ERR_SHAPE)
        s = fwd_simt<T>(L, tokens, (const T*)X, ldx, nullptr, 0, nullptr, 0, (T*)workspace, ldz, st);
    } else {
      s = fwd_simt<float>(L, tokens, (const float*)X, ldx, nullptr, 0, nullptr, 0, (float*)workspace, ldz, st);
    }
    if (s != COMPACT_OK) return s;
  }
  return compact_linear_bwd(L, tokens, dY, lddy, workspace, ldz, W, ldw, dX, lddx, Gc, ldg, accumulate,
                            tokens > 0 ? (char*)workspace + zbytes : workspace,
                            tokens > 0 ? workspace_bytes - zbytes : workspace_bytes, stream);
}

compact_status_t compact_adam_update(compact_layer_t* L, void* W, int64_t ldw, const float* Gc, int64_t ldg, float* M,
                                     float* V, uint32_t epoch_of_Gc, float lr, void* workspace, size_t workspace_bytes,
                                     void* stream) {
  if (!L || !W || !Gc || !M || !V) return COMPACT_ERR_INVALID_ARG;
  if (epoch_of_Gc != L->epoch) return COMPACT_ERR_EPOCH_MISMATCH;
  const size_t es = elem_size(L->cfg.dtype);
  if (!aligned16(W) || !aligned16(Gc) || !aligned16(M) || !aligned16(V)) return COMPACT_ERR_ALIGNMENT;
  if (!pitch_ok(ldw, L->cfg.m, es) || !pitch_ok(ldg, L->cfg.m, 4)) return COMPACT_ERR_ALIGNMENT;
  if (!workspace || workspace_bytes < update_min_bytes(L)) return COMPACT_ERR_WORKSPACE;
  if (!aligned16(workspace)) return COMPACT_ERR_ALIGNMENT;
  compact_status_t s = check_device(L, stream);
  if (s != COMPACT_OK) return s;
  if (isnan(lr)) lr = L->cfg.lr;
  cudaStream_t st = (cudaStream_t)stream;
  if (L->cfg.dtype == COMPACT_BF16) {
    typedef __nv_bfloat16 T;
    s = COMPACT_ERR_SHAPE;
    if (g_family.load() != 1) {
      tc::LaunchInfo li{g_family.load() == 2 ? 1 : CFG_CS, st, status_word(L), sched_words(L), &g_launches};
      // Two routes with the same bits.  With room for P next to N: the Adam kernel, P written out, and the product on
      // pairs of SMs.  Without: the Adam kernel followed by the streaming GEMM that regenerates P tile by tile.
      // (the tiles of a sparse projection hold integer counts: its 1/sqrt(s) rides on the step size)
      const ProjectionParams pp = make_pp(L, L->epoch);
      const float step_scale = lr * L->cfg.alpha * pp.inv_sqrt_s;
      if (g_family.load() == 0 &&
          workspace_bytes >= g2::g2_update_scratch_bytes(L->cfg.n, L->cfg.m, L->cfg.r, (int)compact_z_ld(L)))
        s = g2::g2_update(li, pp, adam_scalars(L, L->step + 1), L->cfg.n, L->cfg.m, L->cfg.r, (int)compact_z_ld(L), (T*)W, ldw,
                          Gc, ldg, M, V, step_scale, workspace, workspace_bytes);
      else
        s = tc::update(li, pp, adam_scalars(L, L->step + 1), L->cfg.n, L->cfg.m, L->cfg.r, (T*)W, ldw,
                       Gc, ldg, M, V, step_scale, workspace, workspace_bytes);
    }
    if (s == COMPACT_ERR_SHAPE) s = update_simt<T>(L, (T*)W, ldw, Gc, ldg, M, V, lr, (float*)workspace, st);
  } else {
    s = update_simt<float>(L, (float*)W, ldw, Gc, ldg, M, V, lr, (float*)workspace, st);
  }
  if (s == COMPACT_OK) L->step += 1;
  return s;
}

// ---- allocation-free update -------------------------------------------------------------
// Scratch for callers that cannot hand over device memory: part of the library image, so
// every GPU that loads the library carries it until the process ends.  In host code the
// array's name is only a handle; the device address comes from cudaGetSymbolAddress, asked
// once per device with that device current.
static __device__ __align__(256) unsigned char g_noalloc_scratch[COMPACT_NOALLOC_SCRATCH_BYTES];

namespace {
std::atomic<void*> g_noalloc_ptr[kMaxDevices];

// Device address of the scratch array on the current device (looked up on first use).
compact_status_t noalloc_scratch(void** out) {
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess) { cudaGetLastError(); return COMPACT_ERR_CUDA; }
  if (dev < 0 || dev >= kMaxDevices) return COMPACT_ERR_INVALID_ARG;
  void* p = g_noalloc_ptr[dev].load(std::memory_order_acquire);
  if (!p) {
    if (cudaGetSymbolAddress(&p, g_noalloc_scratch) != cudaSuccess || !p) { cudaGetLastError(); return COMPACT_ERR_CUDA; }
    g_noalloc_ptr[dev].store(p, std::memory_order_release);
  }
  *out = p;
  return COMPACT_OK;
}
}  // namespace

compact_status_t compact_adam_update_noalloc(compact_layer_t* L, void* W, int64_t ldw, const float* Gc, int64_t ldg,
                                             float* M, float* V, uint32_t epoch_of_Gc, float lr, void* stream) {
  if (!L) return COMPACT_ERR_INVALID_ARG;
  // the update needs r x m scratch entries (fp32 in the plain kernels, bf16 in the tensor-core ones)
  if (update_min_bytes(L) > (size_t)COMPACT_NOALLOC_SCRATCH_BYTES) return COMPACT_ERR_SCRATCH_LIMIT;
  compact_status_t s = check_device(L, stream);
  if (s != COMPACT_OK) return s;
  void* scratch = nullptr;
  s = noalloc_scratch(&scratch);
  if (s != COMPACT_OK) return s;
  return compact_adam_update(L, W, ldw, Gc, ldg, M, V, epoch_of_Gc, lr, scratch, (size_t)COMPACT_NOALLOC_SCRATCH_BYTES, stream);
}

compact_status_t compact_refresh_projection(compact_layer_t* L, int force, uint32_t* new_epoch) {
  if (!L) return COMPACT_ERR_INVALID_ARG;
  const uint32_t T = L->cfg.refresh_T;
  if (force) {
    L->epoch += 1;
  } else if (T > 0 && L->step > 0 && L->step % T == 0 && L->last_refresh_step != L->step) {
    L->epoch += 1;
    L->last_refresh_step = L->step;
  }
  if (new_epoch) *new_epoch = L->epoch;
  return COMPACT_OK;
}

compact_status_t compact_layer_get_state(const compact_layer_t* L, compact_layer_state_t* out) {
  if (!L || !out) return COMPACT_ERR_INVALID_ARG;
  out->seed = L->cfg.seed;
  out->layer_id = L->cfg.layer_id;
  out->epoch = L->epoch;
  out->step = L->step;
  return COMPACT_OK;
}

compact_status_t compact_layer_set_state(compact_layer_t* L, const compact_layer_state_t* in) {
  if (!L || !in) return COMPACT_ERR_INVALID_ARG;
  L->cfg.seed = in->seed;
  L->cfg.layer_id = in->layer_id;
  L->epoch = in->epoch;
  L->step = in->step;
  // A restored step that is a multiple of T has already been refreshed at if
  // the restored epoch accounts for it; the caller restores what get_state gave.
  const uint32_t T = L->cfg.refresh_T;
  L->last_refresh_step = (T > 0 && in->step > 0 && in->step % T == 0 && in->epoch >= in->step / T) ? in->step : 0;
  return COMPACT_OK;
}

compact_status_t compact_layer_status(compact_layer_t* L) {
  if (!L) return COMPACT_ERR_INVALID_ARG;
  if (L->device_checked == 0) return COMPACT_OK;      // nothing has been launched for this layer yet
  if (L->device_checked < 0) return COMPACT_ERR_UNSUPPORTED_ARCH;
  unsigned int* w = status_word(L);
  if (!w) return COMPACT_ERR_CUDA;
  unsigned int v = 0;
  if (cudaDeviceSynchronize() != cudaSuccess) { cudaGetLastError(); return COMPACT_ERR_CUDA; }
  if (cudaMemcpy(&v, w, 4, cudaMemcpyDeviceToHost) != cudaSuccess) { cudaGetLastError(); return COMPACT_ERR_CUDA; }
  if (v) {
    unsigned int z = 0;
    cudaMemcpy(w, &z, 4, cudaMemcpyHostToDevice);
    return COMPACT_ERR_DEVICE_TIMEOUT;
  }
  return COMPACT_OK;
}

compact_status_t compact_debug_wait_that_runs_out(compact_layer_t* L, void* stream) {
  if (!L) return COMPACT_ERR_INVALID_ARG;
  compact_status_t s = check_device(L, stream);
  if (s != COMPACT_OK) return s;
  unsigned int* w = status_word(L);
  if (!w) return COMPACT_ERR_CUDA;
  tc::wait_that_runs_out_kernel<<<1, 64, 0, (cudaStream_t)stream>>>(w, 4096u);
  g_launches++;
  return launch_result();
}

compact_status_t compact_debug_philox_u32(uint64_t seed, uint32_t layer_id, uint32_t epoch, int32_t n, int32_t r,
                                          uint32_t* out_dev, void* stream) {
  if (n < 1 || r < 1 || !out_dev) return COMPACT_ERR_INVALID_ARG;
  if (!aligned16(out_dev)) return COMPACT_ERR_ALIGNMENT;
  const int groups = (r + 7) / 8;
  const int64_t cnt = (int64_t)n * groups;
  debug_philox_words_kernel<<<(unsigned)((cnt + 255) / 256), 256, 0, (cudaStream_t)stream>>>(
      make_philox_key(seed), layer_id, epoch, n, groups, out_dev);
  g_launches++;
  return launch_result();
}

compact_status_t compact_debug_philox_layer_u32(uint64_t seed, uint32_t layer_id, uint32_t epoch, int32_t n, int32_t r,
                                                uint32_t* out_dev, void* stream) {
  if (n < 1 || r < 1 || !out_dev) return COMPACT_ERR_INVALID_ARG;
  if (!aligned16(out_dev)) return COMPACT_ERR_ALIGNMENT;
  const int groups = (r + 7) / 8;
  const int64_t cnt = (int64_t)n * groups;
  const uint64_t pl = (uint64_t)0xCD9E8D57u * (uint64_t)layer_id;
  debug_philox_layer_words_kernel<<<(unsigned)((cnt + 255) / 256), 256, 0, (cudaStream_t)stream>>>(
      make_philox_key(seed), (uint32_t)(pl >> 32), (uint32_t)pl, epoch, n, groups, out_dev);
  g_launches++;
  return launch_result();
}

compact_status_t compact_debug_sparse_terms(const compact_layer_t* L, uint32_t epoch, uint32_t* out_dev, void* stream) {
  if (!L || !out_dev || L->cfg.sparse_s <= 0) return COMPACT_ERR_INVALID_ARG;
  const ProjectionParams pp = make_pp(L, epoch);
  const int64_t cnt = (int64_t)pp.n * pp.sparse_s;
  debug_sparse_terms_kernel<<<(unsigned)((cnt + 255) / 256), 256, 0, (cudaStream_t)stream>>>(pp, out_dev);
  g_launches++;
  return launch_result();
}

compact_status_t compact_debug_projection(const compact_layer_t* L, uint32_t epoch, void* P_dev, void* stream) {
  if (!L || !P_dev) return COMPACT_ERR_INVALID_ARG;
  const ProjectionParams pp = make_pp(L, epoch);
  const int64_t cnt = (int64_t)pp.n * pp.r;
  const unsigned blocks = (unsigned)((cnt + 255) / 256);
  if (L->cfg.dtype == COMPACT_BF16)
    debug_projection_kernel<__nv_bfloat16><<<blocks, 256, 0, (cudaStream_t)stream>>>(pp, (__nv_bfloat16*)P_dev);
  else
    debug_projection_kernel<float><<<blocks, 256, 0, (cudaStream_t)stream>>>(pp, (float*)P_dev);
  g_launches++;
  return launch_result();
}

int compact_set_kernel_family(int family) {
  if (family < 0 || family > 2) return g_family.load();
  return g_family.exchange(family);
}

uint64_t compact_kernel_launch_count(void) { return g_launches.load(); }

const char* compact_status_string(compact_status_t s) {
  switch (s) {
    case COMPACT_OK: return "ok";
    case COMPACT_ERR_INVALID_ARG: return "invalid argument";
    case COMPACT_ERR_SHAPE: return "unsupported shape";
    case COMPACT_ERR_ALIGNMENT: return "pointer or pitch not 16-byte aligned";
    case COMPACT_ERR_DTYPE: return "unsupported dtype";
    case COMPACT_ERR_EPOCH_MISMATCH: return "gradient was produced under another projection epoch";
    case COMPACT_ERR_WORKSPACE: return "workspace missing or too small";
    case COMPACT_ERR_UNSUPPORTED_ARCH: return "device is not compute capability 10.x";
    case COMPACT_ERR_CUDA: return "CUDA runtime error";
    case COMPACT_ERR_DEVICE_TIMEOUT: return "a kernel gave up on a bounded wait";
    case COMPACT_ERR_TOO_MANY_LAYERS: return "too many live layers (4096 status slots); destroy some first";
    case COMPACT_ERR_SCRATCH_LIMIT: return "layer needs more scratch than the allocation-free entry point carries (r*m*4 > 32 MiB)";
  }
  return "unknown status";
}

}  // extern "C"
