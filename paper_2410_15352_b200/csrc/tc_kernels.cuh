// Tensor-core kernels of the CompAct layer for sm_100a: one persistent,
// warp-specialised GEMM (TMA -> 128B-swizzled shared memory rings -> tcgen05.mma
// with fp32 accumulators in TMEM -> tcgen05.ld -> swizzled staging -> TMA store)
// whose operands come from TMA in either major-ness or from the in-kernel
// Philox/Box-Muller generator of P.  It serves
//   forward  : [Y | Z] = X [W | P]        (Algorithm 1; Z computed as Z^T = P^T X^T, P tiles generated as A)
//   backward : dX = dY W^T and Gc = Z^T dY (Algorithm 2; Gc split over tokens)
//   update   : W <- W - eta alpha P N      (Algorithm 3 lines 6-9; P tiles generated as A)
// These are the products with P generated on chip: the route of calls that bring no scratch for P, of the
// cross-check family, and the home of the helpers (barriers, TMA, descriptors, tensor maps) that the pair-of-SMs
// kernel in gemm2_kernel.cuh shares.  Calls with scratch write P out once and run every product there.
// Launches with a generated operand run as clusters of two CTAs that share every generated tile.
// Work items are numbered longest first; those with a generated operand are dealt statically to the
// clusters, the rest come from one atomic counter per launch.
#pragma once
#include <cuda.h>
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

#include <atomic>
#include <unordered_map>

#include "../../include/compact.h"
#include "philox.cuh"
#include "simt_kernels.cuh"

namespace compact {
namespace tc {

struct LaunchInfo {
  int cluster;            // CTAs that share each generated tile of P (1 or 2)
  cudaStream_t stream;
  unsigned int* status;   // device word: kernels OR error bits into it
  unsigned int* sched;    // two device words, zero between launches: next item, finished CTAs
  std::atomic<uint64_t>* launches;
};

constexpr int BM = 128;              // rows of one accumulator (TMEM lanes)
constexpr int BK = 64;               // K elements per pipeline stage (one 128-byte swizzle row)
constexpr int BN_MAX = 256;          // columns of one accumulator slot (TMEM has two slots)
constexpr int A_BYTES = BM * BK * 2;
constexpr int B_BYTES = BN_MAX * BK * 2;
// One pipeline stage holds a B tile and two A tiles under ONE full/empty barrier pair: every
// mbarrier operation of the MMA-issuing thread costs ~150 clocks of its serial time, so a stage
// carries as many MMAs (8) as fit.
//
// The ring memory is cut in one of two ways, chosen per problem:
//   geometry 0: three stages of [B | A0 | A1] (64 KB) for items with two row blocks per stage;
//   geometry 1: four stages of [B | A0] (48 KB) for items with one row block, whose k-steps take two
//               stages when they have two column blocks -- the fourth stage gives them two whole
//               k-steps of look-ahead, which the latency of a generated tile needs.
// Each geometry has its own barriers.  A CTA meets the problems of a launch in order, so it changes
// geometry at most once; the roles that write into the ring first wait until the old ring has drained.
constexpr int STAGE_B_OFF = 0, STAGE_A0_OFF = B_BYTES, STAGE_A1_OFF = B_BYTES + A_BYTES;
constexpr int NS0 = 3, STAGE0_BYTES = B_BYTES + 2 * A_BYTES;
constexpr int NS1 = 4, STAGE1_BYTES = B_BYTES + A_BYTES;
constexpr int RING_BYTES = NS0 * STAGE0_BYTES;
static_assert(NS1 * STAGE1_BYTES <= RING_BYTES, "both geometries share the ring memory");
static_assert(NS1 % 2 == 0, "two-stage k-steps of generated items must keep each stage's role");
constexpr int NUM_RING_BARS = 2 * (NS0 + NS1);
constexpr int STAGING_BYTES = 4096;      // one staged tile: 32 rows x 128 bytes
constexpr int STAGING_BUFS = 1;          // staged tiles per epilogue warp
constexpr int QDEPTH = 4;                // work items the scheduler may run ahead
constexpr int NUM_EPI_WARPS = 8;         // two sets of four (one per TMEM lane quarter); each set drains one accumulator slot
constexpr int NUM_GEN_WARPS = 16;
constexpr int LOADER_WARP = 2 + NUM_EPI_WARPS;      // loads the A tiles
constexpr int MMA1_WARP = 3 + NUM_EPI_WARPS;        // second MMA issuer
constexpr int THREADS_BASE = 32 * (4 + NUM_EPI_WARPS);   // owner/scheduler, two MMA issuers, epilogue, loader
constexpr int THREADS_GEN = THREADS_BASE + 32 * NUM_GEN_WARPS;
constexpr int NUM_BARRIERS = NUM_RING_BARS + 4 + 2 * QDEPTH + NUM_EPI_WARPS * STAGING_BUFS;
constexpr int TAIL_BYTES = 8 * NUM_BARRIERS + 4 * QDEPTH + 16;
constexpr int SMEM_BYTES = 1024 + RING_BYTES + NUM_EPI_WARPS * STAGING_BUFS * STAGING_BYTES + ((TAIL_BYTES + 127) / 128) * 128;
constexpr int NUM_SMS = 148;
static_assert(SMEM_BYTES <= 232448, "shared memory budget");

// Generated operands are always the A operand.  GENERATED: the tile's M index runs over rows of P and its K
// index over columns of P, written K-major (the update).  GENERATED_T: the M index runs over columns of P
// and the K index over its rows, written MN-major -- the operand of Z^T = P^T X^T (the forward).
enum OperandMode { TMA_KMAJOR = 0, TMA_MNMAJOR = 1, GENERATED = 2, GENERATED_T = 3 };
// EPI_BF16_T stores the transpose of the accumulator (lanes become columns of the output).
enum EpiMode { EPI_BF16 = 0, EPI_F32 = 1, EPI_UPDATE_W = 2, EPI_BF16_T = 3 };
enum GenRing { GEN_NONE = 0, GEN_A = 1 };

constexpr unsigned int STATUS_TIMEOUT = 1u;

// One GEMM inside a launch.  An item is nsub row blocks (sharing each B tile) by ncol column
// blocks of bn columns (sharing each A tile; ncol > 1 only with nsub == 1); its accumulators sit
// side by side in TMEM (nsub * ncol * bn <= 512 columns).
struct Problem {
  int M, N, K;
  int tiles_m, tiles_n, splits, ksteps_total, ksteps_per_split;
  int bn;
  int nsub;
  int ncol;
  int a_mode, b_mode, epi_mode;
  int geo;                // ring geometry its items use (0 or 1)
  int a_blocked, b_blocked;   // MN-major operand read through a map that brings a whole tile in one copy
  int map_base;           // its tensor maps: C at map_base, A and B of K segment s at map_base + s
  // the projection a generated operand is a tile of; the Philox key (the seed) is the launch's
  uint32_t pp_layer_hi, pp_layer_lo, pp_epoch;
  int pp_n, pp_r;
  int pp_sparse_s;        // > 0: the generated operand is the sparse projection, as integer counts (scaled in the epilogue)
  float pp_scale;         // -2 ln 2 / r
  // K may run over up to three segments with operands of their own (dX of a group of layers that share
  // their input is the sum over the layers of dY_g W_g^T): segment s covers k-steps seg_begin[s] .. seg_begin[s+1]
  int nseg;
  int seg_begin[4];
  int group_begin;        // generated problems: number of cluster groups before this problem's
  int tile_begin;
  float scale;
};

constexpr int MAXP = 6;     // problems (and tensor-map triples) per launch
constexpr int MAXG = 3;     // layers in a group that shares its input

struct alignas(64) Params {
  CUtensorMap tmA[MAXP];
  CUtensorMap tmB[MAXP];
  CUtensorMap tmC[MAXP];  // output tiles of the epilogue
  Problem prob[MAXP];
  int num_problems;
  int num_gen;            // problems with a generated operand: the first num_gen of the launch
  int total_tiles;
  int gen_ring;
  // Cluster-shared generation: the `cs` CTAs of a cluster take items that need the same tiles of P
  // (same columns of P, different tokens in the forward; same rows of P, different columns of W in
  // the update), each generates 1/cs of every tile and writes it into all cs shared memories.
  int cs;                 // CTAs per cluster (1: every CTA generates for itself)
  int share_n;            // 0: the cs items of a group are neighbours along M, 1: along N
  int gen_groups;         // groups of cs generated items; handed out statically, cluster by cluster
  int dyn_begin;          // first item handed out dynamically (0 when cs == 1)
  PhiloxKey key;          // round keys of the seed shared by the launch's generated problems
  unsigned int* status;
  unsigned int* sched;
};

// --------------------------------------------------------------------------------------
// PTX wrappers
// --------------------------------------------------------------------------------------
__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count));
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void mbar_arrive_n(uint32_t bar, uint32_t count) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes) {
  asm volatile("mbarrier.expect_tx.relaxed.cta.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ void mbar_arrive_expect_tx(uint32_t bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(ok)
      : "r"(bar), "r"(parity)
      : "memory");
  return ok != 0;
}
// Bounded wait: gives up after about a second, records it, and lets the CTA drain.
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, volatile int* abort_flag, unsigned int* status,
                                          uint32_t limit = 8000000u) {
  if (mbar_try_wait(bar, parity)) return true;
  for (uint32_t it = 0; it < limit; ++it) {
    if (mbar_try_wait(bar, parity)) return true;
    if (it > 128) {
      __nanosleep(100);
      if (*abort_flag) return false;
    }
  }
  *abort_flag = 1;
  atomicOr(status, STATUS_TIMEOUT);
  return false;
}

__device__ __forceinline__ void fence_barrier_init() { asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory"); }
__device__ __forceinline__ void fence_proxy_async_smem() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }

__device__ __forceinline__ void tma_load_2d(uint32_t dst, const CUtensorMap* map, uint32_t bar, int x, int y) {
  asm volatile(
      "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4}], [%2];" ::"r"(dst),
      "l"(map), "r"(bar), "r"(x), "r"(y)
      : "memory");
}
__device__ __forceinline__ void tma_load_3d(uint32_t dst, const CUtensorMap* map, uint32_t bar, int x, int y, int z) {
  asm volatile(
      "cp.async.bulk.tensor.3d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5}], [%2];" ::"r"(dst),
      "l"(map), "r"(bar), "r"(x), "r"(y), "r"(z)
      : "memory");
}
__device__ __forceinline__ void tma_store_2d(const CUtensorMap* map, uint32_t src, int x, int y) {
  asm volatile("cp.async.bulk.tensor.2d.global.shared::cta.bulk_group [%0, {%2, %3}], [%1];" ::"l"(map), "r"(src), "r"(x),
               "r"(y)
               : "memory");
}
// global tile += shared tile, element-wise in the tensor map's type (bf16), done by the TMA unit at the L2
__device__ __forceinline__ void tma_reduce_add_2d(const CUtensorMap* map, uint32_t src, int x, int y) {
  asm volatile("cp.reduce.async.bulk.tensor.2d.global.shared::cta.add.tile.bulk_group [%0, {%2, %3}], [%1];" ::"l"(map),
               "r"(src), "r"(x), "r"(y)
               : "memory");
}
__device__ __forceinline__ void tma_store_3d(const CUtensorMap* map, uint32_t src, int x, int y, int z) {
  asm volatile("cp.async.bulk.tensor.3d.global.shared::cta.bulk_group [%0, {%2, %3, %4}], [%1];" ::"l"(map), "r"(src),
               "r"(x), "r"(y), "r"(z)
               : "memory");
}
// asks the L2 for a tile without bringing it into the SM
__device__ __forceinline__ void tma_prefetch_2d(const CUtensorMap* map, int x, int y) {
  asm volatile("cp.async.bulk.prefetch.tensor.2d.L2.global.tile [%0, {%1, %2}];" ::"l"(map), "r"(x), "r"(y) : "memory");
}
__device__ __forceinline__ void tma_store_commit() { asm volatile("cp.async.bulk.commit_group;" ::: "memory"); }
__device__ __forceinline__ void tma_store_wait_read() { asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory"); }
__device__ __forceinline__ void tma_store_wait_all() { asm volatile("cp.async.bulk.wait_group 0;" ::: "memory"); }

__device__ __forceinline__ void tmem_alloc(uint32_t dst_smem, uint32_t ncols) {
  asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(dst_smem), "r"(ncols) : "memory");
}
__device__ __forceinline__ void tmem_relinquish() {
  asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_dealloc(uint32_t taddr, uint32_t ncols) {
  asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(taddr), "r"(ncols) : "memory");
}
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }

// Descriptors travel as (lo, hi) 32-bit halves so that stepping along K is one 32-bit add.
__device__ __forceinline__ void umma_bf16(uint32_t d_tmem, uint32_t a_lo, uint32_t a_hi, uint32_t b_lo, uint32_t b_hi,
                                          uint32_t idesc, uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t.reg .b64 da, db;\n\t"
      "mov.b64 da, {%1, %2};\n\t"
      "mov.b64 db, {%3, %4};\n\t"
      "setp.ne.b32 p, %6, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], da, db, %5, p;\n\t}" ::"r"(d_tmem),
      "r"(a_lo), "r"(a_hi), "r"(b_lo), "r"(b_hi), "r"(idesc), "r"(accumulate)
      : "memory");
}
__device__ __forceinline__ void umma_commit(uint32_t bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}

// Commit that arrives on the barrier at the same offset in every CTA of `mask`.
__device__ __forceinline__ void umma_commit_mc(uint32_t bar, uint16_t mask) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.multicast::cluster.b64 [%0], %1;" ::"r"(bar),
               "h"(mask)
               : "memory");
}
__device__ __forceinline__ uint32_t cluster_ctarank() {
  uint32_t r;
  asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
  return r;
}
__device__ __forceinline__ void cluster_sync_all() {
  asm volatile("barrier.cluster.arrive.release.aligned;\n\tbarrier.cluster.wait.acquire.aligned;" ::: "memory");
}
// Address of the same shared-memory location in CTA `rank` of the cluster.
__device__ __forceinline__ uint32_t map_to_cta(uint32_t addr, uint32_t rank) {
  uint32_t r;
  asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(addr), "r"(rank));
  return r;
}
// 16-byte store into another CTA's shared memory; its bytes complete on that CTA's barrier `rbar`.
__device__ __forceinline__ void st_async_16(uint32_t raddr, uint4 v, uint32_t rbar) {
  asm volatile("st.async.weak.shared::cluster.mbarrier::complete_tx::bytes.v4.b32 [%0], {%1, %2, %3, %4}, [%5];" ::"r"(raddr),
               "r"(v.x), "r"(v.y), "r"(v.z), "r"(v.w), "r"(rbar)
               : "memory");
}

// Barrier among `threads` threads of the CTA (a multiple of 32), by number; 0 is __syncthreads'.
__device__ __forceinline__ void named_barrier(int id, int threads) {
  asm volatile("bar.sync %0, %1;" ::"r"(id), "r"(threads) : "memory");
}

// True in exactly one lane of a converged warp.
__device__ __forceinline__ bool elect_one() {
  uint32_t pred;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "elect.sync _|p, 0xffffffff;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(pred));
  return pred != 0;
}

__device__ __forceinline__ void tmem_ld32(uint32_t taddr, uint32_t (&v)[32]) {
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
      "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
      "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
      : "=r"(v[0]), "=r"(v[1]), "=r"(v[2]), "=r"(v[3]), "=r"(v[4]), "=r"(v[5]), "=r"(v[6]), "=r"(v[7]), "=r"(v[8]),
        "=r"(v[9]), "=r"(v[10]), "=r"(v[11]), "=r"(v[12]), "=r"(v[13]), "=r"(v[14]), "=r"(v[15]), "=r"(v[16]),
        "=r"(v[17]), "=r"(v[18]), "=r"(v[19]), "=r"(v[20]), "=r"(v[21]), "=r"(v[22]), "=r"(v[23]), "=r"(v[24]),
        "=r"(v[25]), "=r"(v[26]), "=r"(v[27]), "=r"(v[28]), "=r"(v[29]), "=r"(v[30]), "=r"(v[31])
      : "r"(taddr)
      : "memory");
}
__device__ __forceinline__ void tmem_ld_wait() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }

// Shared-memory matrix descriptor (64 bits), 128-byte swizzle, 8-row groups 1024 bytes apart:
//   lo: start address >> 4 in bits [0,14), leading byte offset >> 4 in bits [16,30)
//   hi: stride byte offset >> 4 in bits [0,14), descriptor version 1 in bit 14, swizzle mode 2 in bits [29,32)
// The leading byte offset is the distance between 64-element blocks along M/N of an
// MN-major operand (8192 here); K-major operands do not use it.
constexpr uint32_t DESC_HI = (1024u >> 4) | (1u << 14) | (2u << 29);
__device__ __forceinline__ uint32_t desc_lo(uint32_t addr, bool mn_major) {
  return ((addr >> 4) & 0x3FFFu) | ((mn_major ? (8192u >> 4) : 1u) << 16);
}

__device__ __forceinline__ uint32_t pack_bf16x2(float lo, float hi) {
  __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
  return *reinterpret_cast<uint32_t*>(&v);
}
__device__ __forceinline__ float bf16lo(uint32_t w) { return __uint_as_float(w << 16); }
__device__ __forceinline__ float bf16hi(uint32_t w) { return __uint_as_float(w & 0xFFFF0000u); }

// Eight consecutive entries P[i, j0 .. j0+7] (j0 a multiple of 8) of a problem's projection as packed bf16: the
// four words of one Philox call, a Box-Muller pair each; entries outside n x r are zero.
__device__ __forceinline__ uint4 projection8_bf16(const PhiloxKey& key, uint32_t layer_hi, uint32_t layer_lo, uint32_t epoch,
                                                  int n, int r, float neg2ln2_over_r, int i, int j0) {
  const uint4 x = philox4x32_10_layer((uint32_t)(j0 >> 3), (uint32_t)i, epoch, layer_hi, layer_lo, key);
  float g[8];
  box_muller_fast(x.x, neg2ln2_over_r, g[0], g[1]);
  box_muller_fast(x.y, neg2ln2_over_r, g[2], g[3]);
  box_muller_fast(x.z, neg2ln2_over_r, g[4], g[5]);
  box_muller_fast(x.w, neg2ln2_over_r, g[6], g[7]);
  const int left = i < n ? r - j0 : 0;      // valid entries among the eight
  if (left < 8) {
#pragma unroll
    for (int l = 0; l < 8; ++l) g[l] = left > l ? g[l] : 0.f;
  }
  return make_uint4(pack_bf16x2(g[0], g[1]), pack_bf16x2(g[2], g[3]), pack_bf16x2(g[4], g[5]), pack_bf16x2(g[6], g[7]));
}

// Test hook: one CTA waits, with a small limit, on a barrier that nothing will ever arrive at.  The wait gives
// up, records it in the status word and the kernel returns: the path every bounded wait of the kernels takes
// when its signal never comes.
__global__ void wait_that_runs_out_kernel(unsigned int* status, uint32_t limit) {
  __shared__ __align__(8) unsigned long long bar_mem;
  __shared__ int abort_flag;
  if (threadIdx.x == 0) {
    abort_flag = 0;
    mbar_init(smem_u32(&bar_mem), 1);
    fence_barrier_init();
  }
  __syncthreads();
  mbar_wait(smem_u32(&bar_mem), 0u, &abort_flag, status, limit);
}

// Position in a stage ring: the next stage and the parity of the round it is in.
struct Ring {
  int s;
  uint32_t ph;
};
__device__ __forceinline__ void ring_next(Ring& r, int ns) {
  if (++r.s == ns) { r.s = 0; r.ph ^= 1u; }
}
__device__ __forceinline__ void ring_skip(Ring& r, int ns, int count) {
  const int x = r.s + count;
  r.ph ^= (uint32_t)(x / ns) & 1u;
  r.s = x % ns;
}

struct TileCoord {
  int prob, m0, n0, k_begin, k_end, split, nsub, ncol, nst;
};

// kGroup: the launch may hold more than two problems and problems whose K runs over several segments (a group
// of layers that share their input).  The plain instantiation keeps the two-problem arithmetic and reads the
// projection's scalars straight from the constant bank.
template <bool kGroup>
__device__ __forceinline__ TileCoord decode_tile(const Params& prm, int tile) {
  TileCoord t;
  if (kGroup) {
    t.prob = 0;
    for (int i = 1; i < prm.num_problems; ++i)
      if (tile >= prm.prob[i].tile_begin) t.prob = i;
  } else {
    t.prob = (prm.num_problems > 1 && tile >= prm.prob[1].tile_begin) ? 1 : 0;
  }
  const Problem& p = prm.prob[t.prob];
  int local = tile - p.tile_begin;
  const int nb = local % p.tiles_n;
  local /= p.tiles_n;
  const int mb = local % p.tiles_m;
  t.split = local / p.tiles_m;
  t.m0 = mb * BM * p.nsub;
  t.n0 = nb * p.bn * p.ncol;
  t.k_begin = t.split * p.ksteps_per_split;
  t.k_end = min(p.ksteps_total, t.k_begin + p.ksteps_per_split);
  if (prm.cs > 1 && t.prob < prm.num_gen) {
    // items of a cluster walk the stage ring in step: all of them take the full shape, the rows and
    // columns past the edge load as zeros and are never stored
    t.nsub = p.nsub;
    t.ncol = p.ncol;
  } else {
    t.nsub = min(p.nsub, (p.M - t.m0 + BM - 1) / BM);          // row blocks with a valid row
    t.ncol = min(p.ncol, (p.N - t.n0 + p.bn - 1) / p.bn);      // column blocks with a valid column
  }
  // Stages per k-step.  Row blocks come two to a stage and share the B tile of the first stage;
  // column blocks come one to a stage and share the A tile of the first stage.
  t.nst = p.ncol > 1 ? t.ncol : (t.nsub + 1) / 2;
  return t;
}

// --------------------------------------------------------------------------------------
// The kernel.  Warp roles:
//   0      item scheduler and stage owner: waits for a free stage, declares the bytes that will land
//          on its full barrier, arrives, and loads the B tile
//   1, 11  tcgen05.mma issuers (one elected lane each); warp 1 owns TMEM
//   2..9   epilogue: two sets of four warps; with two accumulator slots each set drains one of them
//   10     loader of the A tiles (only issues TMA)
//   12..27 generators of P (launches with a generated operand only)
// --------------------------------------------------------------------------------------
template <bool kGroup>
__global__ void __launch_bounds__(THREADS_GEN, 1) compact_gemm_kernel(const __grid_constant__ Params prm) {
  extern __shared__ uint8_t smem_raw[];
  const uint32_t smem_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
  uint8_t* smem_gen = smem_raw + (smem_base - smem_u32(smem_raw));   // generic pointer to the aligned base
  const uint32_t staging = smem_base + RING_BYTES;
  const uint32_t bars = staging + NUM_EPI_WARPS * STAGING_BUFS * STAGING_BYTES;
  // barrier slots (8 bytes each)
  auto full_bar = [&](int g, int s) { return bars + 8u * ((g ? 2 * NS0 : 0) + s); };
  auto empty_bar = [&](int g, int s) { return bars + 8u * ((g ? 2 * NS0 + NS1 : NS0) + s); };
  auto stage_addr = [&](int g, int s) { return smem_base + (uint32_t)s * (g ? STAGE1_BYTES : STAGE0_BYTES); };
  constexpr int kT = NUM_RING_BARS;
  auto tfull_bar = [&](int a) { return bars + 8u * (kT + a); };
  auto tempty_bar = [&](int a) { return bars + 8u * (kT + 2 + a); };
  auto qfull = [&](int s) { return bars + 8u * (kT + 4 + s); };
  auto qempty = [&](int s) { return bars + 8u * (kT + 4 + QDEPTH + s); };
  auto wbar = [&](int w) { return bars + 8u * (kT + 4 + 2 * QDEPTH + w); };
  uint8_t* tail = smem_gen + RING_BYTES + NUM_EPI_WARPS * STAGING_BUFS * STAGING_BYTES + 8 * NUM_BARRIERS;
  volatile int* tile_q = reinterpret_cast<volatile int*>(tail);
  volatile uint32_t* tmem_slot = reinterpret_cast<volatile uint32_t*>(tail + 4 * QDEPTH);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tail + 4 * QDEPTH + 8);

  const int warp = threadIdx.x >> 5;
  const int lane = threadIdx.x & 31;
  const bool has_gen = prm.gen_ring != GEN_NONE;
  constexpr int GEN_ARRIVALS = NUM_GEN_WARPS;
  const int cs = prm.cs;
  const uint32_t crank = cs > 1 ? cluster_ctarank() : 0u;

  if (threadIdx.x == 0) {
    for (int g = 0; g < 2; ++g)
      for (int s = 0; s < (g ? NS1 : NS0); ++s) {
        mbar_init(full_bar(g, s), 1 + (has_gen ? GEN_ARRIVALS : 0));   // the stage owner, and the generator warps
        // a stage is handed back by up to two MMA issuers in each of cs CTAs (items with a generated
        // operand) or of this CTA; the owner supplies the arrivals that a given use will not get
        mbar_init(empty_bar(g, s), 2 * cs);
      }
    for (int a = 0; a < 2; ++a) {
      mbar_init(tfull_bar(a), 1);
      mbar_init(tempty_bar(a), NUM_EPI_WARPS);
    }
    // consumers of the item queue: MMA thread, loaders, epilogue warps, generator warps
    const int consumers = 3 + NUM_EPI_WARPS + (has_gen ? NUM_GEN_WARPS : 0);
    for (int s = 0; s < QDEPTH; ++s) {
      mbar_init(qfull(s), 1);
      mbar_init(qempty(s), consumers);
    }
    for (int w = 0; w < NUM_EPI_WARPS; ++w) mbar_init(wbar(w), 1);
    *abort_flag = 0;
    fence_barrier_init();
    fence_proxy_async_smem();
  }
  if (warp == 1) {
    tmem_alloc(smem_u32((const void*)tmem_slot), 512);
    tmem_relinquish();
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  if (cs > 1) cluster_sync_all();          // every CTA's barriers exist before anything crosses CTAs
  const uint32_t tmem_base = *tmem_slot;

  // Every consumer role reads the next item from the queue the scheduler fills.
  int qs = 0;
  uint32_t qph = 0;
  auto next_tile = [&](bool whole_warp, bool elected) -> int {
    if (!mbar_wait(qfull(qs), qph, abort_flag, prm.status)) return -1;
    const int tile = tile_q[qs];
    if (whole_warp) __syncwarp();           // every lane has read the slot before it is handed back
    if (elected) mbar_arrive(qempty(qs));
    if (++qs == QDEPTH) { qs = 0; qph ^= 1; }
    return tile;
  };
  // Before the first write into a new geometry: every stage of the old one has been handed back.
  auto drain = [&](int g, const Ring& ro) -> bool {
    for (int s = 0; s < (g ? NS1 : NS0); ++s)
      if (!mbar_wait(empty_bar(g, s), s < ro.s ? ro.ph : ro.ph ^ 1u, abort_flag, prm.status)) return false;
    return true;
  };
  // what stage j of a k-step of item t holds
  auto stage_has_b = [&](const Problem& p, int j) { return p.ncol > 1 || j == 0; };
  auto stage_num_a = [&](const Problem& p, const TileCoord& t, int j) {
    if (p.ncol > 1) return j == 0 ? 1 : 0;
    return min(2, t.nsub - 2 * j);
  };

  // An item whose two accumulators sit in one TMEM slot each is issued by two warps, one accumulator
  // each: a tcgen05.mma costs its issuing thread about as long as the tensor core needs for it, so a
  // single issuer leaves the tensor core idle while it waits on barriers and commits.
  auto item_is_split = [&](const Problem& p, const TileCoord& t) {
    const int naccs = p.nsub * p.ncol;
    return naccs == 2 && t.nsub * t.ncol == 2 && (naccs * p.bn + BN_MAX - 1) / BN_MAX == 2;
  };
  if (warp == 0) {
    // ------------------------- scheduler + stage owner --------------------------
    // Like the MMA warp, these warps walk their loops whole (warp-uniform addresses and counters) and
    // one elected lane touches the barriers and issues the copies.
    {
      Ring r0 = {0, 0u}, r1 = {0, 0u};     // position in each geometry's ring
      int cur_geo = -1;
      bool ok = true;
      int group = (int)(blockIdx.x / cs);  // static part: cluster c takes groups c, c + clusters, ...
      const int group_step = (int)(gridDim.x / cs);
      while (ok) {
        if (!(ok = __all_sync(0xffffffffu, mbar_wait(qempty(qs), qph ^ 1, abort_flag, prm.status)))) break;
        int tile;
        if (cs > 1 && group < prm.gen_groups) {
          int pi = 0;
          if (kGroup)
            for (int i = 1; i < prm.num_gen; ++i)
              if (group >= prm.prob[i].group_begin) pi = i;
          const Problem& p0 = prm.prob[pi];
          const int g = group - p0.group_begin;
          int mb, nb;
          if (prm.share_n) {
            const int per_row = p0.tiles_n / cs;
            mb = g / per_row;
            nb = (g % per_row) * cs + (int)crank;
          } else {
            nb = g % p0.tiles_n;
            mb = (g / p0.tiles_n) * cs + (int)crank;
          }
          tile = p0.tile_begin + mb * p0.tiles_n + nb;
          group += group_step;
        } else {
          tile = 0;
          if (lane == 0) tile = prm.dyn_begin + (int)atomicAdd(prm.sched, 1u);
          tile = __shfl_sync(0xffffffffu, tile, 0);
          if (tile >= prm.total_tiles) tile = -1;
        }
        if (lane == 0) {
          tile_q[qs] = tile;
          mbar_arrive(qfull(qs));
        }
        __syncwarp();
        if (++qs == QDEPTH) { qs = 0; qph ^= 1; }
        if (tile < 0) break;
        const TileCoord t = decode_tile<kGroup>(prm, tile);
        const Problem& p = prm.prob[t.prob];
        const bool a_tma = p.a_mode < GENERATED;
        const bool split = item_is_split(p, t);
        const int geo = p.geo, ns = geo ? NS1 : NS0;
        if (cur_geo >= 0 && geo != cur_geo && !(ok = __all_sync(0xffffffffu, drain(cur_geo, cur_geo ? r1 : r0)))) break;
        cur_geo = geo;
        Ring r = geo ? r1 : r0;
        for (int ks = t.k_begin; ks < t.k_end && ok; ++ks) {
          const int seg = (kGroup && p.nseg > 1) ? (ks >= p.seg_begin[1]) + (ks >= p.seg_begin[2]) : 0;
          const int k0 = kGroup ? (ks - p.seg_begin[seg]) * BK : ks * BK;
          const CUtensorMap* mapB = &prm.tmB[kGroup ? p.map_base + seg : t.prob];
          for (int j = 0; j < t.nst; ++j, ring_next(r, ns)) {
            const int s = r.s;
            if (!(ok = __all_sync(0xffffffffu, mbar_wait(empty_bar(geo, s), r.ph ^ 1u, abort_flag, prm.status)))) break;
            const bool hb = stage_has_b(p, j);
            const int na = stage_num_a(p, t, j);
            uint32_t tx = 0;
            bool gen_here = false;
            // of a generated tile, the shares of the other CTAs arrive as counted bytes
            if (hb) tx += p.bn * BK * 2;
            // (a tile of the sparse projection is cheap: every CTA writes all of it itself)
            if (na > 0) { if (a_tma) tx += na * A_BYTES; else { gen_here = true; if (p.pp_sparse_s == 0) tx += (A_BYTES / cs) * (cs - 1); } }
            if (elect_one()) {
              // A stage that holds a generated tile is handed back with commits from each CTA of the
              // cluster, so that no CTA writes its share of the next tile (or counts its bytes) into a
              // stage that its neighbour has not finished with.  This relies on a stage keeping its role
              // while generated items run: their k-steps take one stage, or two of an even-sized ring.
              // All other stages are handed back locally.  The owner supplies the arrivals that will not
              // come: a use gets commits from both issuers if both read the stage, times cs if shared.
              const int commits = (split && (p.ncol == 1 || j == 0) ? 2 : 1) * (gen_here ? cs : 1);
              if (commits < 2 * cs) mbar_arrive_n(empty_bar(geo, s), 2 * cs - commits);
              const uint32_t fb = full_bar(geo, s);
              if (tx) mbar_expect_tx(fb, tx);
              // arrive for this thread, and for the generator warps when they have nothing to write here
              mbar_arrive_n(fb, 1 + ((has_gen && !gen_here) ? GEN_ARRIVALS : 0));
              if (hb && tx) {
                const uint32_t dst = stage_addr(geo, s) + STAGE_B_OFF;
                const int n0 = t.n0 + (p.ncol > 1 ? j : 0) * p.bn;
                if (p.b_mode == TMA_KMAJOR) {
                  tma_load_2d(dst, mapB, fb, k0, n0);
                } else if (p.b_blocked) {
                  tma_load_3d(dst, mapB, fb, 0, k0, n0 >> 6);
                } else {
                  for (int b = 0; b < p.bn / 64; ++b) tma_load_2d(dst + b * 8192, mapB, fb, n0 + 64 * b, k0);
                }
              }
            }
            __syncwarp();
          }
        }
        if (geo) r1 = r; else r0 = r;
      }
    }
  } else if (warp == LOADER_WARP) {
    // ------------------------------ loader ---------------------------------------
    // Issues the TMA copies of the A tiles; the bytes were declared by the stage owner.
    {
      Ring r0 = {0, 0u}, r1 = {0, 0u};
      int cur_geo = -1;
      bool ok = true;
      while (ok) {
        const int tile = __shfl_sync(0xffffffffu, next_tile(true, lane == 0), 0);
        if (tile < 0) break;
        const TileCoord t = decode_tile<kGroup>(prm, tile);
        const Problem& p = prm.prob[t.prob];
        const int geo = p.geo, ns = geo ? NS1 : NS0;
        if (cur_geo >= 0 && geo != cur_geo && !(ok = __all_sync(0xffffffffu, drain(cur_geo, cur_geo ? r1 : r0)))) break;
        cur_geo = geo;
        Ring r = geo ? r1 : r0;
        bool mine = p.a_mode < GENERATED;
        const int klen = t.k_end - t.k_begin;
        if (!mine) ring_skip(r, ns, klen * t.nst);
        for (int ks = t.k_begin; ks < t.k_end && ok && mine; ++ks) {
          const int seg = (kGroup && p.nseg > 1) ? (ks >= p.seg_begin[1]) + (ks >= p.seg_begin[2]) : 0;
          const int k0 = kGroup ? (ks - p.seg_begin[seg]) * BK : ks * BK;
          const CUtensorMap* mapA = &prm.tmA[kGroup ? p.map_base + seg : t.prob];
          for (int j = 0; j < t.nst; ++j) {
            const int s = r.s;
            const uint32_t eph = r.ph ^ 1u;
            ring_next(r, ns);
            const int na = stage_num_a(p, t, j);
            if (na <= 0) continue;
            if (!(ok = __all_sync(0xffffffffu, mbar_wait(empty_bar(geo, s), eph, abort_flag, prm.status)))) break;
            if (elect_one()) {
              const uint32_t fb = full_bar(geo, s);
              for (int l = 0; l < na; ++l) {
                const int mi = p.ncol > 1 ? 0 : 2 * j + l;
                const int m0 = t.m0 + mi * BM;
                const uint32_t dst = stage_addr(geo, s) + (l == 0 ? STAGE_A0_OFF : STAGE_A1_OFF);
                if (p.a_mode == TMA_KMAJOR) {
                  tma_load_2d(dst, mapA, fb, k0, m0);
                } else if (p.a_blocked) {
                  tma_load_3d(dst, mapA, fb, 0, k0, m0 >> 6);
                } else {
                  tma_load_2d(dst, mapA, fb, m0, k0);
                  tma_load_2d(dst + 8192, mapA, fb, m0 + 64, k0);
                }
              }
            }
            __syncwarp();
          }
        }
        if (geo) r1 = r; else r0 = r;
      }
    }
  } else if (warp == 1 || warp == MMA1_WARP) {
    // ------------------------------ MMA issuers --------------------------------
    // The whole warp walks the loops, so that addresses, descriptors and counters are warp-uniform
    // values; one elected lane issues the MMAs and the commits.  Issuer 0 (warp 1) owns TMEM.  In a
    // split item issuer x computes accumulator x; any other item is issuer 0's alone, and issuer 1
    // only keeps its counters in step.
    {
      const int iss = warp == 1 ? 0 : 1;
      Ring r0 = {0, 0u}, r1 = {0, 0u};
      int acc = 0;
      uint32_t acc_phase = 0;
      bool ok = true;
      const uint16_t cta_mask = (uint16_t)((1u << cs) - 1u);
      while (ok) {
        const int tile = __shfl_sync(0xffffffffu, next_tile(true, lane == 0), 0);
        if (tile < 0) break;
        const TileCoord t = decode_tile<kGroup>(prm, tile);
        const Problem& p = prm.prob[t.prob];
        const bool a_mn = p.a_mode == TMA_MNMAJOR || p.a_mode == GENERATED_T;
        const bool b_mn = p.b_mode != TMA_KMAJOR;
        const uint32_t idesc = (1u << 4) | (1u << 7) | (1u << 10) | ((a_mn ? 1u : 0u) << 15) | ((b_mn ? 1u : 0u) << 16) |
                               ((uint32_t)(p.bn >> 3) << 17) | ((uint32_t)(BM >> 4) << 24);
        const int slots = (p.nsub * p.ncol * p.bn + BN_MAX - 1) / BN_MAX;   // accumulator slots this item occupies
        const bool split = item_is_split(p, t);
        const bool active = split || iss == 0;
        if (slots == 2 && acc == 1) {
          // a two-slot item starts at slot 0: pass slot 1 through unused
          if (!(ok = __all_sync(0xffffffffu, mbar_wait(tempty_bar(1), acc_phase ^ 1, abort_flag, prm.status)))) break;
          if (iss == 0 && elect_one()) umma_commit(tfull_bar(1));
          __syncwarp();
          acc = 0;
          acc_phase ^= 1;
        }
        const int acc0 = acc;
        for (int sl = 0; sl < slots && ok; ++sl) {
          // a split item's issuer x waits for slot x only; an issuer without work in the item waits all the
          // same, so that it never runs more than a phase ahead of these barriers (a parity wait is only
          // sound one phase ahead)
          if (!split || sl == iss)
            ok = __all_sync(0xffffffffu, mbar_wait(tempty_bar(acc), acc_phase ^ 1, abort_flag, prm.status));
          if (++acc == 2) { acc = 0; acc_phase ^= 1; }
        }
        if (!ok) break;
        tc_fence_after();
        const uint32_t d_base = tmem_base + acc0 * BN_MAX;
        // one UMMA consumes K = 16: 32 bytes along a K-major row, or two 8-row groups (2048 bytes) MN-major
        const uint32_t a_step = a_mn ? (2048u >> 4) : (32u >> 4), b_step = b_mn ? (2048u >> 4) : (32u >> 4);
        const int bn = p.bn, nst = t.nst, nsub = t.nsub;
        const bool by_col = p.ncol > 1;
        const int geo = p.geo, ns = geo ? NS1 : NS0;
        Ring r = geo ? r1 : r0;
        if (!active) {
          ring_skip(r, ns, (t.k_end - t.k_begin) * nst);
          if (geo) r1 = r; else r0 = r;
          continue;
        }
        // items with a generated operand walk the ring in step with the other CTAs of the cluster
        const bool gen_shared = cs > 1 && p.a_mode >= GENERATED;
        // accumulator ai of the item sits in slot ai / sps at column (ai % sps) * bn (a slot is 256 columns)
        const int naccs = p.nsub * p.ncol;
        const int sps = BN_MAX / bn > naccs ? naccs : BN_MAX / bn;
        auto acc_col = [&](int ai) -> uint32_t { return (uint32_t)((ai / sps) * BN_MAX + (ai % sps) * bn); };
        // TMEM addresses of the (at most four) accumulators, and the descriptor offsets inside a stage
        const uint32_t d0 = d_base + acc_col(0), d1 = d_base + acc_col(1), d2 = d_base + acc_col(2), d3 = d_base + acc_col(3);
        const uint32_t lbo = (8192u >> 4) << 16, one = 1u << 16;
        const uint32_t a_flags = a_mn ? lbo : one, b_flags = b_mn ? lbo : one;
        const uint32_t stage_step = (uint32_t)(geo ? STAGE1_BYTES : STAGE0_BYTES) >> 4;
        const uint32_t ring_lo = (smem_base >> 4) & 0x3FFFu;
        auto issue4 = [&](uint32_t d, uint32_t a_lo, uint32_t b_lo, uint32_t first) {
          umma_bf16(d, a_lo, DESC_HI, b_lo, DESC_HI, idesc, first);
          umma_bf16(d, a_lo + a_step, DESC_HI, b_lo + b_step, DESC_HI, idesc, 1u);
          umma_bf16(d, a_lo + 2 * a_step, DESC_HI, b_lo + 2 * b_step, DESC_HI, idesc, 1u);
          umma_bf16(d, a_lo + 3 * a_step, DESC_HI, b_lo + 3 * b_step, DESC_HI, idesc, 1u);
        };
        auto commit_stage = [&](int s) {
          if (gen_shared) umma_commit_mc(empty_bar(geo, s), cta_mask);
          else umma_commit(empty_bar(geo, s));
        };
        for (int ks = t.k_begin; ks < t.k_end && ok; ++ks) {
          const uint32_t first = ks > t.k_begin ? 1u : 0u;
          const int s0 = r.s;
          const uint32_t base0 = ring_lo + (uint32_t)s0 * stage_step;       // first stage: holds the shared operand
          for (int j = 0; j < nst; ++j, ring_next(r, ns)) {
            const int s = r.s;
            // split by columns: issuer 0 needs the first stage only, issuer 1 both
            if (split && by_col && iss == 0 && j == 1) continue;
            if (!(ok = __all_sync(0xffffffffu, mbar_wait(full_bar(geo, s), r.ph, abort_flag, prm.status)))) break;
            if (split && by_col && iss == 1 && j == 0) continue;
            tc_fence_after();
            const uint32_t base = ring_lo + (uint32_t)s * stage_step;
            if (elect_one()) {
              if (by_col) {
                if (!split || j == iss)
                  issue4(j == 0 ? d0 : d1, (base0 + (STAGE_A0_OFF >> 4)) | a_flags, (base + (STAGE_B_OFF >> 4)) | b_flags, first);
              } else {
                const uint32_t b_lo = (base0 + (STAGE_B_OFF >> 4)) | b_flags;
                if (!split || iss == 0) issue4(j == 0 ? d0 : d2, (base + (STAGE_A0_OFF >> 4)) | a_flags, b_lo, first);
                if ((!split || iss == 1) && 2 * j + 1 < nsub)
                  issue4(j == 0 ? d1 : d3, (base + (STAGE_A1_OFF >> 4)) | a_flags, b_lo, first);
              }
              // a stage that holds nothing shared goes back at once; the first stage of the k-step goes last
              if (j > 0) umma_commit(empty_bar(geo, s));
              if (j == nst - 1 || (split && by_col && iss == 0)) commit_stage(s0);
            }
            __syncwarp();
          }
        }
        if (!ok) break;
        if (geo) r1 = r; else r0 = r;
        if (elect_one()) {
          if (split) umma_commit(tfull_bar((acc0 + iss) & 1));
          else
            for (int sl = 0; sl < slots; ++sl) umma_commit(tfull_bar((acc0 + sl) & 1));
        }
        __syncwarp();
      }
    }
  } else if (warp < 2 + NUM_EPI_WARPS) {
    // ------------------------------ epilogue ------------------------------------
    // TMEM -> registers -> 128B-swizzled staging tile (32 rows x 128 bytes per warp) -> TMA store.
    // Two sets of four warps (one warp per TMEM lane quarter).  With two accumulator slots in an item
    // set e drains slot e, so both slots empty at the same time; with one slot the sets take alternate
    // chunks.  Every warp still walks every slot (wait for its MMAs, hand it back) so that the
    // hand-back barrier sees a fixed number of arrivals.
    const int q = warp & 3;                 // TMEM lane quarter this warp may read
    const int eset = (warp - 2) >> 2;       // 0 or 1
    const uint32_t stg = staging + (warp - 2) * STAGING_BYTES;
    uint8_t* stg_gen = smem_gen + RING_BYTES + (warp - 2) * STAGING_BYTES;
    int acc = 0;
    uint32_t acc_phase = 0;
    bool ok = true;
    const int sw = lane & 7;
    while (ok) {
      const int tile = next_tile(true, lane == 0);
      if (tile < 0) break;
      const TileCoord t = decode_tile<kGroup>(prm, tile);
      const Problem& p = prm.prob[t.prob];
      const CUtensorMap* mapC = &prm.tmC[kGroup ? p.map_base : t.prob];
      const int naccs = p.nsub * p.ncol;
      const int slots = (naccs * p.bn + BN_MAX - 1) / BN_MAX;
      const int sub_per_slot = BN_MAX / p.bn > naccs ? naccs : BN_MAX / p.bn;
      const int cw = p.epi_mode == EPI_F32 ? 32 : 64;          // columns per staged chunk
      const int cpa = p.bn / cw;                               // chunks per accumulator
      const int row_q = q * 32;
      if (slots == 2 && acc == 1) {
        if (!(ok = mbar_wait(tfull_bar(1), acc_phase, abort_flag, prm.status))) break;
        __syncwarp();
        if (lane == 0) mbar_arrive(tempty_bar(1));
        acc = 0;
        acc_phase ^= 1;
      }
      for (int sl = 0; sl < slots && ok; ++sl) {
        if (!(ok = mbar_wait(tfull_bar(acc), acc_phase, abort_flag, prm.status))) break;
        tc_fence_after();
        bool mine_slot = slots == 2 ? (sl == eset) : true;
        for (int su = 0; su < sub_per_slot && ok && mine_slot; ++su) {
          const int ai = sl * sub_per_slot + su;            // accumulator of the item: a row block or a column block
          const int mi = p.ncol > 1 ? 0 : ai, cb = p.ncol > 1 ? ai : 0;
          if (mi >= t.nsub || cb >= t.ncol) break;
          const int row0 = t.m0 + mi * BM + row_q;
          if (row0 >= p.M) continue;          // this warp's 32 rows are all padding
          const int ncol0 = t.n0 + cb * p.bn;
          const uint32_t tcol = tmem_base + ((uint32_t)(q * 32) << 16) + acc * BN_MAX + su * p.bn;
          for (int ci = (slots == 2 ? 0 : eset); ci < cpa && ok; ci += (slots == 2 ? 1 : 2)) {
            const int col = ncol0 + ci * cw;
            if (col >= p.N) break;
            if (p.epi_mode == EPI_BF16 || p.epi_mode == EPI_UPDATE_W) {
              // convert the whole chunk first; the previous store's read of the staging tile hides behind it.
              // The update stages -(eta alpha) (P N) and lets the TMA unit add it to W (Algorithm 3 line 9).
              uint32_t o[32];
#pragma unroll
              for (int h = 0; h < 2; ++h) {
                uint32_t v[32];
                tmem_ld32(tcol + ci * cw + 32 * h, v);
                tmem_ld_wait();
                if (p.epi_mode == EPI_UPDATE_W) {
                  const float sc = -p.scale;
#pragma unroll
                  for (int j = 0; j < 16; ++j)
                    o[16 * h + j] = pack_bf16x2(sc * __uint_as_float(v[2 * j]), sc * __uint_as_float(v[2 * j + 1]));
                } else {
#pragma unroll
                  for (int j = 0; j < 16; ++j) o[16 * h + j] = pack_bf16x2(__uint_as_float(v[2 * j]), __uint_as_float(v[2 * j + 1]));
                }
              }
              if (lane == 0) tma_store_wait_read();
              __syncwarp();
#pragma unroll
              for (int j = 0; j < 8; ++j)
                *reinterpret_cast<uint4*>(stg_gen + lane * 128 + ((j ^ sw) << 4)) = make_uint4(o[4 * j], o[4 * j + 1], o[4 * j + 2], o[4 * j + 3]);
              fence_proxy_async_smem();
              __syncwarp();
              if (lane == 0) {
                if (p.epi_mode == EPI_UPDATE_W) tma_reduce_add_2d(mapC, stg, col, row0);
                else tma_store_2d(mapC, stg, col, row0);
                tma_store_commit();
              }
              continue;
            }
            if (lane == 0) tma_store_wait_read();          // the previous store has read the staging tile
            __syncwarp();
            if (p.epi_mode == EPI_F32) {
              uint32_t v[32];
              tmem_ld32(tcol + ci * cw, v);
              tmem_ld_wait();
#pragma unroll
              for (int j = 0; j < 8; ++j)
                *reinterpret_cast<uint4*>(stg_gen + lane * 128 + ((j ^ sw) << 4)) =
                    make_uint4(v[4 * j], v[4 * j + 1], v[4 * j + 2], v[4 * j + 3]);
              fence_proxy_async_smem();
              __syncwarp();
              if (lane == 0) {
                tma_store_3d(mapC, stg, col, row0, t.split);
                tma_store_commit();
              }
              continue;
            }
#pragma unroll
            for (int h = 0; h < 2; ++h) {
              uint32_t v[32];
              {
                tmem_ld32(tcol + ci * cw + 32 * h, v);
                tmem_ld_wait();
              }
              if (p.epi_mode == EPI_BF16_T) {
                // lane = output column (row0 + lane), v[z] = output row col + 32 h + z: the staged tile is
                // [64 output rows][32 output columns] of bf16, unswizzled
#pragma unroll
                for (int z = 0; z < 32; ++z)
                  *reinterpret_cast<__nv_bfloat16*>(stg_gen + (32 * h + z) * 64 + lane * 2) =
                      __float2bfloat16_rn(__uint_as_float(v[z]) * p.scale);     // 1, or 1/sqrt(s) of the sparse projection
              }
            }
            if (!ok) break;
            fence_proxy_async_smem();
            __syncwarp();
            if (lane == 0) {
              if (p.epi_mode == EPI_BF16_T) tma_store_2d(mapC, stg, row0, col);
              else tma_store_2d(mapC, stg, col, row0);
              tma_store_commit();
            }
          }
        }
        if (!ok) break;
        tc_fence_before();
        __syncwarp();
        if (lane == 0) mbar_arrive(tempty_bar(acc));
        if (++acc == 2) { acc = 0; acc_phase ^= 1; }
      }
    }
    if (lane == 0) tma_store_wait_all();
  } else {
    // ------------------------------ P generators --------------------------------
    // Write bf16 tiles of P straight into the swizzled operand layout the MMA reads: as the B tile
    // of the first stage of a k-step (forward) or as its A tile 0 (update).
    const int gtid = threadIdx.x - THREADS_BASE;
    constexpr int GSTRIDE = 32 * NUM_GEN_WARPS;
    Ring r0 = {0, 0u}, r1 = {0, 0u};
    bool ok = true;
    const int csh = cs - 1;                                 // log2(cs), cs is 1 or 2
    // the other CTA's window onto the same addresses
    const uint32_t peer_base = cs > 1 ? map_to_cta(smem_base, crank ^ 1u) : 0u;
    const uint32_t peer_full = cs > 1 ? map_to_cta(bars, crank ^ 1u) : 0u;
    while (ok) {
      const int tile = next_tile(true, lane == 0);
      if (tile < 0) break;
      const TileCoord t = decode_tile<kGroup>(prm, tile);
      const Problem& p = prm.prob[t.prob];
      const int klen = t.k_end - t.k_begin;
      const bool gen_a = p.a_mode == GENERATED, gen_at = p.a_mode == GENERATED_T;
      const int geo = p.geo, ns = geo ? NS1 : NS0;
      Ring r = geo ? r1 : r0;
      // The generated problem is the first of its launch, so the generators never write into a ring
      // whose geometry has changed.  In other items the stage owner arrives for them.
      if (!gen_a && !gen_at) ring_skip(r, ns, klen * t.nst);
      // A thread's tasks (eight consecutive entries of a row of P each) keep their place in the tile
      // from k-step to k-step; only the row (transposed forward) or the column (update) of P moves on.
      //   transposed forward: A[m = column j of P][k = row i of P], MN-major, two 64-column blocks of [64 k][128 B]
      //   update:             A[m = row i of P][k = column j of P], K-major, [128 rows][128 B]
      // Of a tile shared by a cluster this CTA writes the rows crank * (rows / cs) onward.
      // When a k-step takes two stages (the generated tiles then live in stages 0 and 2) and a cluster shares them, the
      // sixteen warps work as two halves, one per stage: a half builds every other tile, two tasks per thread, and its
      // fence, arrival and wait for the stage overlap the other half's arithmetic.  A half meets every use of its stage.
      const bool halves = t.nst == 2 && cs == 2;
      const int my_half = (warp - (THREADS_BASE >> 5)) >> 3;
      const int ntask = halves ? 2 : (2 >> csh);        // tasks per thread and tile
      // the plain instantiation's only generated problem is problem 0: constant-bank operands
      const Problem& gp = kGroup ? p : prm.prob[0];
      const int ik = gen_at ? 1 : 0, jk = 1 - ik;       // which index of P advances with k
      int t_i[2], t_j[2];
      uint32_t t_off[2];
#pragma unroll
      for (int u = 0; u < 2; ++u) {
        const int id = halves ? (gtid & (GSTRIDE / 2 - 1)) + u * (GSTRIDE / 2) : gtid + u * GSTRIDE;
        if (gen_at) {
          const int c = id & 15, kr = (int)crank * (BK >> csh) + (id >> 4);
          t_i[u] = kr; t_j[u] = t.m0 + c * 8;
          t_off[u] = STAGE_A0_OFF + (c >> 3) * 8192 + kr * 128 + (((c & 7) ^ (kr & 7)) << 4);
        } else {
          const int c = id & 7, rr = (int)crank * (BM >> csh) + (id >> 3);
          t_i[u] = t.m0 + rr; t_j[u] = c * 8;
          t_off[u] = STAGE_A0_OFF + rr * 128 + ((c ^ (rr & 7)) << 4);
        }
      }
      for (int ks = t.k_begin; ks < t.k_end && ok && (gen_a || gen_at); ++ks) {
        const int s = r.s;
        const uint32_t eph = r.ph ^ 1u;
        ring_next(r, ns);
        if (t.nst > 1) ring_next(r, ns);            // a k-step takes one or two stages
        const uint32_t stage_off = (uint32_t)s * (geo ? STAGE1_BYTES : STAGE0_BYTES);
        const uint32_t full_off = full_bar(geo, s) - bars;
        const int k0 = ks * BK;
        if (gp.pp_sparse_s > 0) {
          // Sparse projection: the tile holds the integer counts and every CTA writes the whole of it.  The
          // sixteen warps work as four groups of four; the group whose number is the stage's builds the tile, so
          // that up to four tiles are under construction at once (one tile is a chain of waits -- free stage,
          // clear, Philox, scatter, fence -- far longer than its arithmetic) and a group meets every use of its
          // stage.  The group's threads clear the tile, then one thread per row of P adds the signs of the row's
          // terms that fall into the tile's columns (a row has one writer: colliding terms add without a race).
          const int grp = (warp - (THREADS_BASE >> 5)) >> 2, gt = gtid & 127;
          if (grp != s) continue;
          const bool w = mbar_wait(empty_bar(geo, s), eph, abort_flag, prm.status);
          uint8_t* tile = smem_gen + stage_off + STAGE_A0_OFF;
          if (w) {
#pragma unroll
            for (int x = 0; x < A_BYTES / 16 / 128; ++x) reinterpret_cast<uint4*>(tile)[gt + 128 * x] = make_uint4(0u, 0u, 0u, 0u);
          }
          named_barrier(2 + grp, 128);
          const int nrows = gen_at ? BK : BM;
          const int i = gen_at ? k0 + gt : t.m0 + gt;                  // the row of P this thread owns
          const int c_first = gen_at ? t.m0 : k0, c_count = gen_at ? BM : BK;
          if (w && gt < nrows && i < gp.pp_n) {
            for (int q = 0; 4 * q < gp.pp_sparse_s; ++q) {
              const uint4 x = sparse_words4((uint32_t)q, (uint32_t)i, gp.pp_epoch, gp.pp_layer_hi, gp.pp_layer_lo, prm.key);
              const uint32_t wd[4] = {x.x, x.y, x.z, x.w};
#pragma unroll
              for (int l = 0; l < 4; ++l) {
                const int c = sparse_col(wd[l], gp.pp_r) - c_first;
                if (4 * q + l < gp.pp_sparse_s && c >= 0 && c < c_count) {
                  const int rr = gt;
                  const uint32_t off = gen_at ? (uint32_t)((c >> 6) * 8192 + rr * 128 + ((((c >> 3) & 7) ^ (rr & 7)) << 4) + (c & 7) * 2)
                                              : (uint32_t)(rr * 128 + (((c >> 3) ^ (rr & 7)) << 4) + (c & 7) * 2);
                  __nv_bfloat16* e = reinterpret_cast<__nv_bfloat16*>(tile + off);
                  *e = __float2bfloat16_rn(__bfloat162float(*e) + sparse_sign(wd[l]));
                }
              }
            }
          }
          fence_proxy_async_smem();
          ok = __all_sync(0xffffffffu, w);
          if (ok && lane == 0) mbar_arrive_n(full_bar(geo, s), NUM_GEN_WARPS / 4);     // four warps stand in for the sixteen
          continue;
        }
        if (halves && ((s >> 1) & 1) != my_half) continue;
        const bool w = mbar_wait(empty_bar(geo, s), eph, abort_flag, prm.status);
#pragma unroll
        for (int u = 0; u < 2; ++u) {
          if (u < ntask && w) {
            const uint4 val = projection8_bf16(prm.key, gp.pp_layer_hi, gp.pp_layer_lo, gp.pp_epoch, gp.pp_n, gp.pp_r,
                                               gp.pp_scale, t_i[u] + ik * k0, t_j[u] + jk * k0);
            const uint32_t off = stage_off + t_off[u];
            *reinterpret_cast<uint4*>(smem_gen + off) = val;
            if (cs > 1) st_async_16(peer_base + off, val, peer_full + full_off);
          }
        }
        fence_proxy_async_smem();
        ok = __all_sync(0xffffffffu, w);
        if (ok && lane == 0) mbar_arrive_n(full_bar(geo, s), halves ? 2 : 1);     // a half's eight warps stand in for the sixteen
        // later stages of the k-step hold no generated data: the stage owner arrives for the generators there
      }
      if (geo) r1 = r; else r0 = r;
    }
  }

  tc_fence_before();
  __syncthreads();
  if (warp == 1) {
    tc_fence_after();
    tmem_dealloc(tmem_base, 512);
  }
  // no CTA leaves while another of its cluster may still signal its barriers
  if (cs > 1) cluster_sync_all();
  // the last CTA to finish re-arms the scheduler words for the next launch
  if (threadIdx.x == 0) {
    __threadfence();
    if (atomicAdd(prm.sched + 1, 1u) == gridDim.x - 1) {
      prm.sched[0] = 0u;
      prm.sched[1] = 0u;
      __threadfence();
    }
  }
}

// --------------------------------------------------------------------------------------
// Element-wise kernels around the GEMMs
// --------------------------------------------------------------------------------------
// Algorithm 3 lines 1-5: moments in place, N rounded to bf16 into scratch (pitch m).
__device__ __forceinline__ void adam_moments_bf16_at(long long idx, const float* __restrict__ Gc, long long ldg,
                                                     float* __restrict__ Mo, float* __restrict__ Vo,
                                                     __nv_bfloat16* __restrict__ Nout, int r, int m,
                                                     const simt::AdamScalars& s) {
  const int m4 = m >> 2;
  if (idx >= (long long)r * m4) return;
  const int j = (int)(idx / m4), c = (int)(idx % m4) * 4;
  const long long off = (long long)j * ldg + c;
  const float4 g = *reinterpret_cast<const float4*>(Gc + off);
  float4 mm = *reinterpret_cast<const float4*>(Mo + off);
  float4 vv = *reinterpret_cast<const float4*>(Vo + off);
  mm.x = fmaf(s.beta1, mm.x, s.one_minus_beta1 * g.x);
  mm.y = fmaf(s.beta1, mm.y, s.one_minus_beta1 * g.y);
  mm.z = fmaf(s.beta1, mm.z, s.one_minus_beta1 * g.z);
  mm.w = fmaf(s.beta1, mm.w, s.one_minus_beta1 * g.w);
  vv.x = fmaf(s.beta2, vv.x, s.one_minus_beta2 * g.x * g.x);
  vv.y = fmaf(s.beta2, vv.y, s.one_minus_beta2 * g.y * g.y);
  vv.z = fmaf(s.beta2, vv.z, s.one_minus_beta2 * g.z * g.z);
  vv.w = fmaf(s.beta2, vv.w, s.one_minus_beta2 * g.w * g.w);
  *reinterpret_cast<float4*>(Mo + off) = mm;
  *reinterpret_cast<float4*>(Vo + off) = vv;
  const float n0 = (mm.x * s.inv_bias1) / (sqrtf(vv.x * s.inv_bias2) + s.eps);
  const float n1 = (mm.y * s.inv_bias1) / (sqrtf(vv.y * s.inv_bias2) + s.eps);
  const float n2 = (mm.z * s.inv_bias1) / (sqrtf(vv.z * s.inv_bias2) + s.eps);
  const float n3 = (mm.w * s.inv_bias1) / (sqrtf(vv.w * s.inv_bias2) + s.eps);
  uint2 o = make_uint2(pack_bf16x2(n0, n1), pack_bf16x2(n2, n3));
  *reinterpret_cast<uint2*>(Nout + (long long)j * m + c) = o;
}
__global__ void adam_moments_bf16_kernel(const float* __restrict__ Gc, long long ldg, float* __restrict__ Mo,
                                         float* __restrict__ Vo, __nv_bfloat16* __restrict__ Nout, int r, int m,
                                         simt::AdamScalars s) {
  adam_moments_bf16_at((long long)blockIdx.x * blockDim.x + threadIdx.x, Gc, ldg, Mo, Vo, Nout, r, m, s);
}

// Deterministic reduction of the split-K partials of Gc, in split order.
__global__ void reduce_partials_kernel(const float* __restrict__ part, long long split_stride, int splits,
                                       float* __restrict__ Gc, long long ldg, int r, int m, int accumulate) {
  const int m4 = m >> 2;
  const long long idx = (long long)blockIdx.x * blockDim.x + threadIdx.x;
  if (idx >= (long long)r * m4) return;
  const int j = (int)(idx / m4), c = (int)(idx % m4) * 4;
  float4 acc = accumulate ? *reinterpret_cast<const float4*>(Gc + (long long)j * ldg + c) : make_float4(0.f, 0.f, 0.f, 0.f);
  for (int s = 0; s < splits; ++s) {
    const float4 p = *reinterpret_cast<const float4*>(part + s * split_stride + (long long)j * m + c);
    acc.x += p.x; acc.y += p.y; acc.z += p.z; acc.w += p.w;
  }
  *reinterpret_cast<float4*>(Gc + (long long)j * ldg + c) = acc;
}

// --------------------------------------------------------------------------------------
// Host side
// --------------------------------------------------------------------------------------
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

inline EncodeTiledFn encode_fn() {
  // initialised exactly once, also when several threads make their first launch together
  static const EncodeTiledFn fn = []() -> EncodeTiledFn {
    void* p = nullptr;
    cudaDriverEntryPointQueryResult q;
    if (cudaGetDriverEntryPointByVersion("cuTensorMapEncodeTiled", &p, 12000, cudaEnableDefault, &q) == cudaSuccess &&
        q == cudaDriverEntryPointSuccess)
      return (EncodeTiledFn)p;
    cudaGetLastError();
    return nullptr;
  }();
  return fn;
}

// Tensor maps are pure functions of (pointer, extents, pitches, box, element type, swizzle): a layer that is
// called step after step on the same buffers asks for the same few maps again and again, so each thread keeps
// the ones it has encoded.
struct MapKey {
  uint64_t v[8];
  bool operator==(const MapKey& o) const { return memcmp(v, o.v, sizeof(v)) == 0; }
};
struct MapKeyHash {
  size_t operator()(const MapKey& k) const {
    uint64_t h = 0x9E3779B97F4A7C15ull;
    for (int i = 0; i < 8; ++i) h = (h ^ k.v[i]) * 0xFF51AFD7ED558CCDull + (h >> 29);
    return (size_t)h;
  }
};

inline bool encode_cached(CUtensorMap* map, CUtensorMapDataType type, uint32_t rank, const void* base, const cuuint64_t* dims,
                          const cuuint64_t* strides, const cuuint32_t* box, CUtensorMapSwizzle swizzle) {
  EncodeTiledFn fn = encode_fn();
  if (!fn) return false;
  MapKey key;
  memset(&key, 0, sizeof(key));
  key.v[0] = (uint64_t)(uintptr_t)base;
  key.v[1] = (uint64_t)type | ((uint64_t)rank << 8) | ((uint64_t)swizzle << 16);
  for (uint32_t i = 0; i < rank; ++i) {
    key.v[2 + i] = dims[i];
    key.v[7] = key.v[7] * 1031u + box[i];
  }
  for (uint32_t i = 0; i + 1 < rank; ++i) key.v[5 + i] = strides[i];
  thread_local std::unordered_map<MapKey, CUtensorMap, MapKeyHash> cache;
  auto it = cache.find(key);
  if (it != cache.end()) {
    *map = it->second;
    return true;
  }
  cuuint32_t estr[3] = {1, 1, 1};
  if (fn(map, type, rank, const_cast<void*>(base), dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE, swizzle,
         CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
    return false;
  if (cache.size() >= 8192) cache.clear();
  cache.emplace(key, *map);
  return true;
}

// 2-D bf16 map over a row-major matrix: `inner` contiguous elements per row, `rows` rows, pitch in elements.
inline bool make_map(CUtensorMap* map, const void* base, int64_t inner, int64_t rows, int64_t pitch, int box_inner,
                     int box_rows, bool swizzle = true) {
  cuuint64_t dims[2] = {(cuuint64_t)inner, (cuuint64_t)rows};
  cuuint64_t strides[1] = {(cuuint64_t)pitch * 2};
  cuuint32_t box[2] = {(cuuint32_t)box_inner, (cuuint32_t)box_rows};
  return encode_cached(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, base, dims, strides, box,
                       swizzle ? CU_TENSOR_MAP_SWIZZLE_128B : CU_TENSOR_MAP_SWIZZLE_NONE);
}

// MN-major operand tiles: the matrix (rows x cols, cols a multiple of 64) seen as [cols / 64][rows][64], so
// that one copy of a {64, box_rows, blocks} box lands as `blocks` consecutive swizzled [box_rows][128 B]
// pieces -- the layout the MMA descriptor of an MN-major operand walks.
inline bool make_map_blocked(CUtensorMap* map, const void* base, int64_t cols, int64_t rows, int64_t pitch, int box_rows,
                             int blocks) {
  cuuint64_t dims[3] = {64, (cuuint64_t)rows, (cuuint64_t)(cols / 64)};
  cuuint64_t strides[2] = {(cuuint64_t)pitch * 2, 128};
  cuuint32_t box[3] = {64, (cuuint32_t)box_rows, (cuuint32_t)blocks};
  return encode_cached(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, base, dims, strides, box, CU_TENSOR_MAP_SWIZZLE_128B);
}

// 3-D fp32 map over `planes` row-major matrices of rows x inner (pitch and plane stride in elements);
// boxes are 32 columns x 32 rows of one plane.
inline bool make_map_f32_3d(CUtensorMap* map, const void* base, int64_t inner, int64_t rows, int64_t planes, int64_t pitch,
                            int64_t plane_stride) {
  cuuint64_t dims[3] = {(cuuint64_t)inner, (cuuint64_t)rows, (cuuint64_t)planes};
  cuuint64_t strides[2] = {(cuuint64_t)pitch * 4, (cuuint64_t)plane_stride * 4};
  cuuint32_t box[3] = {32, 32, 1};
  return encode_cached(map, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 3, base, dims, strides, box, CU_TENSOR_MAP_SWIZZLE_128B);
}

// Tile width: up to 256 columns, in whole 64-column blocks.
inline int pick_bn(int N) { return N >= BN_MAX ? BN_MAX : (int)((N + 63) / 64 * 64); }

#ifndef CFG_NSUB
#define CFG_NSUB 2
#endif

inline void set_projection(Problem& p, const ProjectionParams& pp) {
  p.pp_layer_hi = pp.layer_hi; p.pp_layer_lo = pp.layer_lo; p.pp_epoch = pp.epoch;
  p.pp_n = pp.n; p.pp_r = pp.r; p.pp_scale = pp.neg2ln2_over_r;
  p.pp_sparse_s = pp.sparse_s;
}

inline void finish_problem(Problem& p, int splits_wanted) {
  if (p.bn == 0) p.bn = pick_bn(p.N);
  // two row blocks share each B tile: 256 x 256 items halve the shared-memory refill per flop and
  // put eight MMAs behind every barrier wait
  if (p.nsub == 0) p.nsub = p.M > BM ? CFG_NSUB : 1;
  if (p.ncol == 0) p.ncol = 1;
  p.geo = p.nsub == 1 ? 1 : 0;
  p.tiles_m = (p.M + BM * p.nsub - 1) / (BM * p.nsub);
  p.tiles_n = (p.N + p.bn * p.ncol - 1) / (p.bn * p.ncol);
  p.ksteps_total = (p.K + BK - 1) / BK;
  int s = splits_wanted < 1 ? 1 : splits_wanted;
  if (s > p.ksteps_total) s = p.ksteps_total;
  p.ksteps_per_split = (p.ksteps_total + s - 1) / s;
  p.splits = (p.ksteps_total + p.ksteps_per_split - 1) / p.ksteps_per_split;
  if (p.nseg <= 1) {
    p.nseg = 1;
    p.seg_begin[0] = 0;
    p.seg_begin[1] = p.seg_begin[2] = p.seg_begin[3] = p.ksteps_total;
  }
}

// Number of token splits of Gc = Z^T dY.  A split should be about as long as one dX item
// (m / 64 k-steps) so that the dynamic scheduler balances well, and there should be enough
// items to occupy the SMs; at most 32.
inline int plan_gc_splits(int64_t tokens, int r, int m, int dx_ksteps = 0) {
  const int items = ((r + 2 * BM - 1) / (2 * BM)) * ((m + pick_bn(m) - 1) / pick_bn(m));
  const int ksteps = (int)((tokens + BK - 1) / BK);
  if (ksteps < 1) return 1;
  if (dx_ksteps <= 0) dx_ksteps = (m + BK - 1) / BK;
  const int by_len = (ksteps + dx_ksteps - 1) / dx_ksteps;
  const int by_fill = (NUM_SMS + items - 1) / items;
  int s = by_len > by_fill ? by_len : by_fill;
  if (s < 1) s = 1;
  if (s > 32) s = 32;
  if (s > ksteps) s = ksteps;
  const int per = (ksteps + s - 1) / s;
  return (ksteps + per - 1) / per;
}

// Partials are staged in the workspace when there is more than one split or when the call
// accumulates into Gc; the size covers both.
inline size_t gc_workspace_bytes(int64_t tokens, int r, int m) {
  return (size_t)plan_gc_splits(tokens, r, m) * r * m * sizeof(float);
}

inline compact_status_t launch(const LaunchInfo& li, Params& prm) {
  // the opt-in to large dynamic shared memory is a per-device attribute of the kernel
  static std::atomic<bool> attr_set[64];
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) { cudaGetLastError(); return COMPACT_ERR_CUDA; }
  if (!attr_set[dev].load(std::memory_order_acquire)) {
    if (cudaFuncSetAttribute(compact_gemm_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize, SMEM_BYTES) != cudaSuccess ||
        cudaFuncSetAttribute(compact_gemm_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, SMEM_BYTES) != cudaSuccess) {
      cudaGetLastError();
      return COMPACT_ERR_CUDA;
    }
    attr_set[dev].store(true, std::memory_order_release);
  }
  bool group = prm.num_problems > 2;
  for (int i = 0; i < prm.num_problems; ++i) group = group || prm.prob[i].nseg > 1;
  // The problems with a generated operand come first.  Sharing generated tiles needs the four-stage ring,
  // where a stage keeps its role (see the stage owner).
  prm.num_gen = 0;
  bool gen_geo1 = true;
  while (prm.num_gen < prm.num_problems && prm.prob[prm.num_gen].a_mode >= GENERATED) {
    gen_geo1 = gen_geo1 && prm.prob[prm.num_gen].geo == 1;
    ++prm.num_gen;
  }
  const int cs = (prm.num_gen > 0 && li.cluster > 1 && gen_geo1) ? 2 : 1;
  prm.cs = cs;
  prm.share_n = 1;      // the cs items of a group are neighbours along N (tokens in the forward, columns of W in the update)
  prm.gen_groups = 0;
  int t = 0, maps = 0;
  for (int i = 0; i < prm.num_problems; ++i) {
    Problem& p = prm.prob[i];
    if (cs > 1 && i < prm.num_gen) {
      // items with a generated operand come in groups of cs neighbours
      p.tiles_n = (p.tiles_n + cs - 1) / cs * cs;
      p.group_begin = prm.gen_groups;
      prm.gen_groups += p.tiles_m * p.tiles_n / cs;
    }
    p.tile_begin = t;
    t += p.tiles_m * p.tiles_n * p.splits;
    if (i + 1 == prm.num_gen) prm.dyn_begin = cs > 1 ? t : 0;
    p.map_base = maps;
    maps += p.nseg;
  }
  if (maps > MAXP) return COMPACT_ERR_INVALID_ARG;
  prm.total_tiles = t;
  prm.status = li.status;
  prm.sched = li.sched;
  const int grid = t < NUM_SMS ? (t + cs - 1) / cs * cs : NUM_SMS / cs * cs;
  const int threads = prm.gen_ring != GEN_NONE ? THREADS_GEN : THREADS_BASE;
  cudaLaunchConfig_t cfg;
  memset(&cfg, 0, sizeof(cfg));
  cfg.gridDim = dim3((unsigned)grid, 1, 1);
  cfg.blockDim = dim3((unsigned)threads, 1, 1);
  cfg.dynamicSmemBytes = SMEM_BYTES;
  cfg.stream = li.stream;
  cudaLaunchAttribute attr;
  attr.id = cudaLaunchAttributeClusterDimension;
  attr.val.clusterDim.x = (unsigned)cs;
  attr.val.clusterDim.y = 1;
  attr.val.clusterDim.z = 1;
  cfg.attrs = &attr;
  cfg.numAttrs = 1;
  const cudaError_t e = group ? cudaLaunchKernelEx(&cfg, compact_gemm_kernel<true>, prm)
                              : cudaLaunchKernelEx(&cfg, compact_gemm_kernel<false>, prm);
  (*li.launches)++;
  if (e != cudaSuccess) { cudaGetLastError(); return COMPACT_ERR_CUDA; }
  return cudaGetLastError() == cudaSuccess ? COMPACT_OK : COMPACT_ERR_CUDA;
}

inline bool tc_shape_ok(int64_t tokens, int n, int m) { return tokens >= 1 && n % 8 == 0 && m % 8 == 0; }

// Algorithm 1: problem 0 = Z = X P (generated operand; longest items go first), problem 1 = Y = X W.
// Either output may be absent (nullptr): Y alone is the forward of a layer that will recompute Z in its
// backward, Z alone is that recomputation.
inline compact_status_t forward(const LaunchInfo& li, const ProjectionParams& pp, int64_t tokens, int m,
                                const __nv_bfloat16* X, int64_t ldx, const __nv_bfloat16* W, int64_t ldw,
                                __nv_bfloat16* Y, int64_t ldy, __nv_bfloat16* Z, int64_t ldz, int zcols) {
  const int n = pp.n;
  if (!tc_shape_ok(tokens, n, m)) return COMPACT_ERR_SHAPE;
  if (!li.status || !li.sched) return COMPACT_ERR_CUDA;
  if (!Y && !Z) return COMPACT_OK;
  Params prm;
  memset(&prm, 0, sizeof(prm));
  prm.key = pp.key;
  prm.num_problems = (Y && Z) ? 2 : 1;
  prm.gen_ring = Z ? GEN_A : GEN_NONE;
  const int iy = Z ? 1 : 0;       // where the Y problem sits
  if (Z) {
    // Z is computed transposed, Z^T = P^T X^T: the generated tile of P (64 rows of P by 128 of its columns)
    // is the A operand, and up to 512 tokens of X ride on the N side in two 256-wide accumulators, so the
    // MMAs run at N = 256 and one generated tile feeds 512 tokens.
    Problem& pz = prm.prob[0];
    pz.M = zcols; pz.N = (int)tokens; pz.K = n;
    pz.nsub = 1;
    pz.ncol = tokens > BN_MAX ? 2 : 1;
    pz.a_mode = GENERATED_T; pz.b_mode = TMA_KMAJOR; pz.epi_mode = EPI_BF16_T;
    set_projection(pz, pp);
    pz.scale = pp.inv_sqrt_s;
    finish_problem(pz, 1);
    prm.tmA[0] = prm.tmA[iy];   // unused by the generated operand (set below when Y is present)
    if (!make_map(&prm.tmB[0], X, n, tokens, ldx, BK, pz.bn)) return COMPACT_ERR_CUDA;
    if (!make_map(&prm.tmC[0], Z, zcols, tokens, ldz, 32, 64, false)) return COMPACT_ERR_CUDA;
  }
  if (Y) {
    Problem& py = prm.prob[iy];
    py.M = (int)tokens; py.N = m; py.K = n;
    py.a_mode = TMA_KMAJOR; py.b_mode = TMA_MNMAJOR; py.epi_mode = EPI_BF16;
    finish_problem(py, 1);
    if (!make_map(&prm.tmA[iy], X, n, tokens, ldx, BK, BM)) return COMPACT_ERR_CUDA;
    py.b_blocked = m % 64 == 0;
    if (py.b_blocked ? !make_map_blocked(&prm.tmB[iy], W, m, n, ldw, BK, py.bn / 64) : !make_map(&prm.tmB[iy], W, m, n, ldw, 64, BK))
      return COMPACT_ERR_CUDA;
    if (!make_map(&prm.tmC[iy], Y, m, tokens, ldy, 64, 32)) return COMPACT_ERR_CUDA;
  }
  if (Z) prm.tmA[0] = prm.tmB[0];   // any valid map: the loader never uses it for a generated operand
  return launch(li, prm);
}

// Algorithm 2: problem 0 = Gc = Z^T dY (both operands MN-major, split over tokens), problem 1 = dX = dY W^T.
inline compact_status_t backward(const LaunchInfo& li, int64_t tokens, int n, int m, int r, int zcols,
                                 const __nv_bfloat16* dY, int64_t lddy, const __nv_bfloat16* Z, int64_t ldz,
                                 const __nv_bfloat16* W, int64_t ldw, __nv_bfloat16* dX, int64_t lddx, float* Gc,
                                 int64_t ldg, int accumulate, void* workspace, size_t workspace_bytes) {
  if (!tc_shape_ok(tokens, n, m)) return COMPACT_ERR_SHAPE;
  if (!li.status || !li.sched) return COMPACT_ERR_CUDA;
  Params prm;
  memset(&prm, 0, sizeof(prm));
  prm.num_problems = dX ? 2 : 1;
  prm.gen_ring = GEN_NONE;
  const int splits = plan_gc_splits(tokens, r, m);
  const bool staged = splits > 1 || accumulate;
  if (staged && workspace_bytes < (size_t)splits * r * m * sizeof(float)) return COMPACT_ERR_WORKSPACE;
  Problem& pg = prm.prob[0];
  pg.M = r; pg.N = m; pg.K = (int)tokens;
  pg.a_mode = TMA_MNMAJOR; pg.b_mode = TMA_MNMAJOR; pg.epi_mode = EPI_F32;
  finish_problem(pg, splits);
  if (staged) {
    if (!make_map_f32_3d(&prm.tmC[0], workspace, m, r, pg.splits, m, (int64_t)r * m)) return COMPACT_ERR_CUDA;
  } else {
    if (!make_map_f32_3d(&prm.tmC[0], Gc, m, r, 1, ldg, (int64_t)r * ldg)) return COMPACT_ERR_CUDA;
  }
  pg.a_blocked = zcols % 64 == 0;
  pg.b_blocked = m % 64 == 0;
  if (pg.a_blocked ? !make_map_blocked(&prm.tmA[0], Z, zcols, tokens, ldz, BK, 2) : !make_map(&prm.tmA[0], Z, zcols, tokens, ldz, 64, BK))
    return COMPACT_ERR_CUDA;
  if (pg.b_blocked ? !make_map_blocked(&prm.tmB[0], dY, m, tokens, lddy, BK, pg.bn / 64)
                   : !make_map(&prm.tmB[0], dY, m, tokens, lddy, 64, BK))
    return COMPACT_ERR_CUDA;
  if (dX) {
    Problem& px = prm.prob[1];
    px.M = (int)tokens; px.N = n; px.K = m;
    px.a_mode = TMA_KMAJOR; px.b_mode = TMA_KMAJOR; px.epi_mode = EPI_BF16;
    finish_problem(px, 1);
    if (!make_map(&prm.tmA[1], dY, m, tokens, lddy, BK, BM)) return COMPACT_ERR_CUDA;
    if (!make_map(&prm.tmB[1], W, m, n, ldw, BK, px.bn)) return COMPACT_ERR_CUDA;
    if (!make_map(&prm.tmC[1], dX, n, tokens, lddx, 64, 32)) return COMPACT_ERR_CUDA;
  }
  compact_status_t s = launch(li, prm);
  if (s != COMPACT_OK) return s;
  if (staged) {
    const long long cnt = (long long)r * (m / 4);
    reduce_partials_kernel<<<(unsigned)((cnt + 255) / 256), 256, 0, li.stream>>>(
        (const float*)workspace, (long long)r * m, pg.splits, Gc, ldg, r, m, accumulate);
    (*li.launches)++;
    if (cudaGetLastError() != cudaSuccess) return COMPACT_ERR_CUDA;
  }
  return COMPACT_OK;
}

// --------------------------------------------------------------------------------------
// Groups of layers that share their input (q, k, v; gate, up): each layer has its own W and its own P
// (the paper's appendix on saved tensors lists x P_q, x P_k, x P_v as separate compressed activations).
// One forward launch computes every Z_g = X P_g and Y_g = X W_g; one backward launch computes
// dX = sum_g dY_g W_g^T in a single accumulator (K runs over the layers' segments) and every Gc_g.
// --------------------------------------------------------------------------------------
struct GroupLayer {
  ProjectionParams pp;
  int m, r, zcols;
  const __nv_bfloat16* W; int64_t ldw;
  __nv_bfloat16* Y; int64_t ldy;          // forward
  __nv_bfloat16* Z; int64_t ldz;          // forward (output), backward (input)
  const __nv_bfloat16* dY; int64_t lddy;  // backward
  float* Gc; int64_t ldg;                 // backward
};

inline compact_status_t forward_group(const LaunchInfo& li, int G, const GroupLayer* L, int64_t tokens, int n,
                                      const __nv_bfloat16* X, int64_t ldx) {
  if (G < 1 || G > MAXG) return COMPACT_ERR_INVALID_ARG;
  if (!li.status || !li.sched) return COMPACT_ERR_CUDA;
  for (int g = 0; g < G; ++g)
    if (!tc_shape_ok(tokens, n, L[g].m)) return COMPACT_ERR_SHAPE;
  Params prm;
  memset(&prm, 0, sizeof(prm));
  prm.key = L[0].pp.key;
  prm.num_problems = 2 * G;
  prm.gen_ring = GEN_A;
  for (int g = 0; g < G; ++g) {
    Problem& pz = prm.prob[g];
    pz.M = L[g].zcols; pz.N = (int)tokens; pz.K = n;
    pz.nsub = 1;
    pz.ncol = tokens > BN_MAX ? 2 : 1;
    pz.a_mode = GENERATED_T; pz.b_mode = TMA_KMAJOR; pz.epi_mode = EPI_BF16_T;
    set_projection(pz, L[g].pp);
    pz.scale = L[g].pp.inv_sqrt_s;
    finish_problem(pz, 1);
    if (!make_map(&prm.tmB[g], X, n, tokens, ldx, BK, pz.bn)) return COMPACT_ERR_CUDA;
    prm.tmA[g] = prm.tmB[g];   // unused by the generated operand
    if (!make_map(&prm.tmC[g], L[g].Z, L[g].zcols, tokens, L[g].ldz, 32, 64, false)) return COMPACT_ERR_CUDA;
    Problem& py = prm.prob[G + g];
    py.M = (int)tokens; py.N = L[g].m; py.K = n;
    py.a_mode = TMA_KMAJOR; py.b_mode = TMA_MNMAJOR; py.epi_mode = EPI_BF16;
    finish_problem(py, 1);
    if (!make_map(&prm.tmA[G + g], X, n, tokens, ldx, BK, BM)) return COMPACT_ERR_CUDA;
    py.b_blocked = L[g].m % 64 == 0;
    if (py.b_blocked ? !make_map_blocked(&prm.tmB[G + g], L[g].W, L[g].m, n, L[g].ldw, BK, py.bn / 64)
                     : !make_map(&prm.tmB[G + g], L[g].W, L[g].m, n, L[g].ldw, 64, BK))
      return COMPACT_ERR_CUDA;
    if (!make_map(&prm.tmC[G + g], L[g].Y, L[g].m, tokens, L[g].ldy, 64, 32)) return COMPACT_ERR_CUDA;
  }
  return launch(li, prm);
}

// Workspace of the group backward: the layers' split-K partials, one after the other.
inline size_t group_gc_workspace_bytes(int G, const int* r, const int* m, int64_t tokens) {
  int dx_ksteps = 0;
  for (int g = 0; g < G; ++g) dx_ksteps += (m[g] + BK - 1) / BK;
  size_t total = 0;
  for (int g = 0; g < G; ++g) total += (size_t)plan_gc_splits(tokens, r[g], m[g], dx_ksteps) * r[g] * m[g] * sizeof(float);
  return total;
}

inline compact_status_t backward_group(const LaunchInfo& li, int G, const GroupLayer* L, int64_t tokens, int n,
                                       __nv_bfloat16* dX, int64_t lddx, int accumulate, void* workspace,
                                       size_t workspace_bytes) {
  if (G < 1 || G > MAXG) return COMPACT_ERR_INVALID_ARG;
  if (!li.status || !li.sched) return COMPACT_ERR_CUDA;
  for (int g = 0; g < G; ++g)
    if (!tc_shape_ok(tokens, n, L[g].m)) return COMPACT_ERR_SHAPE;
  Params prm;
  memset(&prm, 0, sizeof(prm));
  prm.gen_ring = GEN_NONE;
  int np = 0, slot = 0, dx_ksteps = 0;
  for (int g = 0; g < G; ++g) dx_ksteps += (L[g].m + BK - 1) / BK;
  if (dX) {
    // dX = sum_g dY_g W_g^T: one problem whose K runs over the layers; its items are the longest, so it goes first
    Problem& px = prm.prob[np++];
    px.M = (int)tokens; px.N = n; px.K = dx_ksteps * BK;
    px.a_mode = TMA_KMAJOR; px.b_mode = TMA_KMAJOR; px.epi_mode = EPI_BF16;
    finish_problem(px, 1);
    px.nseg = G;
    int kb = 0;
    for (int g = 0; g < 4; ++g) {
      px.seg_begin[g] = kb;
      if (g < G) kb += (L[g].m + BK - 1) / BK;
    }
    for (int g = 0; g < G; ++g) {
      if (!make_map(&prm.tmA[slot + g], L[g].dY, L[g].m, tokens, L[g].lddy, BK, BM)) return COMPACT_ERR_CUDA;
      if (!make_map(&prm.tmB[slot + g], L[g].W, L[g].m, n, L[g].ldw, BK, px.bn)) return COMPACT_ERR_CUDA;
    }
    if (!make_map(&prm.tmC[slot], dX, n, tokens, lddx, 64, 32)) return COMPACT_ERR_CUDA;
    slot += G;
  }
  size_t ws_off = 0;
  int splits[MAXG];
  bool staged[MAXG];
  size_t part_off[MAXG];
  for (int g = 0; g < G; ++g) {
    const int r = L[g].r, m = L[g].m;
    splits[g] = plan_gc_splits(tokens, r, m, dx_ksteps);
    staged[g] = splits[g] > 1 || accumulate;
    part_off[g] = ws_off;
    ws_off += (size_t)splits[g] * r * m * sizeof(float);
    if (staged[g] && workspace_bytes < ws_off) return COMPACT_ERR_WORKSPACE;
    Problem& pg = prm.prob[np++];
    pg.M = r; pg.N = m; pg.K = (int)tokens;
    pg.a_mode = TMA_MNMAJOR; pg.b_mode = TMA_MNMAJOR; pg.epi_mode = EPI_F32;
    finish_problem(pg, splits[g]);
    splits[g] = pg.splits;
    float* part = (float*)((char*)workspace + part_off[g]);
    if (staged[g]) {
      if (!make_map_f32_3d(&prm.tmC[slot], part, m, r, pg.splits, m, (int64_t)r * m)) return COMPACT_ERR_CUDA;
    } else {
      if (!make_map_f32_3d(&prm.tmC[slot], L[g].Gc, m, r, 1, L[g].ldg, (int64_t)r * L[g].ldg)) return COMPACT_ERR_CUDA;
    }
    pg.a_blocked = L[g].zcols % 64 == 0;
    pg.b_blocked = m % 64 == 0;
    if (pg.a_blocked ? !make_map_blocked(&prm.tmA[slot], L[g].Z, L[g].zcols, tokens, L[g].ldz, BK, 2)
                     : !make_map(&prm.tmA[slot], L[g].Z, L[g].zcols, tokens, L[g].ldz, 64, BK))
      return COMPACT_ERR_CUDA;
    if (pg.b_blocked ? !make_map_blocked(&prm.tmB[slot], L[g].dY, m, tokens, L[g].lddy, BK, pg.bn / 64)
                     : !make_map(&prm.tmB[slot], L[g].dY, m, tokens, L[g].lddy, 64, BK))
      return COMPACT_ERR_CUDA;
    ++slot;
  }
  prm.num_problems = np;
  compact_status_t s = launch(li, prm);
  if (s != COMPACT_OK) return s;
  for (int g = 0; g < G; ++g) {
    if (!staged[g]) continue;
    const int r = L[g].r, m = L[g].m;
    const long long cnt = (long long)r * (m / 4);
    reduce_partials_kernel<<<(unsigned)((cnt + 255) / 256), 256, 0, li.stream>>>(
        (const float*)((char*)workspace + part_off[g]), (long long)r * m, splits[g], L[g].Gc, L[g].ldg, r, m, accumulate);
    (*li.launches)++;
    if (cudaGetLastError() != cudaSuccess) return COMPACT_ERR_CUDA;
  }
  return COMPACT_OK;
}

// Algorithm 3: Adam moments -> N (bf16 scratch), then W <- W - scale * P N with P generated as the A operand.
inline compact_status_t update(const LaunchInfo& li, const ProjectionParams& pp, const simt::AdamScalars& as, int n, int m,
                               int r, __nv_bfloat16* W, int64_t ldw, const float* Gc, int64_t ldg, float* M, float* V,
                               float scale, void* workspace, size_t workspace_bytes) {
  if (!tc_shape_ok(1, n, m)) return COMPACT_ERR_SHAPE;
  if (!li.status || !li.sched) return COMPACT_ERR_CUDA;
  if (workspace_bytes < (size_t)r * m * 2) return COMPACT_ERR_WORKSPACE;
  __nv_bfloat16* Nbuf = (__nv_bfloat16*)workspace;
  const long long cnt = (long long)r * (m / 4);
  adam_moments_bf16_kernel<<<(unsigned)((cnt + 255) / 256), 256, 0, li.stream>>>(Gc, ldg, M, V, Nbuf, r, m, as);
  (*li.launches)++;
  if (cudaGetLastError() != cudaSuccess) return COMPACT_ERR_CUDA;
  Params prm;
  memset(&prm, 0, sizeof(prm));
  prm.key = pp.key;
  prm.num_problems = 1;
  prm.gen_ring = GEN_A;
  Problem& pu = prm.prob[0];
  pu.M = n; pu.N = m; pu.K = r;
  pu.nsub = 1;
  pu.ncol = m > BN_MAX ? 2 : 1;     // the generator is the bound here: one generated tile of P feeds two column blocks
  pu.a_mode = GENERATED; pu.b_mode = TMA_MNMAJOR; pu.epi_mode = EPI_UPDATE_W;
  set_projection(pu, pp);
  pu.scale = scale;
  finish_problem(pu, 1);
  pu.b_blocked = m % 64 == 0;
  if (pu.b_blocked ? !make_map_blocked(&prm.tmB[0], Nbuf, m, r, m, BK, pu.bn / 64) : !make_map(&prm.tmB[0], Nbuf, m, r, m, 64, BK))
    return COMPACT_ERR_CUDA;
  prm.tmA[0] = prm.tmB[0];
  if (!make_map(&prm.tmC[0], W, m, n, ldw, 64, 32)) return COMPACT_ERR_CUDA;
  return launch(li, prm);
}

}  // namespace tc
}  // namespace compact
