// The TMA-fed products of the CompAct layer on pairs of SMs:
//   Y = X W              (Algorithm 1 line 3)
//   Z = X P              (Algorithm 1 line 2; P of the current epoch expanded once per call into scratch that
//                         stays in the L2, so that Z is further columns of the same product as Y)
//   dX = dY W^T          (Algorithm 2 line 2)
//   Gc = Z^T dY          (Algorithm 2 line 1; split over tokens)
// A cluster of two CTAs computes one 256 x 256 tile with tcgen05.mma.cta_group::2: each CTA holds 128 rows of A, half
// (128 columns) of B and 128 rows of the accumulator, and the leader CTA (rank 0) issues the MMAs for both.  Against a
// 256 x 256 tile per single CTA this moves the same bytes per flop into each SM, but the tile takes only 256 of a
// CTA's 512 TMEM columns, so the accumulator is double-buffered and a tile's epilogue runs under the next tile's MMAs;
// and a stage is 32 KB, so six of them (six k-steps) are in flight.
//
// Protocol (per stage s, per accumulator slot a; every barrier exists in both CTAs at the same offset):
//   empty[s]   each CTA's loader waits on its own; the leader's tcgen05.commit arrives on both (multicast)
//   full[s]    only the leader's is used: its loader declares the bytes of both CTAs' copies, and every copy (the
//              neighbour's too) completes on it
//   tfull[a]   each CTA's epilogue waits on its own; the leader's commit arrives on both
//   tempty[a]  only the leader's is used: the epilogue warps of both CTAs arrive on it
// Items are dealt statically: pair p takes items p, p + pairs, ... (both CTAs walk the same list).
#pragma once
#include "tc_kernels.cuh"

namespace compact {
namespace g2 {

using namespace tc;

constexpr int G2_NS = 6;
constexpr int G2_HALF = 128;                         // rows of A, and columns of B, that one CTA holds
constexpr int G2_A_BYTES = G2_HALF * BK * 2;         // 16 KB
constexpr int G2_STAGE_BYTES = 2 * G2_A_BYTES;       // [A | B]
constexpr int G2_RING_BYTES = G2_NS * G2_STAGE_BYTES;
constexpr int G2_EPI_WARPS = 8;
constexpr int G2_THREADS = 32 * (2 + G2_EPI_WARPS);
constexpr int G2_STAGING_OFF = G2_RING_BYTES;
constexpr int G2_BARS_OFF = G2_STAGING_OFF + G2_EPI_WARPS * STAGING_BYTES;
constexpr int G2_NUM_BARS = 2 * G2_NS + 4;
constexpr int G2_SMEM_BYTES = 1024 + G2_BARS_OFF + 8 * G2_NUM_BARS + 32;
static_assert(G2_SMEM_BYTES <= 232448, "shared memory budget");
// Tile order and the L2.  A round of 74 tiles reads its row blocks of A and its column tiles of B; what the next
// round reads again should still be in the L2, which holds 126 MB in two halves and behaves, for data that all SMs
// read, like about half of that.  A problem whose B operand is larger than G2_PANEL_BYTES is walked in column panels
// of at most that size (row block by row block inside a panel: the panel stays, A streams once per panel); the
// forward numbers the Z and Y tiles of a row block together (X is read once for both) while every B operand of
// the run fits G2_ROWS_BYTES.  Measured on 16384 tokens with 48 MB for both: 4096 x 11008 forward 1.242 -> 1.150 ms,
// 11008 x 4096 backward 1.385 -> 1.283 ms (its launch read 2.7 GB from DRAM for 0.6 GB of operands), 4096 x 11008
// backward 1.307 -> 1.292; sizes from 24 to 80 MB give the same within 1 %.
constexpr long long G2_PANEL_BYTES = 48ll << 20;
constexpr long long G2_ROWS_BYTES = 48ll << 20;
constexpr int G2_MAXP = 6;      // Y and Z of up to three layers that share their input

struct G2Problem {
  int M, N, K;                 // C[M x N] = A[M x K] B[K x N]
  int tiles_m, tiles_n, splits, ksteps_total, ksteps_per_split;
  int a_mode, b_mode;          // TMA_KMAJOR or TMA_MNMAJOR
  int a_blocked, b_blocked;    // MN-major operand read through the blocked map (column count a multiple of 64)
  int epi_mode;                // EPI_BF16, EPI_UPDATE_W (C += -scale * acc) or EPI_F32 (3-D map [split][M][N])
  int map_base;                // index of the problem's tensor maps (A and B: + segment; C: this one)
  int nseg;                    // > 1: K runs over this many operand pairs laid end to end (dX of a group of layers)
  int seg_begin[4];            // first k-step of each segment
  int tile_begin;
  int panel_cols;              // > 0 (and splits == 1): tiles are numbered panel by panel of this many column tiles, and
                               // row block by row block inside a panel, so that a panel of B stays in the L2
  float scale;                 // bf16 epilogues: the accumulator is multiplied by this before it is rounded (1: exact)
};

#ifndef G2_PDL
#define G2_PDL 1
#endif

struct alignas(64) G2Params {
  CUtensorMap tmA[G2_MAXP];
  CUtensorMap tmB[G2_MAXP];
  CUtensorMap tmC[G2_MAXP];
  G2Problem prob[G2_MAXP];
  int num_problems;
  int total_tiles;
  int by_rows;                 // > 0: the problems share A and M, and every run of this many problems is numbered row
                               // block by row block across its problems (tile_begin: a problem's first column tile in its run)
  int run_begin[G2_MAXP / 2 + 1];   // by_rows: first tile of each run
  int run_cols[G2_MAXP / 2];        // by_rows: column tiles of a run's problems together
  int early;                   // host only: launch behind the previous kernel of the stream without waiting for its end
  unsigned int* status;
};

// Copy of a tile into this CTA's shared memory whose bytes complete on a barrier of the pair's leader CTA.
__device__ __forceinline__ void tma2_load_2d(uint32_t dst, const CUtensorMap* map, uint32_t leader_bar, int x, int y) {
  asm volatile(
      "cp.async.bulk.tensor.2d.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4}], [%2];" ::"r"(dst),
      "l"(map), "r"(leader_bar), "r"(x), "r"(y)
      : "memory");
}
__device__ __forceinline__ void tma2_load_3d(uint32_t dst, const CUtensorMap* map, uint32_t leader_bar, int x, int y, int z) {
  asm volatile(
      "cp.async.bulk.tensor.3d.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5}], [%2];" ::"r"(dst),
      "l"(map), "r"(leader_bar), "r"(x), "r"(y), "r"(z)
      : "memory");
}
__device__ __forceinline__ void tmem_alloc2(uint32_t dst_smem, uint32_t ncols) {
  asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(dst_smem), "r"(ncols) : "memory");
}
__device__ __forceinline__ void tmem_relinquish2() {
  asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_dealloc2(uint32_t taddr, uint32_t ncols) {
  asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(taddr), "r"(ncols) : "memory");
}
// D[256 x N] (+)= A[256 x 16] B[16 x N] over the pair: both CTAs' operands sit at these offsets of their shared memory
__device__ __forceinline__ void umma2_bf16(uint32_t d_tmem, uint32_t a_lo, uint32_t a_hi, uint32_t b_lo, uint32_t b_hi,
                                           uint32_t idesc, uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t.reg .b64 da, db;\n\t"
      "mov.b64 da, {%1, %2};\n\t"
      "mov.b64 db, {%3, %4};\n\t"
      "setp.ne.b32 p, %6, 0;\n\t"
      "tcgen05.mma.cta_group::2.kind::f16 [%0], da, db, %5, p;\n\t}" ::"r"(d_tmem),
      "r"(a_lo), "r"(a_hi), "r"(b_lo), "r"(b_hi), "r"(idesc), "r"(accumulate)
      : "memory");
}
// arrives, once the pair's MMAs issued so far are done, on the barrier at this offset in every CTA of `mask`
__device__ __forceinline__ void umma2_commit_mc(uint32_t bar, uint16_t mask) {
  asm volatile("tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.multicast::cluster.b64 [%0], %1;" ::"r"(bar),
               "h"(mask)
               : "memory");
}
__device__ __forceinline__ void mbar_arrive_cluster(uint32_t cluster_addr) {
  asm volatile("mbarrier.arrive.shared::cluster.b64 _, [%0];" ::"r"(cluster_addr) : "memory");
}

struct G2Tile {
  int prob, m0, n0, k_begin, k_end, split;
};

__device__ __forceinline__ G2Tile g2_decode(const G2Params& prm, int tile) {
  G2Tile t;
  t.prob = 0;
  if (prm.by_rows) {
    // consecutive tiles read the same rows of A: (row block, column tile over the problems side by side)
    int q = 0;
#pragma unroll
    for (int i = 1; i < G2_MAXP / 2; ++i)
      if (i * prm.by_rows < prm.num_problems && tile >= prm.run_begin[i]) q = i;
    const int local = tile - prm.run_begin[q];
    const int mb = local / prm.run_cols[q], c = local - mb * prm.run_cols[q];
    t.prob = q * prm.by_rows;
#pragma unroll
    for (int i = 1; i < G2_MAXP; ++i)
      if (i < prm.by_rows && c >= prm.prob[q * prm.by_rows + i].tile_begin) t.prob = q * prm.by_rows + i;
    const G2Problem& p = prm.prob[t.prob];
    t.split = 0;
    t.m0 = mb * 2 * G2_HALF;
    t.n0 = (c - p.tile_begin) * 2 * G2_HALF;
    t.k_begin = 0;
    t.k_end = p.ksteps_total;
    return t;
  }
#pragma unroll
  for (int i = 1; i < G2_MAXP; ++i)
    if (i < prm.num_problems && tile >= prm.prob[i].tile_begin) t.prob = i;
  const G2Problem& p = prm.prob[t.prob];
  int local = tile - p.tile_begin;
  if (p.panel_cols > 0) {
    const int per_panel = p.tiles_m * p.panel_cols;
    const int panel = local / per_panel;
    local -= panel * per_panel;
    const int pc = min(p.panel_cols, p.tiles_n - panel * p.panel_cols);
    const int mb = local / pc;
    t.split = 0;
    t.m0 = mb * 2 * G2_HALF;
    t.n0 = (panel * p.panel_cols + (local - mb * pc)) * 2 * G2_HALF;
    t.k_begin = 0;
    t.k_end = p.ksteps_total;
    return t;
  }
  const int nb = local % p.tiles_n;
  local /= p.tiles_n;
  const int mb = local % p.tiles_m;
  t.split = local / p.tiles_m;
  t.m0 = mb * 2 * G2_HALF;
  t.n0 = nb * 2 * G2_HALF;
  t.k_begin = t.split * p.ksteps_per_split;
  t.k_end = min(p.ksteps_total, t.k_begin + p.ksteps_per_split);
  return t;
}

// Warp roles (in each CTA of the pair): 0 = loader of this CTA's A rows and B columns; 1 = owner of TMEM, and in the
// leader CTA the MMA issuer; 2..9 = epilogue of this CTA's 128 rows of the tile.
__global__ void __launch_bounds__(G2_THREADS, 1) compact_gemm2_kernel(const __grid_constant__ G2Params prm) {
  extern __shared__ uint8_t smem_raw[];
  const uint32_t smem_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
  uint8_t* smem_gen = smem_raw + (smem_base - smem_u32(smem_raw));
  const uint32_t staging = smem_base + G2_STAGING_OFF;
  const uint32_t bars = smem_base + G2_BARS_OFF;
  auto full_bar = [&](int s) { return bars + 8u * s; };
  auto empty_bar = [&](int s) { return bars + 8u * (G2_NS + s); };
  auto tfull_bar = [&](int a) { return bars + 8u * (2 * G2_NS + a); };
  auto tempty_bar = [&](int a) { return bars + 8u * (2 * G2_NS + 2 + a); };
  uint8_t* tail = smem_gen + G2_BARS_OFF + 8 * G2_NUM_BARS;
  volatile uint32_t* tmem_slot = reinterpret_cast<volatile uint32_t*>(tail);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tail + 8);

  const int warp = threadIdx.x >> 5;
  const int lane = threadIdx.x & 31;
  const uint32_t crank = cluster_ctarank();
  const bool leader = crank == 0;
  const int pair_id = (int)(blockIdx.x >> 1);
  const int npairs = (int)(gridDim.x >> 1);

  if (threadIdx.x == 0) {
    for (int s = 0; s < G2_NS; ++s) {
      mbar_init(full_bar(s), 1);          // the leader's loader
      mbar_init(empty_bar(s), 1);         // the leader's commit
    }
    for (int a = 0; a < 2; ++a) {
      mbar_init(tfull_bar(a), 1);                     // the leader's commit
      mbar_init(tempty_bar(a), 2 * G2_EPI_WARPS);     // the epilogue warps of both CTAs
    }
    *abort_flag = 0;
    fence_barrier_init();
    fence_proxy_async_smem();
  }
  if (warp == 1) {
    tmem_alloc2(smem_u32((const void*)tmem_slot), 512);
    tmem_relinquish2();
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  cluster_sync_all();                     // both CTAs' barriers and TMEM exist before anything crosses
#if G2_PDL
  // Launched early (programmatic stream serialization) behind the small kernel that prepares an operand: everything
  // above ran while that kernel was finishing; nothing below touches global memory before it has completed.
  asm volatile("griddepcontrol.wait;" ::: "memory");
#endif
  const uint32_t tmem_base = *tmem_slot;
  const uint32_t leader_bars = map_to_cta(bars, 0u);

  if (warp == 0) {
    // ------------------------------ loader ---------------------------------------
    Ring r = {0, 0u};
    bool ok = true;
    for (int tile = pair_id; tile < prm.total_tiles && ok; tile += npairs) {
      const G2Tile t = g2_decode(prm, tile);
      const G2Problem& p = prm.prob[t.prob];
      const int m0 = t.m0 + (int)crank * G2_HALF, n0 = t.n0 + (int)crank * G2_HALF;
      // everything the k loop needs sits in registers before it starts: the loop is one wait and two copies
      const bool multi = p.nseg > 1;
      const int a_mode = p.a_mode, b_mode = p.b_mode, a_blocked = p.a_blocked, b_blocked = p.b_blocked;
      const int seg1 = multi ? p.seg_begin[1] : 0x7fffffff, seg2 = multi ? p.seg_begin[2] : 0x7fffffff;
      const CUtensorMap* const mapA0 = &prm.tmA[p.map_base];
      const CUtensorMap* const mapB0 = &prm.tmB[p.map_base];
      for (int ks = t.k_begin; ks < t.k_end; ++ks, ring_next(r, G2_NS)) {
        if (!(ok = __all_sync(0xffffffffu, mbar_wait(empty_bar(r.s), r.ph ^ 1u, abort_flag, prm.status)))) break;
        if (elect_one()) {
          const int seg = (ks >= seg1) + (ks >= seg2);
          const CUtensorMap* mapA = mapA0 + seg;
          const CUtensorMap* mapB = mapB0 + seg;
          const int k0 = (ks - (seg == 0 ? 0 : (seg == 1 ? seg1 : seg2))) * BK;
          const uint32_t fb = leader_bars + 8u * r.s;                      // the leader's full barrier of this stage
          if (leader) mbar_arrive_expect_tx(full_bar(r.s), 2 * G2_STAGE_BYTES);
          const uint32_t dstA = smem_base + (uint32_t)r.s * G2_STAGE_BYTES, dstB = dstA + G2_A_BYTES;
          if (a_mode == TMA_KMAJOR) {
            tma2_load_2d(dstA, mapA, fb, k0, m0);
          } else if (a_blocked) {
            tma2_load_3d(dstA, mapA, fb, 0, k0, m0 >> 6);
          } else {
            tma2_load_2d(dstA, mapA, fb, m0, k0);
            tma2_load_2d(dstA + 8192, mapA, fb, m0 + 64, k0);
          }
          if (b_mode == TMA_KMAJOR) {
            tma2_load_2d(dstB, mapB, fb, k0, n0);
          } else if (b_blocked) {
            tma2_load_3d(dstB, mapB, fb, 0, k0, n0 >> 6);
          } else {
            tma2_load_2d(dstB, mapB, fb, n0, k0);
            tma2_load_2d(dstB + 8192, mapB, fb, n0 + 64, k0);
          }
        }
        __syncwarp();
      }
    }
  } else if (warp == 1) {
    // ------------------------------ MMA issuer (leader CTA) ----------------------
    if (leader) {
      Ring r = {0, 0u};
      bool ok = true;
      int slot = 0;
      uint32_t slot_phase = 0;
      const uint32_t ring_lo = (smem_base >> 4) & 0x3FFFu;
      const uint32_t lbo = (8192u >> 4) << 16, one = 1u << 16;
      for (int tile = pair_id; tile < prm.total_tiles && ok; tile += npairs) {
        const G2Tile t = g2_decode(prm, tile);
        const G2Problem& p = prm.prob[t.prob];
        const bool a_mn = p.a_mode == TMA_MNMAJOR, b_mn = p.b_mode == TMA_MNMAJOR;
        // M = 256 over the pair, N = 256
        const uint32_t idesc = (1u << 4) | (1u << 7) | (1u << 10) | ((a_mn ? 1u : 0u) << 15) | ((b_mn ? 1u : 0u) << 16) |
                               ((uint32_t)(256 >> 3) << 17) | ((uint32_t)(256 >> 4) << 24);
        const uint32_t a_step = a_mn ? (2048u >> 4) : (32u >> 4), b_step = b_mn ? (2048u >> 4) : (32u >> 4);
        const uint32_t a_flags = a_mn ? lbo : one, b_flags = b_mn ? lbo : one;
        if (!(ok = __all_sync(0xffffffffu, mbar_wait(tempty_bar(slot), slot_phase ^ 1u, abort_flag, prm.status)))) break;
        tc_fence_after();
        const uint32_t d = tmem_base + (uint32_t)slot * 256;
        for (int ks = t.k_begin; ks < t.k_end && ok; ++ks, ring_next(r, G2_NS)) {
          if (!(ok = __all_sync(0xffffffffu, mbar_wait(full_bar(r.s), r.ph, abort_flag, prm.status)))) break;
          tc_fence_after();
          if (elect_one()) {
            const uint32_t base = ring_lo + (((uint32_t)r.s * G2_STAGE_BYTES) >> 4);
            const uint32_t a_lo = base | a_flags, b_lo = (base + (G2_A_BYTES >> 4)) | b_flags;
            umma2_bf16(d, a_lo, DESC_HI, b_lo, DESC_HI, idesc, ks > t.k_begin ? 1u : 0u);
            umma2_bf16(d, a_lo + a_step, DESC_HI, b_lo + b_step, DESC_HI, idesc, 1u);
            umma2_bf16(d, a_lo + 2 * a_step, DESC_HI, b_lo + 2 * b_step, DESC_HI, idesc, 1u);
            umma2_bf16(d, a_lo + 3 * a_step, DESC_HI, b_lo + 3 * b_step, DESC_HI, idesc, 1u);
            umma2_commit_mc(empty_bar(r.s), (uint16_t)3);          // the stage goes back to both loaders
          }
          __syncwarp();
        }
        if (!ok) break;
        if (elect_one()) umma2_commit_mc(tfull_bar(slot), (uint16_t)3);   // the accumulator is complete in both CTAs
        __syncwarp();
        if (++slot == 2) { slot = 0; slot_phase ^= 1u; }
      }
    }
  } else {
    // ------------------------------ epilogue ------------------------------------
    // This CTA's 128 rows of the tile: TMEM -> registers -> 128B-swizzled staging tile -> TMA store.
    const int q = warp & 3;                 // TMEM lane quarter this warp may read
    const int eset = (warp - 2) >> 2;       // the two sets take alternate chunks
    const uint32_t stg = staging + (warp - 2) * STAGING_BYTES;
    uint8_t* stg_gen = smem_gen + G2_STAGING_OFF + (warp - 2) * STAGING_BYTES;
    const uint32_t leader_tempty = leader_bars + 8u * (2 * G2_NS + 2);
    const int sw = lane & 7;
    int slot = 0;
    uint32_t slot_phase = 0;
    bool ok = true;
    for (int tile = pair_id; tile < prm.total_tiles && ok; tile += npairs) {
      const G2Tile t = g2_decode(prm, tile);
      const G2Problem& p = prm.prob[t.prob];
      const CUtensorMap* mapC = &prm.tmC[p.map_base];
      if (!(ok = mbar_wait(tfull_bar(slot), slot_phase, abort_flag, prm.status))) break;
      tc_fence_after();
      const int row0 = t.m0 + (int)crank * G2_HALF + q * 32;
      const uint32_t tcol = tmem_base + ((uint32_t)(q * 32) << 16) + (uint32_t)slot * 256;
      const int epi_mode = p.epi_mode, pM = p.M, pN = p.N;
      const float sc = epi_mode == EPI_UPDATE_W ? -p.scale : p.scale;
      const int cw = epi_mode == EPI_F32 ? 32 : 64;
      for (int ci = eset; ci < 256 / cw && row0 < pM; ci += 2) {
        const int col = t.n0 + ci * cw;
        if (col >= pN) break;
        if (epi_mode == EPI_BF16 || epi_mode == EPI_UPDATE_W) {
          // The update stages -(eta alpha) (P N) and lets the TMA unit add it to W (Algorithm 3 line 9).
          uint32_t o[32];
#pragma unroll
          for (int h = 0; h < 2; ++h) {
            uint32_t v[32];
            tmem_ld32(tcol + ci * cw + 32 * h, v);
            tmem_ld_wait();
#pragma unroll
            for (int j = 0; j < 16; ++j) o[16 * h + j] = pack_bf16x2(__uint_as_float(v[2 * j]) * sc, __uint_as_float(v[2 * j + 1]) * sc);
          }
          if (lane == 0) tma_store_wait_read();          // the previous store has read the staging tile
          __syncwarp();
#pragma unroll
          for (int j = 0; j < 8; ++j)
            *reinterpret_cast<uint4*>(stg_gen + lane * 128 + ((j ^ sw) << 4)) = make_uint4(o[4 * j], o[4 * j + 1], o[4 * j + 2], o[4 * j + 3]);
          fence_proxy_async_smem();
          __syncwarp();
          if (lane == 0) {
            if (epi_mode == EPI_UPDATE_W) tma_reduce_add_2d(mapC, stg, col, row0);
            else tma_store_2d(mapC, stg, col, row0);
            tma_store_commit();
          }
        } else {
          uint32_t v[32];
          tmem_ld32(tcol + ci * cw, v);
          tmem_ld_wait();
          if (lane == 0) tma_store_wait_read();
          __syncwarp();
#pragma unroll
          for (int j = 0; j < 8; ++j)
            *reinterpret_cast<uint4*>(stg_gen + lane * 128 + ((j ^ sw) << 4)) = make_uint4(v[4 * j], v[4 * j + 1], v[4 * j + 2], v[4 * j + 3]);
          fence_proxy_async_smem();
          __syncwarp();
          if (lane == 0) {
            tma_store_3d(mapC, stg, col, row0, t.split);
            tma_store_commit();
          }
        }
      }
      tc_fence_before();
      __syncwarp();
      if (lane == 0) {
        if (leader) mbar_arrive(tempty_bar(slot));
        else mbar_arrive_cluster(leader_tempty + 8u * slot);
      }
      if (++slot == 2) { slot = 0; slot_phase ^= 1u; }
    }
    if (lane == 0) tma_store_wait_all();
  }

  tc_fence_before();
  __syncthreads();
  cluster_sync_all();                     // neither CTA frees TMEM, or leaves, while the pair may still use or signal it
  if (warp == 1) {
    tc_fence_after();
    tmem_dealloc2(tmem_base, 512);
  }
}

// --------------------------------------------------------------------------------------
// Host side
// --------------------------------------------------------------------------------------
inline void g2_finish(G2Problem& p, int splits_wanted) {
  p.tiles_m = (p.M + 2 * G2_HALF - 1) / (2 * G2_HALF);
  p.tiles_n = (p.N + 2 * G2_HALF - 1) / (2 * G2_HALF);
  p.ksteps_total = (p.K + BK - 1) / BK;
  int s = splits_wanted < 1 ? 1 : splits_wanted;
  if (s > p.ksteps_total) s = p.ksteps_total;
  p.ksteps_per_split = (p.ksteps_total + s - 1) / s;
  p.splits = (p.ksteps_total + p.ksteps_per_split - 1) / p.ksteps_per_split;
  if (p.scale == 0.f) p.scale = 1.f;
  // A B operand that does not fit the L2 next to the stream of A goes through it panel by panel.
  p.panel_cols = 0;
  const size_t b_bytes = (size_t)p.K * (size_t)p.N * sizeof(__nv_bfloat16);
  if (p.splits == 1 && b_bytes > (size_t)G2_PANEL_BYTES) {
    const int npanels = (int)((b_bytes + G2_PANEL_BYTES - 1) / G2_PANEL_BYTES);
    p.panel_cols = (p.tiles_n + npanels - 1) / npanels;
    // never narrower than a round of tiles is tall (74 tiles = 9 x 8): with a long K even such a panel exceeds the
    // L2, and a narrower one only streams A more often (dX of the gate/up group, K = 22016: 2.67 ms with panels of
    // four column tiles against 2.56 without panels)
    if (p.panel_cols < 8) p.panel_cols = 8;
    if (p.panel_cols >= p.tiles_n) p.panel_cols = 0;
  }
}

inline compact_status_t g2_launch(const LaunchInfo& li, G2Params& prm) {
  static std::atomic<bool> attr_set[64];
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) { cudaGetLastError(); return COMPACT_ERR_CUDA; }
  if (!attr_set[dev].load(std::memory_order_acquire)) {
    if (cudaFuncSetAttribute(compact_gemm2_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, G2_SMEM_BYTES) != cudaSuccess) {
      cudaGetLastError();
      return COMPACT_ERR_CUDA;
    }
    attr_set[dev].store(true, std::memory_order_release);
  }
  for (int i = 0; i < prm.num_problems; ++i) {
    G2Problem& p = prm.prob[i];
    if (p.nseg < 1) { p.nseg = 1; p.map_base = i; }      // a plain problem: its own maps, one segment
  }
  int t = 0;
  if (prm.by_rows) {
    for (int q = 0; q * prm.by_rows < prm.num_problems; ++q) {
      int cols = 0;
      for (int i = q * prm.by_rows; i < (q + 1) * prm.by_rows && i < prm.num_problems; ++i) {
        prm.prob[i].tile_begin = cols;
        cols += prm.prob[i].tiles_n;
      }
      prm.run_begin[q] = t;
      prm.run_cols[q] = cols;
      t += cols * prm.prob[0].tiles_m;
    }
  } else {
    for (int i = 0; i < prm.num_problems; ++i) {
      prm.prob[i].tile_begin = t;
      t += prm.prob[i].tiles_m * prm.prob[i].tiles_n * prm.prob[i].splits;
    }
  }
  prm.total_tiles = t;
  prm.status = li.status;
  const int pairs = t < NUM_SMS / 2 ? t : NUM_SMS / 2;
  cudaLaunchConfig_t cfg;
  memset(&cfg, 0, sizeof(cfg));
  cfg.gridDim = dim3((unsigned)(2 * pairs), 1, 1);
  cfg.blockDim = dim3((unsigned)G2_THREADS, 1, 1);
  cfg.dynamicSmemBytes = G2_SMEM_BYTES;
  cfg.stream = li.stream;
  cudaLaunchAttribute attr;
  attr.id = cudaLaunchAttributeClusterDimension;
  attr.val.clusterDim.x = 2;
  attr.val.clusterDim.y = 1;
  attr.val.clusterDim.z = 1;
  cudaLaunchAttribute attrs[2];
  attrs[0] = attr;
  cfg.attrs = attrs;
  cfg.numAttrs = 1;
#if G2_PDL
  if (prm.early) {
    attrs[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attrs[1].val.programmaticStreamSerializationAllowed = 1;
    cfg.numAttrs = 2;
  }
#endif
  const cudaError_t e = cudaLaunchKernelEx(&cfg, compact_gemm2_kernel, prm);
  (*li.launches)++;
  if (e != cudaSuccess) { cudaGetLastError(); return COMPACT_ERR_CUDA; }
  return cudaGetLastError() == cudaSuccess ? COMPACT_OK : COMPACT_ERR_CUDA;
}

// Y = X W (Algorithm 1 line 3): A = X (K-major), B = W (MN-major).
inline compact_status_t g2_forward_y(const LaunchInfo& li, int64_t tokens, int n, int m, const __nv_bfloat16* X, int64_t ldx,
                                     const __nv_bfloat16* W, int64_t ldw, __nv_bfloat16* Y, int64_t ldy) {
  if (!tc_shape_ok(tokens, n, m)) return COMPACT_ERR_SHAPE;
  if (!li.status) return COMPACT_ERR_CUDA;
  G2Params prm;
  memset(&prm, 0, sizeof(prm));
  prm.num_problems = 1;
  G2Problem& py = prm.prob[0];
  py.M = (int)tokens; py.N = m; py.K = n;
  py.a_mode = TMA_KMAJOR; py.b_mode = TMA_MNMAJOR; py.epi_mode = EPI_BF16;
  py.b_blocked = m % 64 == 0;
  g2_finish(py, 1);
  if (!make_map(&prm.tmA[0], X, n, tokens, ldx, BK, G2_HALF)) return COMPACT_ERR_CUDA;
  if (py.b_blocked ? !make_map_blocked(&prm.tmB[0], W, m, n, ldw, BK, G2_HALF / 64) : !make_map(&prm.tmB[0], W, m, n, ldw, 64, BK))
    return COMPACT_ERR_CUDA;
  if (!make_map(&prm.tmC[0], Y, m, tokens, ldy, 64, 32)) return COMPACT_ERR_CUDA;
  return g2_launch(li, prm);
}

// --------------------------------------------------------------------------------------
// The projection of one epoch, written out (Section 3.3: P is a function of the seed, the layer and the epoch,
// so it can be rebuilt wherever it is needed).  The forward of a long batch uses every entry of P once per
// 256 tokens; building the n x r entries once per call (a few microseconds; at most some tens of MB, which
// stay in the L2 while the product runs) and reading them with the TMA unit like any other operand costs far
// less than building every tile again for every block of tokens.  The scratch is the caller's; nothing of it
// is kept between calls.
// --------------------------------------------------------------------------------------
// Pitch of the expanded projection in elements: the row of Z rounded up to whole 64-column blocks.
inline int64_t expanded_ld(int zcols) { return ((int64_t)zcols + 63) / 64 * 64; }
inline size_t expanded_bytes(int n, int zcols) { return (size_t)n * (size_t)expanded_ld(zcols) * sizeof(__nv_bfloat16); }

struct ExpandArgs {
  PhiloxKey key;
  uint32_t layer_hi, layer_lo, epoch;
  int n, r, sparse_s, groups;      // groups: eight-entry groups per row of the scratch (its pitch / 8)
  float neg2ln2_over_r;
  __nv_bfloat16* P;
};

// Gaussian projection: a thread writes eight consecutive entries of a row (one Philox call); columns from r to
// the pitch are zeros.  This is block `block` of `nblocks` blocks of 256 threads.
__device__ __forceinline__ void expand_gaussian_blocks(const ExpandArgs& a, int block, int nblocks) {
  const PhiloxKey& key = a.key;
  const uint32_t layer_hi = a.layer_hi, layer_lo = a.layer_lo, epoch = a.epoch;
  const int n = a.n, r = a.r, groups = a.groups;
  const float neg2ln2_over_r = a.neg2ln2_over_r;
  __nv_bfloat16* __restrict__ P = a.P;
  const long long total = (long long)n * groups;
  for (long long task = (long long)block * 256 + threadIdx.x; task < total; task += (long long)nblocks * 256) {
    const int i = (int)(task / groups), g = (int)(task - (long long)i * groups);
    const uint4 val = g * 8 < r ? projection8_bf16(key, layer_hi, layer_lo, epoch, n, r, neg2ln2_over_r, i, g * 8)
                                : make_uint4(0u, 0u, 0u, 0u);
    *reinterpret_cast<uint4*>(P + ((long long)i * groups + g) * 8) = val;
  }
}

// Sparse projection: the integer counts (the product's epilogue applies 1 / sqrt(s)).  A warp owns a row: it
// clears it, then lane 0 adds the signs of the row's terms one after another, so that terms that hash to the
// same column add without a race.
__device__ __forceinline__ void expand_sparse_blocks(const ExpandArgs& a, int block, int nblocks) {
  const PhiloxKey& key = a.key;
  const uint32_t layer_hi = a.layer_hi, layer_lo = a.layer_lo, epoch = a.epoch;
  const int n = a.n, r = a.r, s = a.sparse_s, groups = a.groups;
  __nv_bfloat16* __restrict__ P = a.P;
  const int lane = threadIdx.x & 31;
  const int warps = nblocks * 8;
  for (int i = block * 8 + (int)(threadIdx.x >> 5); i < n; i += warps) {
    __nv_bfloat16* row = P + (long long)i * groups * 8;
    for (int g = lane; g < groups; g += 32) reinterpret_cast<uint4*>(row)[g] = make_uint4(0u, 0u, 0u, 0u);
    __syncwarp();
    if (lane == 0) {
      for (int q = 0; 4 * q < s; ++q) {
        const uint4 x = sparse_words4((uint32_t)q, (uint32_t)i, epoch, layer_hi, layer_lo, key);
        const uint32_t w[4] = {x.x, x.y, x.z, x.w};
#pragma unroll
        for (int l = 0; l < 4; ++l) {
          if (4 * q + l < s) {
            const int c = sparse_col(w[l], r);
            row[c] = __float2bfloat16_rn(__bfloat162float(row[c]) + sparse_sign(w[l]));
          }
        }
      }
    }
    __syncwarp();
  }
}

__global__ void __launch_bounds__(256) expand_projection_kernel(const __grid_constant__ ExpandArgs a) {
#if G2_PDL
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
#endif
  if (a.sparse_s > 0) expand_sparse_blocks(a, (int)blockIdx.x, (int)gridDim.x);
  else expand_gaussian_blocks(a, (int)blockIdx.x, (int)gridDim.x);
}

// The update's two preparations in one launch: Algorithm 3 lines 1-5 (moments in place, N in bf16) and P written out.
// Neither reads what the other writes; the Adam blocks are bound by memory, the expansion by instruction issue, so
// their blocks alternate and the two run side by side.
__global__ void __launch_bounds__(256) adam_and_expand_kernel(const float* __restrict__ Gc, long long ldg, float* __restrict__ Mo,
                                                              float* __restrict__ Vo, __nv_bfloat16* __restrict__ Nout, int r, int m,
                                                              const __grid_constant__ simt::AdamScalars as, int adam_blocks,
                                                              const __grid_constant__ ExpandArgs a) {
#if G2_PDL
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
#endif
  const int b = (int)blockIdx.x, expand_blocks = (int)gridDim.x - adam_blocks;
  const int paired = 2 * (adam_blocks < expand_blocks ? adam_blocks : expand_blocks);
  bool is_adam;
  int idx;
  if (b < paired) { is_adam = (b & 1) == 0; idx = b >> 1; }
  else { is_adam = adam_blocks > expand_blocks; idx = b - paired / 2; }
  if (is_adam) adam_moments_bf16_at((long long)idx * 256 + threadIdx.x, Gc, ldg, Mo, Vo, Nout, r, m, as);
  else if (a.sparse_s > 0) expand_sparse_blocks(a, idx, expand_blocks);
  else expand_gaussian_blocks(a, idx, expand_blocks);
}

inline ExpandArgs make_expand_args(const ProjectionParams& pp, int zcols, __nv_bfloat16* P) {
  ExpandArgs a;
  a.key = pp.key; a.layer_hi = pp.layer_hi; a.layer_lo = pp.layer_lo; a.epoch = pp.epoch;
  a.n = pp.n; a.r = pp.r; a.sparse_s = pp.sparse_s; a.groups = (int)(expanded_ld(zcols) / 8);
  a.neg2ln2_over_r = pp.neg2ln2_over_r; a.P = P;
  return a;
}
inline unsigned expand_blocks_for(const ExpandArgs& a) {
  const long long threads = a.sparse_s > 0 ? (long long)a.n * 32 : (long long)a.n * a.groups;
  const long long blocks = (threads + 255) / 256;
  return (unsigned)(blocks < 8 * NUM_SMS ? blocks : 8 * NUM_SMS);
}

inline compact_status_t expand_projection(const LaunchInfo& li, const ProjectionParams& pp, int zcols, __nv_bfloat16* P) {
  const ExpandArgs a = make_expand_args(pp, zcols, P);
  expand_projection_kernel<<<expand_blocks_for(a), 256, 0, li.stream>>>(a);
  (*li.launches)++;
  return cudaGetLastError() == cudaSuccess ? COMPACT_OK : COMPACT_ERR_CUDA;
}

// Algorithm 1 for G layers that share their input (G = 1: one layer): every layer's P is expanded into its part of
// the scratch, then one launch computes Z_g = X P_g and Y_g = X W_g, row block by row block of X.
struct G2Layer {
  ProjectionParams pp;
  int m, zcols;
  const __nv_bfloat16* W; int64_t ldw;
  __nv_bfloat16* Y; int64_t ldy;
  __nv_bfloat16* Z; int64_t ldz;
};

inline size_t g2_forward_scratch_bytes(int G, const G2Layer* L) {
  size_t b = 0;
  for (int g = 0; g < G; ++g) b += (expanded_bytes(L[g].pp.n, L[g].zcols) + 255) / 256 * 256;
  return b;
}

inline compact_status_t g2_forward(const LaunchInfo& li, int G, const G2Layer* L, int64_t tokens, int n, const __nv_bfloat16* X,
                                   int64_t ldx, void* scratch) {
  if (G < 1 || 2 * G > G2_MAXP) return COMPACT_ERR_INVALID_ARG;
  if (!li.status) return COMPACT_ERR_CUDA;
  for (int g = 0; g < G; ++g)
    if (!tc_shape_ok(tokens, n, L[g].m)) return COMPACT_ERR_SHAPE;
  G2Params prm;
  memset(&prm, 0, sizeof(prm));
  prm.num_problems = 2 * G;
  char* at = (char*)scratch;
  for (int g = 0; g < G; ++g) {
    __nv_bfloat16* P = (__nv_bfloat16*)at;
    at += (expanded_bytes(n, L[g].zcols) + 255) / 256 * 256;
    const compact_status_t s = expand_projection(li, L[g].pp, L[g].zcols, P);
    if (s != COMPACT_OK) return s;
    const int64_t ldp = expanded_ld(L[g].zcols);
    const int iz = 2 * g, iy = 2 * g + 1;
    G2Problem& pz = prm.prob[iz];
    pz.M = (int)tokens; pz.N = L[g].zcols; pz.K = n;
    pz.a_mode = TMA_KMAJOR; pz.b_mode = TMA_MNMAJOR; pz.epi_mode = EPI_BF16;
    pz.b_blocked = 1;
    pz.scale = L[g].pp.inv_sqrt_s;
    g2_finish(pz, 1);
    if (!make_map(&prm.tmA[iz], X, n, tokens, ldx, BK, G2_HALF)) return COMPACT_ERR_CUDA;
    if (!make_map_blocked(&prm.tmB[iz], P, ldp, n, ldp, BK, G2_HALF / 64)) return COMPACT_ERR_CUDA;
    if (!make_map(&prm.tmC[iz], L[g].Z, L[g].zcols, tokens, L[g].ldz, 64, 32)) return COMPACT_ERR_CUDA;
    G2Problem& py = prm.prob[iy];
    py.M = (int)tokens; py.N = L[g].m; py.K = n;
    py.a_mode = TMA_KMAJOR; py.b_mode = TMA_MNMAJOR; py.epi_mode = EPI_BF16;
    py.b_blocked = L[g].m % 64 == 0;
    g2_finish(py, 1);
    prm.tmA[iy] = prm.tmA[iz];
    if (py.b_blocked ? !make_map_blocked(&prm.tmB[iy], L[g].W, L[g].m, n, L[g].ldw, BK, G2_HALF / 64)
                     : !make_map(&prm.tmB[iy], L[g].W, L[g].m, n, L[g].ldw, 64, BK))
      return COMPACT_ERR_CUDA;
    if (!make_map(&prm.tmC[iy], L[g].Y, L[g].m, tokens, L[g].ldy, 64, 32)) return COMPACT_ERR_CUDA;
  }
  // Row block by row block, X is read from DRAM once instead of once per problem -- as long as the B operands
  // (every W and P of the run, which each round of tiles walks in full) stay in the L2 beside it.
  // A group of layers whose operands together are too large runs layer after layer, each by rows if it fits.
  const size_t fits = (size_t)G2_ROWS_BYTES;
  size_t all = 0, largest = 0;
  for (int g = 0; g < G; ++g) {
    const size_t b = (size_t)n * (size_t)(L[g].m + expanded_ld(L[g].zcols)) * sizeof(__nv_bfloat16);
    all += b;
    largest = b > largest ? b : largest;
  }
  prm.by_rows = all <= fits ? 2 * G : (largest <= fits ? 2 : 0);
  prm.early = 1;
  return g2_launch(li, prm);
}

// Z = X P alone (Algorithm 1 line 2, for the backward that recomputes it): P written out into `scratch`
// (expanded_bytes(n, zcols)), then one product.
inline compact_status_t g2_project(const LaunchInfo& li, const ProjectionParams& pp, int64_t tokens, const __nv_bfloat16* X,
                                   int64_t ldx, __nv_bfloat16* Z, int64_t ldz, int zcols, void* scratch) {
  const int n = pp.n;
  if (!tc_shape_ok(tokens, n, 8)) return COMPACT_ERR_SHAPE;
  if (!li.status) return COMPACT_ERR_CUDA;
  __nv_bfloat16* P = (__nv_bfloat16*)scratch;
  const compact_status_t s = expand_projection(li, pp, zcols, P);
  if (s != COMPACT_OK) return s;
  const int64_t ldp = expanded_ld(zcols);
  G2Params prm;
  memset(&prm, 0, sizeof(prm));
  prm.num_problems = 1;
  G2Problem& pz = prm.prob[0];
  pz.M = (int)tokens; pz.N = zcols; pz.K = n;
  pz.a_mode = TMA_KMAJOR; pz.b_mode = TMA_MNMAJOR; pz.epi_mode = EPI_BF16;
  pz.b_blocked = 1;
  pz.scale = pp.inv_sqrt_s;
  g2_finish(pz, 1);
  if (!make_map(&prm.tmA[0], X, n, tokens, ldx, BK, G2_HALF)) return COMPACT_ERR_CUDA;
  if (!make_map_blocked(&prm.tmB[0], P, ldp, n, ldp, BK, G2_HALF / 64)) return COMPACT_ERR_CUDA;
  if (!make_map(&prm.tmC[0], Z, zcols, tokens, ldz, 64, 32)) return COMPACT_ERR_CUDA;
  return g2_launch(li, prm);
}

// Algorithm 3: Adam moments -> N (bf16, front of the scratch), P written out behind it, then W <- W - scale * P N as
// one product on pairs of SMs whose epilogue adds the increment to W.  Same N, same entries of P, same order of accumulation and the same roundings as the
// streaming update on single SMs (which needs no room for P and remains the route when the scratch is small).
inline size_t g2_update_scratch_bytes(int n, int m, int r, int zcols) {
  return ((size_t)r * m * sizeof(__nv_bfloat16) + 255) / 256 * 256 + expanded_bytes(n, zcols);
}

inline compact_status_t g2_update(const LaunchInfo& li, const ProjectionParams& pp, const simt::AdamScalars& as, int n, int m, int r,
                                  int zcols, __nv_bfloat16* W, int64_t ldw, const float* Gc, int64_t ldg, float* M, float* V,
                                  float scale, void* workspace, size_t workspace_bytes) {
  if (!tc_shape_ok(1, n, m)) return COMPACT_ERR_SHAPE;
  if (!li.status) return COMPACT_ERR_CUDA;
  if (workspace_bytes < g2_update_scratch_bytes(n, m, r, zcols)) return COMPACT_ERR_WORKSPACE;
  __nv_bfloat16* Nbuf = (__nv_bfloat16*)workspace;
  __nv_bfloat16* P = (__nv_bfloat16*)((char*)workspace + ((size_t)r * m * sizeof(__nv_bfloat16) + 255) / 256 * 256);
  const long long cnt = (long long)r * (m / 4);
  const unsigned adam_blocks = (unsigned)((cnt + 255) / 256);
  const ExpandArgs ea = make_expand_args(pp, zcols, P);
  adam_and_expand_kernel<<<adam_blocks + expand_blocks_for(ea), 256, 0, li.stream>>>(Gc, ldg, M, V, Nbuf, r, m, as, (int)adam_blocks, ea);
  (*li.launches)++;
  if (cudaGetLastError() != cudaSuccess) return COMPACT_ERR_CUDA;
  const int64_t ldp = expanded_ld(zcols);
  G2Params prm;
  memset(&prm, 0, sizeof(prm));
  prm.num_problems = 1;
  G2Problem& pu = prm.prob[0];
  pu.M = n; pu.N = m; pu.K = r;
  pu.a_mode = TMA_KMAJOR; pu.b_mode = TMA_MNMAJOR; pu.epi_mode = EPI_UPDATE_W;
  pu.b_blocked = m % 64 == 0;
  pu.scale = scale;
  g2_finish(pu, 1);
  if (!make_map(&prm.tmA[0], P, ldp, n, ldp, BK, G2_HALF)) return COMPACT_ERR_CUDA;
  if (pu.b_blocked ? !make_map_blocked(&prm.tmB[0], Nbuf, m, r, m, BK, G2_HALF / 64) : !make_map(&prm.tmB[0], Nbuf, m, r, m, 64, BK))
    return COMPACT_ERR_CUDA;
  if (!make_map(&prm.tmC[0], W, m, n, ldw, 64, 32)) return COMPACT_ERR_CUDA;
  prm.early = 1;
  return g2_launch(li, prm);
}

// Algorithm 2: dX = dY W^T, and Gc = Z^T dY (both operands MN-major, split over tokens).
inline compact_status_t g2_backward(const LaunchInfo& li, int64_t tokens, int n, int m, int r, int zcols,
                                    const __nv_bfloat16* dY, int64_t lddy, const __nv_bfloat16* Z, int64_t ldz,
                                    const __nv_bfloat16* W, int64_t ldw, __nv_bfloat16* dX, int64_t lddx, float* Gc,
                                    int64_t ldg, int accumulate, void* workspace, size_t workspace_bytes) {
  if (!tc_shape_ok(tokens, n, m)) return COMPACT_ERR_SHAPE;
  if (!li.status) return COMPACT_ERR_CUDA;
  G2Params prm;
  memset(&prm, 0, sizeof(prm));
  prm.num_problems = dX ? 2 : 1;
  const int splits = plan_gc_splits(tokens, r, m);
  const bool staged = splits > 1 || accumulate;
  if (staged && workspace_bytes < (size_t)splits * r * m * sizeof(float)) return COMPACT_ERR_WORKSPACE;
  // dX first, Gc after: a launch that ends on the shorter tiles has the shorter tail (0.3-0.5 % on the backward)
  const int ig = dX ? 1 : 0, ix = 1 - ig;
  G2Problem& pg = prm.prob[ig];
  pg.M = r; pg.N = m; pg.K = (int)tokens;
  pg.a_mode = TMA_MNMAJOR; pg.b_mode = TMA_MNMAJOR; pg.epi_mode = EPI_F32;
  pg.a_blocked = zcols % 64 == 0;
  pg.b_blocked = m % 64 == 0;
  g2_finish(pg, splits);
  if (staged) {
    if (!make_map_f32_3d(&prm.tmC[ig], workspace, m, r, pg.splits, m, (int64_t)r * m)) return COMPACT_ERR_CUDA;
  } else {
    if (!make_map_f32_3d(&prm.tmC[ig], Gc, m, r, 1, ldg, (int64_t)r * ldg)) return COMPACT_ERR_CUDA;
  }
  if (pg.a_blocked ? !make_map_blocked(&prm.tmA[ig], Z, zcols, tokens, ldz, BK, G2_HALF / 64) : !make_map(&prm.tmA[ig], Z, zcols, tokens, ldz, 64, BK))
    return COMPACT_ERR_CUDA;
  if (pg.b_blocked ? !make_map_blocked(&prm.tmB[ig], dY, m, tokens, lddy, BK, G2_HALF / 64) : !make_map(&prm.tmB[ig], dY, m, tokens, lddy, 64, BK))
    return COMPACT_ERR_CUDA;
  if (dX) {
    G2Problem& px = prm.prob[ix];
    px.M = (int)tokens; px.N = n; px.K = m;
    px.a_mode = TMA_KMAJOR; px.b_mode = TMA_KMAJOR; px.epi_mode = EPI_BF16;
    g2_finish(px, 1);
    if (!make_map(&prm.tmA[ix], dY, m, tokens, lddy, BK, G2_HALF)) return COMPACT_ERR_CUDA;
    if (!make_map(&prm.tmB[ix], W, m, n, ldw, BK, G2_HALF)) return COMPACT_ERR_CUDA;
    if (!make_map(&prm.tmC[ix], dX, n, tokens, lddx, 64, 32)) return COMPACT_ERR_CUDA;
  }
  compact_status_t s = g2_launch(li, prm);
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

// Algorithm 2 for G layers that share their input: dX = sum_g dY_g W_g^T is ONE problem whose K runs over the
// layers (segment g reads dY_g and W_g), so the input gradient accumulates in the tensor cores instead of in G
// tensors added afterwards; the Gc_g are G more problems of the same launch, each split over tokens.
inline compact_status_t g2_backward_group(const LaunchInfo& li, int G, const GroupLayer* L, int64_t tokens, int n,
                                          __nv_bfloat16* dX, int64_t lddx, int accumulate, void* workspace,
                                          size_t workspace_bytes) {
  if (G < 1 || G > MAXG || 2 * G > G2_MAXP) return COMPACT_ERR_INVALID_ARG;
  if (!li.status) return COMPACT_ERR_CUDA;
  for (int g = 0; g < G; ++g)
    if (!tc_shape_ok(tokens, n, L[g].m)) return COMPACT_ERR_SHAPE;
  G2Params prm;
  memset(&prm, 0, sizeof(prm));
  int np = 0, slot = 0, dx_ksteps = 0;
  for (int g = 0; g < G; ++g) dx_ksteps += (L[g].m + BK - 1) / BK;
  // dX first: its tiles are the long ones (K runs over all layers), and the launch should end on short ones
  if (dX) {
    G2Problem& px = prm.prob[np++];
    px.M = (int)tokens; px.N = n; px.K = dx_ksteps * BK;
    px.a_mode = TMA_KMAJOR; px.b_mode = TMA_KMAJOR; px.epi_mode = EPI_BF16;
    g2_finish(px, 1);
    px.nseg = G; px.map_base = slot;
    int kb = 0;
    for (int g = 0; g < 4; ++g) {
      px.seg_begin[g] = kb;
      if (g < G) kb += (L[g].m + BK - 1) / BK;
    }
    for (int g = 0; g < G; ++g) {
      if (!make_map(&prm.tmA[slot + g], L[g].dY, L[g].m, tokens, L[g].lddy, BK, G2_HALF)) return COMPACT_ERR_CUDA;
      if (!make_map(&prm.tmB[slot + g], L[g].W, L[g].m, n, L[g].ldw, BK, G2_HALF)) return COMPACT_ERR_CUDA;
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
    G2Problem& pg = prm.prob[np++];
    pg.M = r; pg.N = m; pg.K = (int)tokens;
    pg.a_mode = TMA_MNMAJOR; pg.b_mode = TMA_MNMAJOR; pg.epi_mode = EPI_F32;
    pg.a_blocked = L[g].zcols % 64 == 0;
    pg.b_blocked = m % 64 == 0;
    g2_finish(pg, splits[g]);
    splits[g] = pg.splits;
    pg.nseg = 1; pg.map_base = slot;
    float* part = (float*)((char*)workspace + part_off[g]);
    if (staged[g]) {
      if (!make_map_f32_3d(&prm.tmC[slot], part, m, r, pg.splits, m, (int64_t)r * m)) return COMPACT_ERR_CUDA;
    } else {
      if (!make_map_f32_3d(&prm.tmC[slot], L[g].Gc, m, r, 1, L[g].ldg, (int64_t)r * L[g].ldg)) return COMPACT_ERR_CUDA;
    }
    if (pg.a_blocked ? !make_map_blocked(&prm.tmA[slot], L[g].Z, L[g].zcols, tokens, L[g].ldz, BK, G2_HALF / 64)
                     : !make_map(&prm.tmA[slot], L[g].Z, L[g].zcols, tokens, L[g].ldz, 64, BK))
      return COMPACT_ERR_CUDA;
    if (pg.b_blocked ? !make_map_blocked(&prm.tmB[slot], L[g].dY, m, tokens, L[g].lddy, BK, G2_HALF / 64)
                     : !make_map(&prm.tmB[slot], L[g].dY, m, tokens, L[g].lddy, 64, BK))
      return COMPACT_ERR_CUDA;
    ++slot;
  }
  prm.num_problems = np;
  compact_status_t s = g2_launch(li, prm);
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

}  // namespace g2
}  // namespace compact
