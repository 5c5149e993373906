// The update of the CompAct layer (Algorithm 3 lines 1-9) as ONE launch for layers whose rank fits a resident
// panel (r rounded up to 64 is at most 512):
//   phase 1  every CTA runs Adam on its slice of the r x m grid: M, V in place, N = M^/(sqrt(V^)+eps) as bf16 into
//            scratch (pitch m); meanwhile its generator warps build the projection panel it will need;
//   barrier  one counter in global memory: all of N is written before any CTA's loader reads it;
//   phase 2  W <- W - eta alpha P N on the tensor cores: a cluster of two CTAs owns 128 rows of W and a range of
//            column blocks; the 128 x r panel of P for those rows is generated ONCE (each CTA half, the halves
//            exchanged through distributed shared memory), stays resident in shared memory as the A operand, and
//            the CTA sweeps its column blocks: tiles of N stream in by TMA as the B operand, the 128 x 256
//            accumulator of one block drains (scaled, rounded to bf16, added to W by a TMA reduce) while the next
//            block's MMAs run into the other half of TMEM.
// Each entry of P is generated once per 128 x (columns of the cluster's range) of W instead of once per 1024
// columns, and no generation sits inside the sweep.
#pragma once
#include "tc_kernels.cuh"

namespace compact {
namespace upd {

using namespace tc;

constexpr int U_BN = 256;                        // columns of one block = one accumulator slot of TMEM
constexpr int U_KT = 8;                          // 64-wide k-tiles the resident panel holds (r_pad <= 512)
constexpr int U_PANEL_BYTES = U_KT * A_BYTES;    // 128 KB: [k-tile][128 rows][128 B], K-major, 128-byte swizzle
constexpr int U_SK = 32;                         // rows of N (k) per B stage
constexpr int U_STAGE_BYTES = U_SK * U_BN * 2;   // 16 KB: [4 column blocks of 64][32 k][128 B], MN-major
constexpr int U_NS = 5;                          // the sweep is bound by the latency of these loads: as many in flight as fit
constexpr int U_EPI_WARPS = 4;                   // one warp per TMEM lane quarter
constexpr int U_GEN_WARPS = 16;
constexpr int U_THREADS = 32 * (2 + U_EPI_WARPS + U_GEN_WARPS);
constexpr int U_STAGING_OFF = U_PANEL_BYTES + U_NS * U_STAGE_BYTES;
constexpr int U_BARS_OFF = U_STAGING_OFF + U_EPI_WARPS * STAGING_BYTES;
constexpr int U_NUM_BARS = U_KT + 1 + 2 * U_NS + 4;      // panel full per k-tile, panel free, ring full/empty, accumulators
constexpr int U_SMEM_BYTES = 1024 + U_BARS_OFF + 8 * U_NUM_BARS + 32;     // tail: TMEM address, abort flag, phase-1 counter
static_assert(U_SMEM_BYTES <= 232448, "shared memory budget");

struct alignas(64) UpdParams {
  CUtensorMap tmN;          // N (bf16 scratch, r x m, pitch ldn) seen as [m / 64][r][64]: box {64, U_SK, 4}
  CUtensorMap tmW;          // W (n x m bf16): box {64, 32}, 128-byte swizzle; target of the reduce-add
  const float* Gc;
  float* M;
  float* V;
  __nv_bfloat16* Nbuf;
  long long ldn;            // pitch of the scratch N in elements
  long long ldg;            // pitch of Gc, M, V in elements
  int n, m, r;
  int ktiles;               // ceil(r / 64)
  int nblocks;              // ceil(m / 256)
  int J;                    // column ranges per row panel
  int jobs;                 // row panels * J
  float scale;              // eta * alpha
  simt::AdamScalars as;
  PhiloxKey key;
  uint32_t layer_hi, layer_lo, epoch;
  float pp_scale;           // -2 ln 2 / r
  int sparse_s;             // > 0: sparse projection (the panel holds integer counts; 1/sqrt(s) is part of `scale`)
  unsigned int* status;
  unsigned int* sched;      // three words, zero between launches: CTAs done with phase 1, CTAs finished, next run of phase 1
};

__device__ __forceinline__ void fence_proxy_async_all() { asm volatile("fence.proxy.async;" ::: "memory"); }
__device__ __forceinline__ unsigned int ld_acquire_gpu(const unsigned int* p) {
  unsigned int v;
  asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
  return v;
}

// Warp roles:
//   0       loader of the tiles of N (waits for the phase-1 counter first)
//   1       tcgen05.mma issuer; owns TMEM
//   2..5    epilogue (one warp per TMEM lane quarter)
//   6..21   generators of the panel of P
// Every warp first takes part in phase 1 (the generators after their first panel).
__global__ void __launch_bounds__(U_THREADS, 1) compact_update_kernel(const __grid_constant__ UpdParams prm) {
  extern __shared__ uint8_t smem_raw[];
  const uint32_t smem_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
  uint8_t* smem_gen = smem_raw + (smem_base - smem_u32(smem_raw));
  const uint32_t ring = smem_base + U_PANEL_BYTES;
  const uint32_t staging = smem_base + U_STAGING_OFF;
  const uint32_t bars = smem_base + U_BARS_OFF;
  auto pfull_bar = [&](int kt) { return bars + 8u * kt; };
  const uint32_t pfree_bar = bars + 8u * U_KT;
  auto full_bar = [&](int s) { return bars + 8u * (U_KT + 1 + s); };
  auto empty_bar = [&](int s) { return bars + 8u * (U_KT + 1 + U_NS + s); };
  auto tfull_bar = [&](int a) { return bars + 8u * (U_KT + 1 + 2 * U_NS + a); };
  auto tempty_bar = [&](int a) { return bars + 8u * (U_KT + 1 + 2 * U_NS + 2 + a); };
  uint8_t* tail = smem_gen + U_BARS_OFF + 8 * U_NUM_BARS;
  volatile uint32_t* tmem_slot = reinterpret_cast<volatile uint32_t*>(tail);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tail + 8);

  const int warp = threadIdx.x >> 5;
  const int lane = threadIdx.x & 31;
  const uint32_t crank = cluster_ctarank();
  const int cluster_id = (int)(blockIdx.x >> 1);
  const int nclusters = (int)(gridDim.x >> 1);

  if (threadIdx.x == 0) {
    for (int kt = 0; kt < U_KT; ++kt) mbar_init(pfull_bar(kt), 1 + U_GEN_WARPS);   // the arming thread, the generator warps
    mbar_init(pfree_bar, 2);                                                      // the issuers of both CTAs
    for (int s = 0; s < U_NS; ++s) {
      mbar_init(full_bar(s), 1);
      mbar_init(empty_bar(s), 1);
    }
    for (int a = 0; a < 2; ++a) {
      mbar_init(tfull_bar(a), 1);
      mbar_init(tempty_bar(a), U_EPI_WARPS);
    }
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
  cluster_sync_all();                        // both CTAs' barriers exist before anything crosses
  const uint32_t tmem_base = *tmem_slot;

  // A cluster's jobs: job -> (row panel, column range); its two CTAs take alternate column blocks of the range.
  // A CTA visits its `cnt` blocks starting at a position that depends on its row panel, so that the CTAs of
  // different panels (which sweep the same columns of N) do not ask for the same tile at the same moment.
  struct JobBlocks { int panel, first, cnt, rot; };
  auto job_blocks = [&](int job) {
    JobBlocks jb;
    jb.panel = job / prm.J;
    const int part = job % prm.J;
    const int lo = (int)((long long)part * prm.nblocks / prm.J);
    const int end = (int)((long long)(part + 1) * prm.nblocks / prm.J);
    jb.first = lo + (int)crank;
    jb.cnt = jb.first < end ? (end - jb.first + 1) / 2 : 0;
    jb.rot = jb.cnt > 0 ? jb.panel % jb.cnt : 0;
    return jb;
  };
  auto block_at = [&](const JobBlocks& jb, int idx) {
    int k = idx + jb.rot;
    if (k >= jb.cnt) k -= jb.cnt;
    return jb.first + 2 * k;
  };

  // Phase 1 (Algorithm 3 lines 1-5) on the r x m grid.  Every warp of every CTA takes part -- the generators
  // once their first panel is written -- claiming runs of 64 four-column groups; a lane keeps two groups in
  // flight.  When no run is left the CTA reports its share as written.
  auto adam_slice = [&]() {
    const int m4 = prm.m >> 2;
    const long long g1 = (long long)prm.r * m4;
    const simt::AdamScalars s = prm.as;
    constexpr int kU = 2;                      // groups a lane keeps in flight
    for (;;) {
      // runs of 32 kU groups come from one counter for the whole grid: CTAs whose warps are all free from the
      // start (no panel to generate) take more of them
      unsigned int base = 0;
      if (lane == 0) base = atomicAdd(prm.sched + 2, 32u * kU);
      base = __shfl_sync(0xffffffffu, base, 0);
      const long long g0 = 0;
      if (base >= g1) break;
      float4 gr[kU], mm[kU], vv[kU];
      long long off[kU], noff[kU];
#pragma unroll
      for (int u = 0; u < kU; ++u) {
        const long long g = g0 + base + 32 * u + lane;
        const bool in = g < g1;
        const int j = in ? (int)(g / m4) : 0, c = in ? (int)(g % m4) * 4 : 0;
        off[u] = in ? (long long)j * prm.ldg + c : -1;
        noff[u] = (long long)j * prm.ldn + c;
        if (in) {
          gr[u] = *reinterpret_cast<const float4*>(prm.Gc + off[u]);
          mm[u] = *reinterpret_cast<const float4*>(prm.M + off[u]);
          vv[u] = *reinterpret_cast<const float4*>(prm.V + off[u]);
        }
      }
#pragma unroll
      for (int u = 0; u < kU; ++u) {
        if (off[u] < 0) continue;
        float4 m1 = mm[u], v1 = vv[u];
        const float4 g4 = gr[u];
        m1.x = fmaf(s.beta1, m1.x, s.one_minus_beta1 * g4.x);
        m1.y = fmaf(s.beta1, m1.y, s.one_minus_beta1 * g4.y);
        m1.z = fmaf(s.beta1, m1.z, s.one_minus_beta1 * g4.z);
        m1.w = fmaf(s.beta1, m1.w, s.one_minus_beta1 * g4.w);
        v1.x = fmaf(s.beta2, v1.x, s.one_minus_beta2 * g4.x * g4.x);
        v1.y = fmaf(s.beta2, v1.y, s.one_minus_beta2 * g4.y * g4.y);
        v1.z = fmaf(s.beta2, v1.z, s.one_minus_beta2 * g4.z * g4.z);
        v1.w = fmaf(s.beta2, v1.w, s.one_minus_beta2 * g4.w * g4.w);
        *reinterpret_cast<float4*>(prm.M + off[u]) = m1;
        *reinterpret_cast<float4*>(prm.V + off[u]) = v1;
        const float n0 = (m1.x * s.inv_bias1) / (sqrtf(v1.x * s.inv_bias2) + s.eps);
        const float n1 = (m1.y * s.inv_bias1) / (sqrtf(v1.y * s.inv_bias2) + s.eps);
        const float n2 = (m1.z * s.inv_bias1) / (sqrtf(v1.z * s.inv_bias2) + s.eps);
        const float n3 = (m1.w * s.inv_bias1) / (sqrtf(v1.w * s.inv_bias2) + s.eps);
        *reinterpret_cast<uint2*>(prm.Nbuf + noff[u]) = make_uint2(pack_bf16x2(n0, n1), pack_bf16x2(n2, n3));
      }
    }
    // this thread's part of N is visible to the other SMs, and to their TMA units, before the CTA reports
    fence_proxy_async_all();
    __threadfence();
    named_barrier(1, U_THREADS);
    if (threadIdx.x == 0) atomicAdd(prm.sched, 1u);
  };

  if (warp == 0) {
    // ------------------------------ loader of N ---------------------------------
    bool ok = true;
    constexpr int kAhead = 2;
    // asks the L2 for the 128 x 256 tile of W that block b of a row panel will be added to
    auto prefetch_w = [&](int panel, int b) {
      for (int rq = 0; rq < BM / 32; ++rq)
        for (int ci = 0; ci < U_BN / 64; ++ci) {
          const int row = panel * BM + rq * 32, col = b * U_BN + ci * 64;
          if (row < prm.n && col < prm.m) tma_prefetch_2d(&prm.tmW, col, row);
        }
    };
    if (cluster_id < prm.jobs) {
      // while phase 1 runs elsewhere: the first tiles of W start their way from DRAM
      if (elect_one()) {
        const JobBlocks jb = job_blocks(cluster_id);
        for (int idx = 0; idx < kAhead && idx < jb.cnt; ++idx) prefetch_w(jb.panel, block_at(jb, idx));
      }
      __syncwarp();
    }
    adam_slice();
    if (cluster_id < prm.jobs) {
      // every CTA has written its slice of N (phase 1) before the first tile of N is read
      if (lane == 0) {
        uint32_t it = 0;
        while (ld_acquire_gpu(prm.sched) < gridDim.x) {
          if (*abort_flag || ++it > 4000000u) {
            *abort_flag = 1;
            atomicOr(prm.status, STATUS_TIMEOUT);
            ok = false;
            break;
          }
          __nanosleep(200);
        }
        fence_proxy_async_all();             // those writes were generic-proxy writes; the TMA reads through the async proxy
      }
      ok = __shfl_sync(0xffffffffu, ok ? 1 : 0, 0) != 0;
    }
    Ring r = {0, 0u};
    for (int job = cluster_id; job < prm.jobs && ok; job += nclusters) {
      const JobBlocks jb = job_blocks(job);
      for (int idx = 0; idx < jb.cnt && ok; ++idx) {
        const int b = block_at(jb, idx);
        // the tiles of W that the block after next will be added to: on their way into L2 by then
        if (idx + kAhead < jb.cnt && elect_one()) prefetch_w(jb.panel, block_at(jb, idx + kAhead));
        __syncwarp();
        for (int st = 0; st < 2 * prm.ktiles; ++st, ring_next(r, U_NS)) {
          if (!(ok = __all_sync(0xffffffffu, mbar_wait(empty_bar(r.s), r.ph ^ 1u, abort_flag, prm.status)))) break;
          if (elect_one()) {
            mbar_arrive_expect_tx(full_bar(r.s), U_STAGE_BYTES);
            tma_load_3d(ring + (uint32_t)r.s * U_STAGE_BYTES, &prm.tmN, full_bar(r.s), 0, st * U_SK, b * (U_BN / 64));
          }
          __syncwarp();
        }
      }
    }
  } else if (warp == 1) {
    // ------------------------------ MMA issuer ----------------------------------
    adam_slice();
    bool ok = true;
    Ring r = {0, 0u};
    int slot = 0;
    uint32_t slot_phase = 0, job_phase = 0;
    // A: K-major (128 rows of 128 B per k-tile), B: MN-major; D: 128 x 256 fp32
    const uint32_t idesc = (1u << 4) | (1u << 7) | (1u << 10) | (1u << 16) | ((uint32_t)(U_BN >> 3) << 17) | ((uint32_t)(BM >> 4) << 24);
    const uint32_t panel_lo = ((smem_base >> 4) & 0x3FFFu) | (1u << 16);
    const uint32_t b_flags = ((uint32_t)(U_SK * 128) >> 4) << 16;      // distance between the stage's 64-column blocks
    for (int job = cluster_id; job < prm.jobs && ok; job += nclusters, job_phase ^= 1u) {
      const JobBlocks jb = job_blocks(job);
      bool first_block = true;
      for (int idx = 0; idx < jb.cnt && ok; ++idx, first_block = false) {
        if (!(ok = __all_sync(0xffffffffu, mbar_wait(tempty_bar(slot), slot_phase ^ 1u, abort_flag, prm.status)))) break;
        tc_fence_after();
        const uint32_t d = tmem_base + (uint32_t)slot * U_BN;
        for (int kt = 0; kt < prm.ktiles && ok; ++kt) {
          // the first block of a job meets the panel while it is being generated
          if (first_block && !(ok = __all_sync(0xffffffffu, mbar_wait(pfull_bar(kt), job_phase, abort_flag, prm.status)))) break;
          for (int h = 0; h < 2; ++h, ring_next(r, U_NS)) {
            if (!(ok = __all_sync(0xffffffffu, mbar_wait(full_bar(r.s), r.ph, abort_flag, prm.status)))) break;
            tc_fence_after();
            if (elect_one()) {
              const uint32_t a_lo = panel_lo + (uint32_t)((kt * A_BYTES + h * 64) >> 4);
              const uint32_t b_lo = (((ring + (uint32_t)r.s * U_STAGE_BYTES) >> 4) & 0x3FFFu) | b_flags;
              umma_bf16(d, a_lo, DESC_HI, b_lo, DESC_HI, idesc, (kt | h) ? 1u : 0u);
              umma_bf16(d, a_lo + (32u >> 4), DESC_HI, b_lo + (2048u >> 4), DESC_HI, idesc, 1u);
              umma_commit(empty_bar(r.s));
            }
            __syncwarp();
          }
        }
        if (!ok) break;
        if (elect_one()) umma_commit(tfull_bar(slot));
        __syncwarp();
        if (++slot == 2) { slot = 0; slot_phase ^= 1u; }
      }
      // a CTA without a block in this job still meets every tile of the panel, so that it cannot hand back a
      // panel (and run on to the next job) before that panel exists
      for (int kt = 0; kt < prm.ktiles && ok && jb.cnt == 0; ++kt)
        ok = __all_sync(0xffffffffu, mbar_wait(pfull_bar(kt), job_phase, abort_flag, prm.status));
      if (!ok) break;
      // with a block of its own or without: this CTA no longer reads the panel once these MMAs are done
      if (elect_one()) umma_commit_mc(pfree_bar, (uint16_t)3);
      __syncwarp();
    }
  } else if (warp < 2 + U_EPI_WARPS) {
    // ------------------------------ Adam, then epilogue -------------------------
    adam_slice();
    const int q = warp & 3;                 // TMEM lane quarter this warp may read
    const uint32_t stg = staging + (warp - 2) * STAGING_BYTES;
    uint8_t* stg_gen = smem_gen + U_STAGING_OFF + (warp - 2) * STAGING_BYTES;
    const int sw = lane & 7;
    int slot = 0;
    uint32_t slot_phase = 0;
    bool ok = true;
    const float sc = -prm.scale;
    for (int job = cluster_id; job < prm.jobs && ok; job += nclusters) {
      const JobBlocks jb = job_blocks(job);
      const int row0 = jb.panel * BM + q * 32;
      for (int idx = 0; idx < jb.cnt && ok; ++idx) {
        const int b = block_at(jb, idx);
        if (!(ok = mbar_wait(tfull_bar(slot), slot_phase, abort_flag, prm.status))) break;
        tc_fence_after();
        const uint32_t tcol = tmem_base + ((uint32_t)(q * 32) << 16) + (uint32_t)slot * U_BN;
        for (int ci = 0; ci < U_BN / 64 && row0 < prm.n; ++ci) {
          const int col = b * U_BN + ci * 64;
          if (col >= prm.m) break;
          uint32_t o[32];
#pragma unroll
          for (int h = 0; h < 2; ++h) {
            uint32_t v[32];
            tmem_ld32(tcol + ci * 64 + 32 * h, v);
            tmem_ld_wait();
#pragma unroll
            for (int j = 0; j < 16; ++j)
              o[16 * h + j] = pack_bf16x2(sc * __uint_as_float(v[2 * j]), sc * __uint_as_float(v[2 * j + 1]));
          }
          if (lane == 0) tma_store_wait_read();       // the previous reduce has read the staging tile
          __syncwarp();
#pragma unroll
          for (int j = 0; j < 8; ++j)
            *reinterpret_cast<uint4*>(stg_gen + lane * 128 + ((j ^ sw) << 4)) = make_uint4(o[4 * j], o[4 * j + 1], o[4 * j + 2], o[4 * j + 3]);
          fence_proxy_async_smem();
          __syncwarp();
          if (lane == 0) {
            tma_reduce_add_2d(&prm.tmW, stg, col, row0);   // W += -(eta alpha) (P N), Algorithm 3 line 9
            tma_store_commit();
          }
        }
        tc_fence_before();
        __syncwarp();
        if (lane == 0) mbar_arrive(tempty_bar(slot));
        if (++slot == 2) { slot = 0; slot_phase ^= 1u; }
      }
    }
    if (lane == 0) tma_store_wait_all();
  } else {
    // ------------------------------ generators of the panel ---------------------
    // Tile kt of the panel is A[row of P][64 columns of P], K-major.  This CTA writes rows crank*64 .. +63 of it,
    // into its own shared memory and into its neighbour's, whose barrier counts the bytes.
    const int gtid = threadIdx.x - 32 * (2 + U_EPI_WARPS);       // 0 .. 511: one task of eight entries per tile
    const uint32_t peer_base = map_to_cta(smem_base, crank ^ 1u);
    const uint32_t peer_bars = map_to_cta(bars, crank ^ 1u);
    const int c = gtid & 7, rr = (int)crank * (BM / 2) + (gtid >> 3);
    const uint32_t t_off = (uint32_t)(rr * 128 + ((c ^ (rr & 7)) << 4));
    bool ok = true;
    uint32_t free_phase = 0;
    bool first_job = true;
    for (int job = cluster_id; job < prm.jobs && ok; job += nclusters, first_job = false) {
      const int panel = job_blocks(job).panel;
      if (!first_job) {
        // both CTAs are done reading the previous job's panel
        ok = __all_sync(0xffffffffu, mbar_wait(pfree_bar, free_phase, abort_flag, prm.status));
        free_phase ^= 1u;
        if (!ok) break;
      }
      if (prm.sparse_s > 0) {
        // Sparse projection: every CTA builds the whole panel itself.  All threads clear it, then one thread per
        // row adds the signs of the row's terms at their columns (one writer per row: colliding terms add).
        if (gtid == 0)
          for (int kt = 0; kt < prm.ktiles; ++kt) mbar_arrive(pfull_bar(kt));
        for (int x = gtid; x < prm.ktiles * (A_BYTES / 16); x += 32 * U_GEN_WARPS)
          reinterpret_cast<uint4*>(smem_gen)[x] = make_uint4(0u, 0u, 0u, 0u);
        named_barrier(2, 32 * U_GEN_WARPS);
        const int row = panel * BM + gtid;
        if (gtid < BM && row < prm.n) {
          for (int q = 0; 4 * q < prm.sparse_s; ++q) {
            const uint4 x = sparse_words4((uint32_t)q, (uint32_t)row, prm.epoch, prm.layer_hi, prm.layer_lo, prm.key);
            const uint32_t wd[4] = {x.x, x.y, x.z, x.w};
#pragma unroll
            for (int l = 0; l < 4; ++l) {
              if (4 * q + l >= prm.sparse_s) continue;
              const int col = sparse_col(wd[l], prm.r), kt = col >> 6, cc = col & 63;
              __nv_bfloat16* e = reinterpret_cast<__nv_bfloat16*>(smem_gen + kt * A_BYTES + gtid * 128 + (((cc >> 3) ^ (gtid & 7)) << 4) + (cc & 7) * 2);
              *e = __float2bfloat16_rn(__bfloat162float(*e) + sparse_sign(wd[l]));
            }
          }
        }
        fence_proxy_async_smem();
        __syncwarp();
        if (lane == 0)
          for (int kt = 0; kt < prm.ktiles; ++kt) mbar_arrive(pfull_bar(kt));
        if (first_job) adam_slice();
        continue;
      }
      // the neighbour's half of every tile arrives as counted bytes
      if (gtid == 0)
        for (int kt = 0; kt < prm.ktiles; ++kt) mbar_arrive_expect_tx(pfull_bar(kt), A_BYTES / 2);
      const int i = panel * BM + rr;
      for (int kt = 0; kt < prm.ktiles; ++kt) {
        const uint4 val = projection8_bf16(prm.key, prm.layer_hi, prm.layer_lo, prm.epoch, prm.n, prm.r, prm.pp_scale, i, kt * BK + c * 8);
        const uint32_t off = (uint32_t)kt * A_BYTES + t_off;
        *reinterpret_cast<uint4*>(smem_gen + off) = val;
        st_async_16(peer_base + off, val, peer_bars + 8u * kt);
        fence_proxy_async_smem();
        __syncwarp();
        if (lane == 0) mbar_arrive(pfull_bar(kt));
      }
      if (first_job) adam_slice();
    }
    if (cluster_id >= prm.jobs) adam_slice();       // a cluster without a job has nothing to generate
  }

  tc_fence_before();
  __syncthreads();
  if (warp == 1) {
    tc_fence_after();
    tmem_dealloc(tmem_base, 512);
  }
  cluster_sync_all();                        // no CTA leaves while its neighbour may still signal it
  if (threadIdx.x == 0) {
    __threadfence();
    if (atomicAdd(prm.sched + 1, 1u) == gridDim.x - 1) {
      prm.sched[0] = 0u;
      prm.sched[1] = 0u;
      prm.sched[2] = 0u;
      __threadfence();
    }
  }
}

// Shapes this kernel takes: the panel must fit (r_pad <= 512) and N is read through the blocked map (m % 64 == 0).
inline bool fused_update_ok(int n, int m, int r) {
  return n % 8 == 0 && m % 64 == 0 && r >= 1 && (r + BK - 1) / BK <= U_KT;
}

inline compact_status_t fused_update(const LaunchInfo& li, const ProjectionParams& pp, const simt::AdamScalars& as, int n,
                                     int m, int r, __nv_bfloat16* W, int64_t ldw, const float* Gc, int64_t ldg, float* M,
                                     float* V, float scale, void* workspace, size_t workspace_bytes) {
  if (!fused_update_ok(n, m, r)) return COMPACT_ERR_SHAPE;
  if (!li.status || !li.sched) return COMPACT_ERR_CUDA;
  // rows of the scratch N sit a 128-byte line further apart than their length: with a pitch that is a large power
  // of two the 32 rows of a tile fall on few L2 slices and the sweep ran at half its speed
  const int64_t ldn = (int64_t)m + 64;
  if (workspace_bytes < (size_t)r * ldn * 2) return COMPACT_ERR_WORKSPACE;
  static std::atomic<bool> attr_set[64];
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) { cudaGetLastError(); return COMPACT_ERR_CUDA; }
  if (!attr_set[dev].load(std::memory_order_acquire)) {
    if (cudaFuncSetAttribute(compact_update_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, U_SMEM_BYTES) != cudaSuccess) {
      cudaGetLastError();
      return COMPACT_ERR_CUDA;
    }
    attr_set[dev].store(true, std::memory_order_release);
  }
  UpdParams prm;
  memset(&prm, 0, sizeof(prm));
  prm.Gc = Gc; prm.M = M; prm.V = V; prm.Nbuf = (__nv_bfloat16*)workspace; prm.ldn = ldn; prm.ldg = ldg;
  prm.n = n; prm.m = m; prm.r = r;
  prm.ktiles = (r + BK - 1) / BK;
  prm.nblocks = (m + U_BN - 1) / U_BN;
  const int panels = (n + BM - 1) / BM;
  const int nclusters = NUM_SMS / 2;
  int J = nclusters / panels;                       // as many column ranges per panel as there are clusters for
  if (J > (prm.nblocks + 1) / 2) J = (prm.nblocks + 1) / 2;     // a range holds at least a block per CTA
  if (J < 1) J = 1;
  prm.J = J;
  prm.jobs = panels * J;
  prm.scale = scale;
  prm.as = as;
  prm.key = pp.key;
  prm.layer_hi = pp.layer_hi; prm.layer_lo = pp.layer_lo; prm.epoch = pp.epoch;
  prm.pp_scale = pp.neg2ln2_over_r;
  prm.sparse_s = pp.sparse_s;
  prm.status = li.status;
  prm.sched = li.sched;
  if (!make_map_blocked(&prm.tmN, workspace, m, r, ldn, U_SK, U_BN / 64)) return COMPACT_ERR_CUDA;
  if (!make_map(&prm.tmW, W, m, n, ldw, 64, 32)) return COMPACT_ERR_CUDA;
  cudaLaunchConfig_t cfg;
  memset(&cfg, 0, sizeof(cfg));
  cfg.gridDim = dim3((unsigned)(2 * nclusters), 1, 1);
  cfg.blockDim = dim3((unsigned)U_THREADS, 1, 1);
  cfg.dynamicSmemBytes = U_SMEM_BYTES;
  cfg.stream = li.stream;
  // The grid is one CTA per SM at most, so all of it is resident at once; the wait at the phase barrier is bounded
  // like every other wait.  (A cooperative launch would state that requirement to the driver; it is left out
  // because the profiler could not launch the kernel with it.)
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeClusterDimension;
  attr[0].val.clusterDim.x = 2;
  attr[0].val.clusterDim.y = 1;
  attr[0].val.clusterDim.z = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  const cudaError_t e = cudaLaunchKernelEx(&cfg, compact_update_kernel, prm);
  (*li.launches)++;
  if (e != cudaSuccess) { cudaGetLastError(); return COMPACT_ERR_CUDA; }
  return cudaGetLastError() == cudaSuccess ? COMPACT_OK : COMPACT_ERR_CUDA;
}

}  // namespace upd
}  // namespace compact
