// bf16 linear for passes of many rows (batched verification: M = sequences x tree nodes = 1024, batched
// prompt processing), where the projections are compute-bound: y = x W^T on the 5th-generation tensor
// cores with every weight tile kept for 256 activation rows at a time.
//
// Operands are swapped as in gemm_stream (128 weight rows are the MMA's M) but the activation side is the
// full 256-wide MMA N: an output tile is [128 weight rows] x [256 activation rows], its accumulator takes 256
// of the 512 tensor-memory columns, and two of them alternate so that the epilogue of one tile runs under
// the MMAs of the next. The K loop of a tile walks all K chunks (no split K: there are at least as many
// tiles as SMs for every projection of a 7B-class model at M = 1024), so the kernel writes finished float32
// sums -- in the layout gemm_stream's consumers read, as a single slot. Persistent: CTA c takes tiles
// c, c + gridDim.x, ...; tile = weight tile * m_tiles + activation tile, so the CTAs that share a weight
// tile run side by side and the weights cross HBM once.
//
// Warp roles: warp 0 feeds a ring of 48 KB stages (16 KB weight unit by bulk copy or TMA, 32 KB activation
// tile by TMA, 128-byte swizzle), warp 1 issues tcgen05.mma (M 128, N 256, K 16), warps 2..9 drain: two warps
// per SM quarter, one for each half of the tile's 256 activation rows, so that the drain of the last tile (which
// nothing hides) takes half as long.
#pragma once
#include <cuda.h>

#include "common.cuh"
#include "gemm_stream.cuh"

namespace spec {

constexpr int GW_NT = 256;                  // activation rows per tile (MMA N)
constexpr int GW_STAGES = 4;

struct WideGemmParams {
  int M, K, KC;
  int n_mats;
  int mat_tile0[GS_MAX_MATS + 1];           // first weight tile of each stacked matrix
  const uint8_t* packed[GS_MAX_MATS];       // pre-tiled images or nullptr -> tensor maps a[i]
  int n_tiles, m_tiles;                     // weight tiles (all matrices), activation tiles of 256 rows
  float* part;                              // [M][n_tiles * 128] float32 (padded column space)
  int* status;
  unsigned long long* trace;
};

struct WideCfg {
  static constexpr int BK = 64;
  static constexpr int A_BYTES = 128 * BK * 2;
  static constexpr int B_BYTES = GW_NT * BK * 2;
  static constexpr int STAGE_BYTES = A_BYTES + B_BYTES;
  static constexpr int SMEM_BYTES = GW_STAGES * STAGE_BYTES + 1024 + 256;
  static constexpr int TMEM_COLS = 2 * GW_NT;
};

constexpr int GW_THREADS = 320;

__global__ void __launch_bounds__(GW_THREADS, 1)
gemm_wide(const __grid_constant__ StreamTmaps tm, const WideGemmParams p) {
  using Cfg = WideCfg;
  constexpr int STAGES = GW_STAGES;
  extern __shared__ uint8_t smem_raw[];
  const uint32_t raw = smem_u32(smem_raw);
  uint8_t* tiles = smem_raw + (((raw + 1023u) & ~1023u) - raw);
  uint64_t* bars = reinterpret_cast<uint64_t*>(tiles + STAGES * Cfg::STAGE_BYTES);
  uint64_t* full = bars;
  uint64_t* empty = bars + STAGES;
  uint64_t* acc_full = bars + 2 * STAGES;
  uint64_t* acc_empty = bars + 2 * STAGES + 2;
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + 2 * STAGES + 4);

  KTrace kt(p.trace);
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int KC = p.KC;
  const int total_tiles = p.n_tiles * p.m_tiles;
  const int my_tiles = (int)blockIdx.x < total_tiles ? (total_tiles - 1 - (int)blockIdx.x) / (int)gridDim.x + 1 : 0;

  pdl_launch_dependents();

  if (threadIdx.x == 0) {
    for (int i = 0; i < STAGES; ++i) { mbar_init(&full[i], 1); mbar_init(&empty[i], 1); }
    mbar_init(&acc_full[0], 1); mbar_init(&acc_full[1], 1);
    mbar_init(&acc_empty[0], 8); mbar_init(&acc_empty[1], 8);
    mbar_fence_init();
    for (int i = 0; i < p.n_mats; ++i) if (!p.packed[i]) tma_prefetch_desc(&tm.a[i]);
    tma_prefetch_desc(&tm.b);
  }
  if (warp == 1) { tmem_alloc(tmem_slot, Cfg::TMEM_COLS); tmem_relinquish(); }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;

  if (warp == 0) {
    if (lane == 0) {
      // ---- producer ----
      auto load_a = [&](uint8_t* dst, int nt, int kc, uint64_t* bar) {
        int mat = 0;
#pragma unroll
        for (int i = 1; i < GS_MAX_MATS; ++i)
          if (i < p.n_mats && nt >= p.mat_tile0[i]) mat = i;
        const int t_in = nt - p.mat_tile0[mat];
        // four CTAs read the same unit at about the same time (the other activation tiles): normal L2 priority
        if (p.packed[mat]) bulk_load_1d(dst, p.packed[mat] + ((size_t)t_in * KC + kc) * Cfg::A_BYTES, Cfg::A_BYTES, bar);
        else tma_load_2d(dst, &tm.a[mat], kc * Cfg::BK, t_in * 128, bar);
      };
      const int n_units = my_tiles * KC;
      const int n_pre = n_units < STAGES ? n_units : STAGES;
      auto unit = [&](int u, int& nt, int& mt, int& kc) {
        const int tau = (int)blockIdx.x + (u / KC) * (int)gridDim.x;
        kc = u % KC; nt = tau / p.m_tiles; mt = tau % p.m_tiles;
      };
      // weights do not depend on the kernel before this one
      for (int i = 0; i < n_pre; ++i) {
        int nt, mt, kc;
        unit(i, nt, mt, kc);
        mbar_expect_tx(&full[i], Cfg::STAGE_BYTES);
        load_a(tiles + i * Cfg::STAGE_BYTES, nt, kc, &full[i]);
      }
      pdl_wait();
      for (int i = 0; i < n_pre; ++i) {
        int nt, mt, kc;
        unit(i, nt, mt, kc);
        tma_load_2d(tiles + i * Cfg::STAGE_BYTES + Cfg::A_BYTES, &tm.b, kc * Cfg::BK, mt * GW_NT, &full[i]);
      }
      bool ok = true;
      int issued = n_pre;
      for (; issued < n_units; ++issued) {
        const int st = issued % STAGES;
        const uint32_t ph = (issued / STAGES) & 1;
        if (!mbar_wait(&empty[st], ph ^ 1, p.status, 40)) { ok = false; break; }
        int nt, mt, kc;
        unit(issued, nt, mt, kc);
        uint8_t* a = tiles + st * Cfg::STAGE_BYTES;
        mbar_expect_tx(&full[st], Cfg::STAGE_BYTES);
        load_a(a, nt, kc, &full[st]);
        tma_load_2d(a + Cfg::A_BYTES, &tm.b, kc * Cfg::BK, mt * GW_NT, &full[st]);
      }
      if (!ok) {
        for (int i = issued > STAGES ? issued - STAGES : 0; i < issued; ++i)
          mbar_wait(&full[i % STAGES], (i / STAGES) & 1, p.status, 43);
      }
    }
  } else if (warp == 1) {
    if (lane == 0) {
      // ---- MMA issuer ----
      const uint32_t idesc = make_idesc_bf16(128, GW_NT);
      bool ok = true;
      int done = 0;
      for (int i = 0; i < my_tiles && ok; ++i) {
        const int buf = i & 1;
        if (!mbar_wait(&acc_empty[buf], ((i >> 1) & 1) ^ 1, p.status, 44)) { ok = false; break; }
        tc_fence_after();
        const uint32_t d_addr = tmem_base + (uint32_t)(buf * GW_NT);
        for (int kc = 0; kc < KC; ++kc, ++done) {
          const int st = done % STAGES;
          const uint32_t ph = (done / STAGES) & 1;
          if (!mbar_wait(&full[st], ph, p.status, 41)) { ok = false; break; }
          if (done == 0) trace_mark_min(p.trace, 2);
          tc_fence_after();
          const uint32_t a_addr = smem_u32(tiles + st * Cfg::STAGE_BYTES);
          const uint64_t adesc = make_kmajor_sw128_desc(a_addr);
          const uint64_t bdesc = make_kmajor_sw128_desc(a_addr + Cfg::A_BYTES);
#pragma unroll
          for (int k = 0; k < Cfg::BK / 16; ++k)
            tc_mma_f16(d_addr, adesc + 2 * k, bdesc + 2 * k, idesc, (kc > 0 || k > 0) ? 1u : 0u);
          tc_commit(&empty[st]);
        }
        if (!ok) break;
        tc_commit(&acc_full[buf]);
      }
      trace_mark_max(p.trace, 3);
    }
  } else {
    // ---- epilogue: warps 2..9; warp w may touch tensor-memory lanes [32 (w % 4), +32); warps 2..5 take
    // activation rows [0, 128) of the tile, warps 6..9 rows [128, 256) ----
    const int q = warp & 3, hf = warp >= 6 ? 1 : 0;
    pdl_wait();
    const size_t ld = (size_t)p.n_tiles * 128;
    for (int i = 0; i < my_tiles; ++i) {
      const int buf = i & 1;
      const int tau = (int)blockIdx.x + i * (int)gridDim.x;
      const int nt = tau / p.m_tiles, mt = tau % p.m_tiles;
      if (!mbar_wait(&acc_full[buf], (i >> 1) & 1, p.status, 42)) break;
      tc_fence_after();
      const uint32_t taddr = tmem_base + ((uint32_t)(q * 32) << 16) + (uint32_t)(buf * GW_NT);
      float* dst = p.part + (size_t)nt * 128 + q * 32 + lane;
      const int m0 = mt * GW_NT;
#pragma unroll 2
      for (int g = hf * (GW_NT / 64); g < (hf + 1) * (GW_NT / 64); ++g) {
        uint32_t r[32];
        tmem_ld32(taddr + g * 32, r);
        tmem_ld_wait();
#pragma unroll
        for (int j = 0; j < 32; ++j) {
          const int m = m0 + g * 32 + j;
          if (m < p.M) dst[(size_t)m * ld] = __uint_as_float(r[j]);
        }
      }
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(&acc_empty[buf]);
    }
  }

  tc_fence_before();
  __syncthreads();
  if (warp == 1) tmem_dealloc(tmem_base, Cfg::TMEM_COLS);
}

}  // namespace spec
