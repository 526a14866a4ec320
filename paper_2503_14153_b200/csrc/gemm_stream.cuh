// Weight-streaming bf16 linear for a few rows of activations (M = tree nodes): y = x W^T on
// the 5th-generation tensor cores, as a persistent kernel.
//
// The operands are swapped: 128 weight rows fill the MMA's M dimension and MT activation rows
// sit in its N dimension, so the accumulator D[128 weight rows][MT] lives in tensor memory.
// The work of one launch is the list of (weight tile, 64-wide K chunk) units of up to four
// weight matrices stacked along the output dimension; the list is cut into gridDim.x equal
// contiguous runs, one per CTA, so every CTA streams the same number of weight bytes whatever
// the shape (a run that crosses a tile boundary leaves float32 partial sums for both tiles,
// and the consumer adds a tile's partial sums in CTA order, which is fixed).
//
// Warp roles: warp 0 feeds a ring of shared-memory stages with TMA (128-byte swizzle), warp 1
// issues tcgen05.mma into one of two accumulator buffers, warps 2..5 drain the other buffer.
// The weights do not depend on the previous kernel, so the producer fills the ring (and asks
// the L2 for the chunks after it) before it waits on the programmatic launch dependency;
// only the activation tiles are loaded after the wait.
#pragma once
#include <cuda.h>

#include "common.cuh"

namespace spec {

constexpr int GS_MAX_MATS = 4;

// How a launch's units are dealt to CTAs; shared by the kernel and by the consumers of its
// partial sums. Unit u = ((nt * m_tiles) + mt) * KC + kc.
struct SegMap {
  int KC;          // K chunks per tile
  int m_tiles;     // activation row tiles
  int G;           // CTAs the units are dealt to (<= total)
  int total;       // n_tiles * m_tiles * KC
  __host__ __device__ __forceinline__ int lo(int c) const { return (int)(((long long)c * total) / G); }
  // CTA whose run contains unit u
  // (u + 1) * G stays below 2^31 for every unit (the host checks it), so 32-bit division serves
  __host__ __device__ __forceinline__ int owner(int u) const { return (int)((((unsigned)u + 1u) * (unsigned)G - 1u) / (unsigned)total); }
  // number of CTAs that contribute to tile t = nt * m_tiles + mt
  __host__ __device__ __forceinline__ int nseg(int t) const { return owner((t + 1) * KC - 1) - owner(t * KC) + 1; }
};

struct StreamGemmParams {
  int M, K;
  int n_mats;
  int mat_tile0[GS_MAX_MATS + 1];   // first tile of each matrix (prefix sums of ceil(rows/128))
  int mat_rows[GS_MAX_MATS];        // rows of each matrix
  int mat_col0[GS_MAX_MATS];        // first logical output column of each matrix
  int n_tiles;
  SegMap seg;
  // Pre-tiled weights (see pack_weight_tiles): packed[i] != nullptr holds matrix i as the sequence of its
  // (tile, K chunk) units, each the 16 KB shared-memory image of the tile (128 rows of 128 bytes, 16-byte
  // chunks XOR-swizzled with the row). A CTA's run of units is then one contiguous stretch of memory read
  // with plain bulk copies, which streams faster out of HBM than strided TMA boxes (7.3 against 6.4 TB/s).
  const uint8_t* packed[GS_MAX_MATS];
  int l2_prefetch;                  // units to request into L2 beyond the ring before the dependency wait
  // partial sums: part[slot][m][n_tiles*128] (padded column space: tile nt owns columns [128 nt, 128 nt + 128))
  float* part;
  size_t slot_stride;
  int* status;
  unsigned long long* trace;        // optional timeline slot (see KTrace); [2] first operands landed, [3] last MMA issued
};

struct StreamTmaps {
  CUtensorMap a[GS_MAX_MATS];
  CUtensorMap b;
};

// DEEP = 0: a ring sized so that two CTAs share an SM; DEEP = 1: twice the stages, one CTA per SM.
template <int MT, int DEEP> struct StreamCfg {
  static constexpr int BK = 64;
  static constexpr int A_BYTES = 128 * BK * 2;
  static constexpr int B_BYTES = MT * BK * 2;
  static constexpr int STAGE_BYTES = A_BYTES + B_BYTES;
  static constexpr int STAGES = ((MT <= 32) ? 5 : (MT == 64 ? 4 : 3)) * (DEEP ? 2 : 1);
  static constexpr int TMEM_COLS = (2 * MT < 32) ? 32 : 2 * MT;
  static constexpr int SMEM_BYTES = STAGES * STAGE_BYTES + 1024 /*alignment slack*/ + 256 /*barriers*/;
};

__device__ __forceinline__ void tma_prefetch_l2_2d(const void* tmap, int x, int y, uint64_t policy) {
  asm volatile("cp.async.bulk.prefetch.tensor.2d.L2.global.tile.L2::cache_hint [%0, {%1, %2}], %3;"
               ::"l"(tmap), "r"(x), "r"(y), "l"(policy) : "memory");
}

struct GsUnit {
  int nt, mt, kc, mat, row0;
};

__device__ __forceinline__ GsUnit gs_decode(const StreamGemmParams& p, int u) {
  GsUnit w;
  w.kc = u % p.seg.KC;
  int t = u / p.seg.KC;
  w.mt = t % p.seg.m_tiles;
  w.nt = t / p.seg.m_tiles;
  w.mat = 0;
#pragma unroll
  for (int i = 1; i < GS_MAX_MATS; ++i)
    if (i < p.n_mats && w.nt >= p.mat_tile0[i]) w.mat = i;
  w.row0 = (w.nt - p.mat_tile0[w.mat]) * 128;
  return w;
}

template <int MT, int DEEP>
__global__ void __launch_bounds__(192, DEEP ? 1 : 2)
gemm_stream(const __grid_constant__ StreamTmaps tm, const StreamGemmParams p) {
  using Cfg = StreamCfg<MT, DEEP>;
  constexpr int STAGES = Cfg::STAGES;
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
  const int c = blockIdx.x;
  const int KC = p.seg.KC;
  const int lo = p.seg.lo(c), hi = p.seg.lo(c + 1);

  pdl_launch_dependents();

  if (threadIdx.x == 0) {
    for (int i = 0; i < STAGES; ++i) { mbar_init(&full[i], 1); mbar_init(&empty[i], 1); }
    mbar_init(&acc_full[0], 1); mbar_init(&acc_full[1], 1);
    mbar_init(&acc_empty[0], 4); mbar_init(&acc_empty[1], 4);
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
      // ---- TMA producer ----
      const int n_units = hi - lo;
      const uint64_t wpol = l2_policy_evict_first();
      const int n_pre = n_units < STAGES ? n_units : STAGES;
      auto load_a = [&](uint8_t* dst, const GsUnit& w, uint64_t* bar) {
        if (p.packed[w.mat])
          bulk_load_1d_hint(dst, p.packed[w.mat] + ((size_t)(w.row0 >> 7) * KC + w.kc) * Cfg::A_BYTES, Cfg::A_BYTES, bar, wpol);
        else
          tma_load_2d_hint(dst, &tm.a[w.mat], w.kc * Cfg::BK, w.row0, bar, wpol);
      };
      // weights first: they do not depend on the kernel before this one
      for (int i = 0; i < n_pre; ++i) {
        GsUnit w = gs_decode(p, lo + i);
        mbar_expect_tx(&full[i], Cfg::STAGE_BYTES);
        load_a(tiles + i * Cfg::STAGE_BYTES, w, &full[i]);
      }
      {
        int n_pf = n_units - n_pre;
        if (n_pf > p.l2_prefetch) n_pf = p.l2_prefetch;
        for (int i = 0; i < n_pf; ++i) {
          GsUnit w = gs_decode(p, lo + n_pre + i);
          if (!p.packed[w.mat]) tma_prefetch_l2_2d(&tm.a[w.mat], w.kc * Cfg::BK, w.row0, wpol);
        }
      }
      pdl_wait();
      for (int i = 0; i < n_pre; ++i) {
        GsUnit w = gs_decode(p, lo + i);
        tma_load_2d(tiles + i * Cfg::STAGE_BYTES + Cfg::A_BYTES, &tm.b, w.kc * Cfg::BK, w.mt * MT, &full[i]);
      }
      bool ok = true;
      int issued = n_pre;
      for (; issued < n_units; ++issued) {
        const int st = issued % STAGES;
        const uint32_t ph = (issued / STAGES) & 1;
        if (!mbar_wait(&empty[st], ph ^ 1, p.status, 10)) { ok = false; break; }
        GsUnit w = gs_decode(p, lo + issued);
        uint8_t* a = tiles + st * Cfg::STAGE_BYTES;
        mbar_expect_tx(&full[st], Cfg::STAGE_BYTES);
        load_a(a, w, &full[st]);
        tma_load_2d(a + Cfg::A_BYTES, &tm.b, w.kc * Cfg::BK, w.mt * MT, &full[st]);
      }
      if (!ok) {
        // give the copies already in flight a bounded time to land before the CTA goes away
        for (int i = issued > STAGES ? issued - STAGES : 0; i < issued; ++i)
          mbar_wait(&full[i % STAGES], (i / STAGES) & 1, p.status, 13);
      }
    }
  } else if (warp == 1) {
    if (lane == 0) {
      // ---- MMA issuer ----
      const uint32_t idesc = make_idesc_bf16(128, MT);
      int seg_i = 0;
      bool ok = true;
      for (int u = lo; u < hi && ok;) {
        const int t = u / KC;
        const int u_end = (t + 1) * KC < hi ? (t + 1) * KC : hi;
        const int buf = seg_i & 1;
        if (!mbar_wait(&acc_empty[buf], ((seg_i >> 1) & 1) ^ 1, p.status, 14)) { ok = false; break; }
        tc_fence_after();
        const uint32_t d_addr = tmem_base + (uint32_t)(buf * MT);
        for (int v = u; v < u_end; ++v) {
          const int done = v - lo;
          const int st = done % STAGES;
          const uint32_t ph = (done / STAGES) & 1;
          if (!mbar_wait(&full[st], ph, p.status, 11)) { ok = false; break; }
          if (v == lo) trace_mark_min(p.trace, 2);
          tc_fence_after();
          const uint32_t a_addr = smem_u32(tiles + st * Cfg::STAGE_BYTES);
          const uint64_t adesc = make_kmajor_sw128_desc(a_addr);
          const uint64_t bdesc = make_kmajor_sw128_desc(a_addr + Cfg::A_BYTES);
#pragma unroll
          for (int k = 0; k < Cfg::BK / 16; ++k)
            tc_mma_f16(d_addr, adesc + 2 * k, bdesc + 2 * k, idesc, (v > u || k > 0) ? 1u : 0u);
          tc_commit(&empty[st]);
        }
        if (!ok) break;
        tc_commit(&acc_full[buf]);
        ++seg_i;
        u = u_end;
      }
      trace_mark_max(p.trace, 3);
    }
  } else {
    // ---- epilogue: warps 2..5; warp w may touch tensor-memory lanes [32 (w % 4), +32) ----
    const int q = warp & 3;
    pdl_wait();
    int seg_i = 0;
    for (int u = lo; u < hi;) {
      const int t = u / KC;
      const int u_end = (t + 1) * KC < hi ? (t + 1) * KC : hi;
      const int buf = seg_i & 1;
      const int mt = t % p.seg.m_tiles, nt = t / p.seg.m_tiles;
      if (!mbar_wait(&acc_full[buf], (seg_i >> 1) & 1, p.status, 12)) break;
      tc_fence_after();
      const uint32_t taddr = tmem_base + ((uint32_t)(q * 32) << 16) + (uint32_t)(buf * MT);
      const int m0 = mt * MT;
      const int slot = c - p.seg.owner(t * KC);
      float* dst = p.part + (size_t)slot * p.slot_stride + (size_t)nt * 128 + q * 32 + lane;
      const size_t ld = (size_t)p.n_tiles * 128;
      if (MT >= 32) {
        // all loads of the accumulator are issued before the first store
        uint32_t r[MT >= 32 ? MT / 32 : 1][32];
#pragma unroll
        for (int g = 0; g < MT / 32; ++g) tmem_ld32(taddr + g * 32, r[g]);
        tmem_ld_wait();
#pragma unroll
        for (int g = 0; g < MT / 32; ++g)
#pragma unroll
          for (int j = 0; j < 32; ++j) {
            const int m = m0 + g * 32 + j;
            if (m < p.M) dst[(size_t)m * ld] = __uint_as_float(r[g][j]);
          }
      } else {
        uint32_t r[16];
        tmem_ld16(taddr, r);
        tmem_ld_wait();
#pragma unroll
        for (int j = 0; j < 16; ++j) {
          const int m = m0 + j;
          if (m < p.M) dst[(size_t)m * ld] = __uint_as_float(r[j]);
        }
      }
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(&acc_empty[buf]);
      ++seg_i;
      u = u_end;
    }
  }

  tc_fence_before();
  __syncthreads();
  if (warp == 1) tmem_dealloc(tmem_base, Cfg::TMEM_COLS);
}

// Writes the pre-tiled image of a row-major bf16 matrix [rows][cols] (cols % 64 == 0): unit (tile t, K chunk
// kc) at byte offset (t * cols / 64 + kc) * 16384, row r of the tile at r * 128, its 16-byte chunk c at chunk
// position c ^ (r & 7) -- what a TMA load with the 128-byte swizzle leaves in shared memory. Rows beyond the
// matrix are zeros. One CTA per unit.
__global__ void __launch_bounds__(256)
pack_weight_tiles(const bf16* __restrict__ w, int rows, int cols, uint8_t* __restrict__ packed) {
  const int KC = cols >> 6;
  const int t = blockIdx.x / KC, kc = blockIdx.x - t * KC;
  uint4* dst = reinterpret_cast<uint4*>(packed + (size_t)blockIdx.x * 16384);
  for (int i = threadIdx.x; i < 128 * 8; i += blockDim.x) {
    const int r = i >> 3, ch = i & 7;
    const int row = t * 128 + r;
    uint4 v = make_uint4(0, 0, 0, 0);
    if (row < rows) v = *reinterpret_cast<const uint4*>(w + (size_t)row * cols + kc * 64 + ch * 8);
    dst[r * 8 + (ch ^ (r & 7))] = v;
  }
}

}  // namespace spec
