// Weight-streaming bf16 linear for a few rows of activations (M = tree nodes): y = x W^T on
// the 5th-generation tensor cores. The operands are swapped so that 128 weight rows fill the
// MMA's M dimension and the MT activation rows sit in its N dimension: the accumulator
// D[128 weight rows][MT] lives in tensor memory, the weight tile and the activation tile are
// staged in shared memory by TMA (128-byte swizzle) through a multi-stage mbarrier ring, and
// a single thread issues tcgen05.mma. Each CTA computes one (weight tile, K slice, row tile)
// unit; K slices leave float32 partial sums that the consumer adds in slice order.
#pragma once
#include <cuda.h>

#include "common.cuh"

namespace spec {

enum { EPI_PARTIAL = 0, EPI_SWIGLU = 1, EPI_ARGMAX = 2 };

struct GemmTcParams {
  int M, N, K;          // activation rows, weight rows (output features), reduction length
  int splits;           // K slices (gridDim.y)
  int a2_row_offset;    // second 64-row half of the weight tile: row offset within its map
  int tile_rows;        // output features per tile: 128, or 64 gate + 64 up rows for SwiGLU
  // EPI_PARTIAL: out[s][m][n]
  float* out;
  size_t split_stride;
  int ldo;
  // EPI_SWIGLU: act[m][f] = bf16(SiLU(gate) * up), N = d_ffn
  bf16* act;
  int ld_act;
  // EPI_ARGMAX: per-tile (value, index) partials [tile][pstride]; optional logits [m][N]
  float* logits;
  float* pval;
  int* pidx;
  int pstride;
  int* status;
};

template <int MT> struct GemmTcCfg {
  static constexpr int BK = 64;                         // bf16 elements per stage along K (128 bytes)
  static constexpr int A_BYTES = 128 * BK * 2;          // 16 KiB
  static constexpr int B_BYTES = MT * BK * 2;
  static constexpr int STAGE_BYTES = A_BYTES + B_BYTES;
  static constexpr int STAGES = (MT <= 32) ? 5 : (MT == 64 ? 4 : 3);
  static constexpr int TMEM_COLS = MT < 32 ? 32 : MT;
  static constexpr int SMEM_BYTES = STAGES * STAGE_BYTES + 1024 /*alignment slack*/ + 256 /*barriers*/;
};

template <int MT, int EPI>
__global__ void __launch_bounds__(128, 1)
gemm_tc(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmA2,
        const __grid_constant__ CUtensorMap tmB, const GemmTcParams p) {
  using Cfg = GemmTcCfg<MT>;
  constexpr int STAGES = Cfg::STAGES;
  extern __shared__ uint8_t smem_raw[];
  const uint32_t raw = smem_u32(smem_raw);
  uint8_t* tiles = smem_raw + (((raw + 1023u) & ~1023u) - raw);
  uint64_t* bars = reinterpret_cast<uint64_t*>(tiles + STAGES * Cfg::STAGE_BYTES);
  uint64_t* full = bars;
  uint64_t* empty = bars + STAGES;
  uint64_t* accum = bars + 2 * STAGES;
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + 2 * STAGES + 1);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int nt = blockIdx.x, s = blockIdx.y, mt = blockIdx.z;
  const int KC = p.K / Cfg::BK;
  const int c0 = (int)(((long long)s * KC) / p.splits), c1 = (int)(((long long)(s + 1) * KC) / p.splits);
  const int n0 = nt * p.tile_rows;
  const int m0 = mt * MT;

  if (threadIdx.x == 0) {
    for (int i = 0; i < STAGES; ++i) { mbar_init(&full[i], 1); mbar_init(&empty[i], 1); }
    mbar_init(accum, 1);
    mbar_fence_init();
    tma_prefetch_desc(&tmA);
    tma_prefetch_desc(&tmA2);
    tma_prefetch_desc(&tmB);
  }
  if (warp == 1) { tmem_alloc(tmem_slot, Cfg::TMEM_COLS); tmem_relinquish(); }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;

  if (threadIdx.x == 0) {
    // ---- TMA producer ----
    int issued = 0;
    for (int c = c0; c < c1; ++c, ++issued) {
      int st = issued % STAGES;
      uint32_t ph = (issued / STAGES) & 1;
      if (!mbar_wait(&empty[st], ph ^ 1, p.status, 10)) break;
      uint8_t* a = tiles + st * Cfg::STAGE_BYTES;
      mbar_expect_tx(&full[st], Cfg::STAGE_BYTES);
      tma_load_2d(a, &tmA, c * Cfg::BK, n0, &full[st]);
      tma_load_2d(a + Cfg::A_BYTES / 2, &tmA2, c * Cfg::BK, n0 + p.a2_row_offset, &full[st]);
      tma_load_2d(a + Cfg::A_BYTES, &tmB, c * Cfg::BK, m0, &full[st]);
    }
  } else if (threadIdx.x == 32) {
    // ---- MMA issuer ----
    const uint32_t idesc = make_idesc_bf16(128, MT);
    int done = 0;
    bool ok = true;
    for (int c = c0; c < c1; ++c, ++done) {
      int st = done % STAGES;
      uint32_t ph = (done / STAGES) & 1;
      if (!mbar_wait(&full[st], ph, p.status, 11)) { ok = false; break; }
      tc_fence_after();
      uint32_t a_addr = smem_u32(tiles + st * Cfg::STAGE_BYTES);
      uint64_t adesc = make_kmajor_sw128_desc(a_addr);
      uint64_t bdesc = make_kmajor_sw128_desc(a_addr + Cfg::A_BYTES);
#pragma unroll
      for (int k = 0; k < Cfg::BK / 16; ++k) {
        // advance 16 bf16 = 32 bytes along K inside the swizzle atom: +2 in the address field
        tc_mma_f16(tmem_base, adesc + 2 * k, bdesc + 2 * k, idesc, (done > 0 || k > 0) ? 1u : 0u);
      }
      tc_commit(&empty[st]);
    }
    (void)ok;
    tc_commit(accum);
  }
  __syncwarp();

  // ---- epilogue: all four warps; warp w owns tensor-memory lanes [32w, 32w+32) ----
  bool have = mbar_wait(accum, 0, p.status, 12);
  tc_fence_after();
  const int nl = warp * 32 + lane;                 // lane in the accumulator = weight row in tile
  const uint32_t taddr = tmem_base + ((uint32_t)(warp * 32) << 16);

  if (EPI == EPI_PARTIAL) {
    const int n = n0 + nl;
    if (have) {
#pragma unroll 1
      for (int col = 0; col < MT; col += 16) {
        uint32_t r[16];
        tmem_ld16(taddr + col, r);
        tmem_ld_wait();
        if (n < p.N) {
#pragma unroll
          for (int j = 0; j < 16; ++j) {
            int m = m0 + col + j;
            if (m < p.M) p.out[(size_t)s * p.split_stride + (size_t)m * p.ldo + n] = __uint_as_float(r[j]);
          }
        }
      }
    }
  } else if (EPI == EPI_SWIGLU) {
    // lanes 0..63 hold gate rows, lanes 64..127 the matching up rows; exchange through the
    // (now idle) stage buffers
    float* ex = reinterpret_cast<float*>(tiles);   // [64][MT+1]
    if (have && warp >= 2) {
#pragma unroll 1
      for (int col = 0; col < MT; col += 16) {
        uint32_t r[16];
        tmem_ld16(taddr + col, r);
        tmem_ld_wait();
#pragma unroll
        for (int j = 0; j < 16; ++j) ex[(nl - 64) * (MT + 1) + col + j] = __uint_as_float(r[j]);
      }
    }
    __syncthreads();
    if (have && warp < 2) {
      const int f = n0 + nl;
#pragma unroll 1
      for (int col = 0; col < MT; col += 16) {
        uint32_t r[16];
        tmem_ld16(taddr + col, r);
        tmem_ld_wait();
        if (f < p.N) {
#pragma unroll
          for (int j = 0; j < 16; ++j) {
            int m = m0 + col + j;
            if (m < p.M) {
              float g = __uint_as_float(r[j]), u = ex[nl * (MT + 1) + col + j];
              p.act[(size_t)m * p.ld_act + f] = __float2bfloat16_rn(silu_f(g) * u);
            }
          }
        }
      }
    }
  } else {  // EPI_ARGMAX
    float* rv = reinterpret_cast<float*>(tiles);            // [4][MT]
    int* ri = reinterpret_cast<int*>(tiles + 4 * MT * 4);   // [4][MT]
    const int n = n0 + nl;
    if (have) {
#pragma unroll 1
      for (int col = 0; col < MT; col += 16) {
        uint32_t r[16];
        tmem_ld16(taddr + col, r);
        tmem_ld_wait();
#pragma unroll
        for (int j = 0; j < 16; ++j) {
          int m = m0 + col + j;
          float v = (n < p.N) ? __uint_as_float(r[j]) : -INFINITY;
          if (p.logits && n < p.N && m < p.M) p.logits[(size_t)m * p.N + n] = v;
          int idx = (n < p.N) ? n : 0x7fffffff;
          warp_argmax(v, idx);
          if (lane == 0) { rv[warp * MT + col + j] = v; ri[warp * MT + col + j] = idx; }
        }
      }
    }
    __syncthreads();
    if (have && threadIdx.x < MT && m0 + threadIdx.x < p.M) {
      float bv = rv[threadIdx.x];
      int bi = ri[threadIdx.x];
      for (int w = 1; w < 4; ++w)
        if (better(rv[w * MT + threadIdx.x], ri[w * MT + threadIdx.x], bv, bi)) {
          bv = rv[w * MT + threadIdx.x];
          bi = ri[w * MT + threadIdx.x];
        }
      p.pval[(size_t)nt * p.pstride + m0 + threadIdx.x] = bv;
      p.pidx[(size_t)nt * p.pstride + m0 + threadIdx.x] = bi;
    }
  }

  tc_fence_before();
  __syncthreads();
  if (warp == 1) tmem_dealloc(tmem_base, Cfg::TMEM_COLS);
}

}  // namespace spec
