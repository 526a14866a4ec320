// Weight-streaming bf16 linear whose split-K partial sums never leave the chip: the CTAs that
// share an output tile form a thread-block cluster and exchange their float32 accumulators through
// distributed shared memory, so the kernel writes finished results and the element-wise step that
// used to follow in a kernel of its own runs in the epilogue. The residual and SwiGLU modes push: once
// every CTA's MMAs are complete (first cluster barrier; every ring is free then) a thread sends the
// values of its weight row with remote stores, which nobody waits for, into the shared memory of the
// CTA that finishes that column; after the second barrier each CTA reads only its own shared memory.
// (Reading the parts out of the other CTAs' shared memory instead cost 3 us more per kernel.)
//
// Three modes (operands swapped as in gemm_stream: 128 weight rows are the MMA's M, the MT activation
// rows its N; MT covers all rows of the pass):
//  * GC_RESIDUAL (output and down projections): a cluster of 8 CTAs per 128-row weight tile, CTA r
//    streaming the r-th eighth of the K chunks. CTA r owns output columns [16 r, 16 r + 16) of the
//    tile: it adds the eight parts in rank order, adds the residual stream x in place (old values
//    fetched during the exchange) and leaves the sum of squares of its piece of every row (the RMSNorm
//    that follows needs the row's mean square) in ss_part[m][tile * 8 + r].
//  * GC_SWIGLU (gate and up projections): a cluster of 3 CTAs per pair (gate tile t, up tile t); the
//    2 KC units of the pair are cut into three equal runs, so CTA 0 holds a gate part, CTA 1 a gate
//    and an up part (two accumulators) and CTA 2 an up part. Once every CTA's MMAs are complete (first
//    barrier) each thread sends the values of its weight row into the shared memory of the CTA that finishes
//    that column (remote stores); after the second barrier each CTA finishes a third of the tile's columns
//    from its own shared memory: gate = G0 + G1, up = U1 + U2, act = bf16(SiLU(gate) * up).
//  * GC_ROPE (query, key and value projections, stacked): a cluster of 2 CTAs per 128-row tile of the
//    stacked matrices, each streaming half of the K chunks (96 pairs on the 7B shape: all co-resident, which
//    96 clusters of 3 are not). A tile holds whole heads (head_dim 64 or
//    128), so after the barrier the cluster rotates the query / key pairs (i, i + head_dim / 2) by the
//    row's position, writes the bf16 query rows and puts the bf16 key and value rows into the paged cache
//    at the row's slot; CTA r takes every second activation row.
// Sums are added in a fixed order: results are bit-reproducible. Every wait is bounded; a CTA whose
// wait ran out still arrives at both cluster barriers, so its cluster mates never wait for it.
#pragma once
#include <cuda.h>

#include "common.cuh"
#include "gemm_stream.cuh"

namespace spec {

constexpr int GC_RESIDUAL = 0, GC_SWIGLU = 1, GC_ROPE = 2;
constexpr int GC_RES_CLUSTER = 8, GC_GLU_CLUSTER = 3, GC_ROPE_CLUSTER = 2;

struct ClusterGemmParams {
  int M, K, KC;                 // activation rows (<= MT), inner size, K / 64
  int N;                        // weight rows of one matrix (output columns)
  const uint8_t* packed[3];     // pre-tiled images (GC_RESIDUAL: [0]; GC_SWIGLU: gate, up; GC_ROPE: q, k, v) or nullptr -> tensor maps a[i]
  float* x;                     // GC_RESIDUAL: [M][N] float32 residual stream, updated in place
  float* ss_part;               // GC_RESIDUAL: [M][ceil(N/128) * 8] sums of squares of the updated pieces, or nullptr
  bf16* act;                    // GC_SWIGLU: [M][N] bf16
  // GC_ROPE: tiles [0, tile0[1]) belong to q, [tile0[1], tile0[2]) to k, the rest to v
  int tile0[3];
  int H;                        // query heads
  int layer;
  Rows rows;
  const float2* cs;             // [position][head_dim / 2] (cos, sin)
  bf16* q;                      // [M][H * head_dim]
  bf16* pool;                   // paged KV cache
  KVGeom g;
  const int* page_table;
  int* status;
  unsigned long long* trace;
};

template <int MT> struct ClusterCfg {
  static constexpr int BK = 64;
  static constexpr int A_BYTES = 128 * BK * 2;
  static constexpr int B_BYTES = MT * BK * 2;
  static constexpr int STAGE_BYTES = A_BYTES + B_BYTES;
  static constexpr int STAGES = (MT <= 32) ? 5 : (MT == 64 ? 4 : 3);
  static constexpr int PITCH = 132;                          // floats per staged activation row: 128 weight rows + 4 (16-byte aligned rows, banks shifted by 4)
  static constexpr int STAGING_FLOATS = MT * PITCH;          // one accumulator, staged as [activation row][weight row]
  static constexpr int RING_BYTES = STAGES * STAGE_BYTES;
  static constexpr int SMEM_BYTES = RING_BYTES + 1024 /*alignment slack*/ + 256 /*barriers*/;
};

__device__ __forceinline__ uint32_t cluster_ctarank() {
  uint32_t r;
  asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
  return r;
}
__device__ __forceinline__ void cluster_sync_all() {
  asm volatile("barrier.cluster.arrive.release.aligned;\n\tbarrier.cluster.wait.acquire.aligned;" ::: "memory");
}
__device__ __forceinline__ uint32_t dsmem_addr(uint32_t local_smem_addr, uint32_t rank) {
  uint32_t a;
  asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(a) : "r"(local_smem_addr), "r"(rank));
  return a;
}
__device__ __forceinline__ float4 dsmem_ld4(uint32_t addr) {
  float4 v;
  asm volatile("ld.shared::cluster.v4.f32 {%0, %1, %2, %3}, [%4];" : "=f"(v.x), "=f"(v.y), "=f"(v.z), "=f"(v.w) : "r"(addr) : "memory");
  return v;
}
__device__ __forceinline__ void dsmem_st(uint32_t addr, float v) {
  asm volatile("st.shared::cluster.f32 [%0], %1;" ::"r"(addr), "f"(v) : "memory");
}
__device__ __forceinline__ void add4(float4& a, const float4& b) { a.x += b.x; a.y += b.y; a.z += b.z; a.w += b.w; }

__device__ __forceinline__ uint32_t pack_bf16x2(float lo, float hi) {
  __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
  return *reinterpret_cast<uint32_t*>(&v);
}

// One run of K chunks of one weight tile, accumulated into one tensor-memory buffer.
struct GcSeg {
  int mat, kc0, kc1;
};

template <int MT, int MODE>
__global__ void __launch_bounds__(192, 2)
gemm_cluster(const __grid_constant__ StreamTmaps tm, const ClusterGemmParams p) {
  using Cfg = ClusterCfg<MT>;
  constexpr int STAGES = Cfg::STAGES;
  constexpr int CS = MODE == GC_RESIDUAL ? GC_RES_CLUSTER : (MODE == GC_SWIGLU ? GC_GLU_CLUSTER : GC_ROPE_CLUSTER);
  constexpr int TMEM_COLS = ((MODE == GC_SWIGLU ? 2 : 1) * MT < 32) ? 32 : (MODE == GC_SWIGLU ? 2 : 1) * MT;   // 32, 64 or 128
  static_assert(MODE != GC_SWIGLU || 2 * Cfg::STAGING_FLOATS * 4 <= Cfg::RING_BYTES, "two staged accumulators must fit the ring");
  static_assert(Cfg::STAGING_FLOATS * 4 <= Cfg::RING_BYTES, "a staged accumulator must fit the ring");
  extern __shared__ uint8_t smem_raw[];
  const uint32_t raw = smem_u32(smem_raw);
  uint8_t* tiles = smem_raw + (((raw + 1023u) & ~1023u) - raw);
  uint64_t* bars = reinterpret_cast<uint64_t*>(tiles + Cfg::RING_BYTES);
  uint64_t* full = bars;
  uint64_t* empty = bars + STAGES;
  uint64_t* acc_full = bars + 2 * STAGES;
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + 2 * STAGES + 1);
  float* staging = reinterpret_cast<float*>(tiles);          // reuses the ring once every MMA is complete

  KTrace kt(p.trace);
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int rank = (int)cluster_ctarank();
  const int t = blockIdx.x / CS;                             // weight tile (GC_SWIGLU: tile pair; GC_ROPE: of the stacked q, k, v)
  const int KC = p.KC;
  int rope_mat = 0;
  if (MODE == GC_ROPE) rope_mat = t >= p.tile0[2] ? 2 : (t >= p.tile0[1] ? 1 : 0);
  const int t_in_mat = MODE == GC_ROPE ? t - p.tile0[rope_mat] : t;

  // this CTA's runs
  GcSeg seg[2];
  int nseg = 0;
  if (MODE != GC_SWIGLU) {
    seg[0] = GcSeg{rope_mat, rank * KC / CS, (rank + 1) * KC / CS};
    nseg = 1;
  } else {
    const int u_lo = rank * 2 * KC / CS, u_hi = (rank + 1) * 2 * KC / CS;
    if (u_lo < KC) seg[nseg++] = GcSeg{0, u_lo, u_hi < KC ? u_hi : KC};
    if (u_hi > KC) seg[nseg++] = GcSeg{1, u_lo > KC ? u_lo - KC : 0, u_hi - KC};
  }
  const int n_units = (seg[0].kc1 - seg[0].kc0) + (nseg > 1 ? seg[1].kc1 - seg[1].kc0 : 0);

  pdl_launch_dependents();

  if (threadIdx.x == 0) {
    for (int i = 0; i < STAGES; ++i) { mbar_init(&full[i], 1); mbar_init(&empty[i], 1); }
    mbar_init(acc_full, 1);
    mbar_fence_init();
    for (int i = 0; i < (MODE == GC_RESIDUAL ? 1 : (MODE == GC_SWIGLU ? 2 : 3)); ++i) if (!p.packed[i]) tma_prefetch_desc(&tm.a[i]);
    tma_prefetch_desc(&tm.b);
  }
  if (warp == 1) { tmem_alloc(tmem_slot, TMEM_COLS); tmem_relinquish(); }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;

  // unit i of this CTA -> (segment, K chunk)
  auto unit = [&](int i, int& s, int& kc) {
    const int n0 = seg[0].kc1 - seg[0].kc0;
    if (i < n0) { s = 0; kc = seg[0].kc0 + i; } else { s = 1; kc = seg[1].kc0 + (i - n0); }
  };

  // GC_ROPE: what a finishing thread needs to know about its items (row bookkeeping, cos / sin, destination) is
  // fetched by the epilogue warps while the MMAs run, not after the cluster barrier
  constexpr int R_ROWS_MAX = (MT + GC_ROPE_CLUSTER - 1) / GC_ROPE_CLUSTER, R_ITEMS = R_ROWS_MAX * 16;
  constexpr int R_PER = MODE == GC_ROPE ? (R_ITEMS + 127) / 128 : 1;
  bool r_on[R_PER];
  int r_mrow[R_PER], r_lo_c[R_PER];
  float4 r_cs01[R_PER], r_cs23[R_PER];
  bf16* r_dst[R_PER];
  auto rope_meta = [&]() {
    constexpr int ITEMS = R_ITEMS, PER = R_PER;
    const int e = threadIdx.x - 64;
    const int D = p.g.head_dim, half = D >> 1, gph = half >> 2;       // pair groups per head
    const int n_rows_mat = rope_mat == 0 ? p.H * D : p.g.n_kv_heads * D;
    bool (&on)[R_PER] = r_on;
    int (&mrow)[R_PER] = r_mrow, (&lo_c)[R_PER] = r_lo_c;
    float4 (&cs01)[R_PER] = r_cs01, (&cs23)[R_PER] = r_cs23;
    bf16* (&dst)[R_PER] = r_dst;
#pragma unroll
      for (int k = 0; k < PER; ++k) {
        const int it = e + 128 * k, ml = it >> 4, pg = it & 15;
        const int m = rank + CS * ml;
        const int hh = pg / gph, g = pg % gph;
        lo_c[k] = hh * D + 4 * g;
        mrow[k] = m;
        const int row_lo = t_in_mat * 128 + lo_c[k];                      // weight row within its matrix
        on[k] = it < ITEMS && m < p.M && row_lo < n_rows_mat;
        cs01[k] = cs23[k] = make_float4(1.f, 0.f, 1.f, 0.f);
        dst[k] = nullptr;
        if (on[k]) {
          const int b = m / p.rows.R, ri = m % p.rows.R;
          on[k] = ri < p.rows.cnt[b];
          const int head = row_lo / D, i = 4 * g;
          if (rope_mat < 2) {
            const float2* c = p.cs + (size_t)p.rows.pos[m] * half + i;
            cs01[k] = *reinterpret_cast<const float4*>(c);
            cs23[k] = *reinterpret_cast<const float4*>(c + 2);
          }
          if (rope_mat == 0) {
            dst[k] = p.q + (size_t)m * p.H * D + head * D + i;
          } else {
            const int slot = p.rows.slot[m];
            const int page = p.page_table[b * p.g.pages_per_seq + slot / p.g.page_size], prow = slot % p.g.page_size;
            // (a group of four lies inside one 16-byte chunk of the row: the chunk swizzle keeps it contiguous)
            dst[k] = p.pool + p.g.block_offset(page, p.layer, rope_mat - 1, head) + (size_t)prow * D + kv_elem<bf16>(prow, i, D, p.g.page_size);
            lo_c[k] |= (kv_elem<bf16>(prow, i + half, D, p.g.page_size) - kv_elem<bf16>(prow, i, D, p.g.page_size)) << 16;   // distance to the upper half's group
          }
        }
      }
  };

  if (warp == 0) {
    if (lane == 0) {
      // ---- producer: weights before the dependency wait, activation tiles after it ----
      const uint64_t wpol = l2_policy_evict_first();
      const int n_pre = n_units < STAGES ? n_units : STAGES;
      auto load_a = [&](uint8_t* dst, int s, int kc, uint64_t* bar) {
        const int mat = seg[s].mat;
        if (p.packed[mat])
          bulk_load_1d_hint(dst, p.packed[mat] + ((size_t)t_in_mat * KC + kc) * Cfg::A_BYTES, Cfg::A_BYTES, bar, wpol);
        else
          tma_load_2d_hint(dst, &tm.a[mat], kc * Cfg::BK, t_in_mat * 128, bar, wpol);
      };
      for (int i = 0; i < n_pre; ++i) {
        int s, kc;
        unit(i, s, kc);
        mbar_expect_tx(&full[i], Cfg::STAGE_BYTES);
        load_a(tiles + i * Cfg::STAGE_BYTES, s, kc, &full[i]);
      }
      pdl_wait();
      for (int i = 0; i < n_pre; ++i) {
        int s, kc;
        unit(i, s, kc);
        tma_load_2d(tiles + i * Cfg::STAGE_BYTES + Cfg::A_BYTES, &tm.b, kc * Cfg::BK, 0, &full[i]);
      }
      bool ok = true;
      int issued = n_pre;
      for (; issued < n_units; ++issued) {
        const int st = issued % STAGES;
        const uint32_t ph = (issued / STAGES) & 1;
        if (!mbar_wait(&empty[st], ph ^ 1, p.status, 30)) { ok = false; break; }
        int s, kc;
        unit(issued, s, kc);
        uint8_t* a = tiles + st * Cfg::STAGE_BYTES;
        mbar_expect_tx(&full[st], Cfg::STAGE_BYTES);
        load_a(a, s, kc, &full[st]);
        tma_load_2d(a + Cfg::A_BYTES, &tm.b, kc * Cfg::BK, 0, &full[st]);
      }
      if (!ok) {
        for (int i = issued > STAGES ? issued - STAGES : 0; i < issued; ++i)
          mbar_wait(&full[i % STAGES], (i / STAGES) & 1, p.status, 33);
      }
    }
  } else if (warp == 1) {
    if (lane == 0) {
      // ---- MMA issuer: one accumulator per run ----
      const uint32_t idesc = make_idesc_bf16(128, MT);
      bool ok = true;
      int done = 0;
      for (int s = 0; s < nseg && ok; ++s) {
        const uint32_t d_addr = tmem_base + (uint32_t)(s * MT);
        const int n = seg[s].kc1 - seg[s].kc0;
        for (int v = 0; v < n; ++v, ++done) {
          const int st = done % STAGES;
          const uint32_t ph = (done / STAGES) & 1;
          if (!mbar_wait(&full[st], ph, p.status, 31)) { ok = false; break; }
          if (done == 0) trace_mark_min(p.trace, 2);
          tc_fence_after();
          const uint32_t a_addr = smem_u32(tiles + st * Cfg::STAGE_BYTES);
          const uint64_t adesc = make_kmajor_sw128_desc(a_addr);
          const uint64_t bdesc = make_kmajor_sw128_desc(a_addr + Cfg::A_BYTES);
#pragma unroll
          for (int k = 0; k < Cfg::BK / 16; ++k)
            tc_mma_f16(d_addr, adesc + 2 * k, bdesc + 2 * k, idesc, (v > 0 || k > 0) ? 1u : 0u);
          tc_commit(&empty[st]);
        }
      }
      if (ok) tc_commit(acc_full);         // arrives once every MMA above is complete (and has read its operands)
      trace_mark_max(p.trace, 3);
    }
  } else {
    // ---- epilogue, part 1: accumulators -> staged float32 rows [weight row][activation row] ----
    const int q = warp & 3;
    pdl_wait();
    if (MODE == GC_ROPE) rope_meta();
    if (MODE == GC_SWIGLU || MODE == GC_RESIDUAL) {
      // the accumulators stay in tensor memory until every CTA of the cluster has finished its MMAs (below)
      if (n_units > 0) mbar_wait(acc_full, 0, p.status, 32);
    } else if (n_units > 0 && mbar_wait(acc_full, 0, p.status, 32)) {
      tc_fence_after();
      for (int s = 0; s < nseg; ++s) {
        const uint32_t taddr = tmem_base + ((uint32_t)(q * 32) << 16) + (uint32_t)(s * MT);
        // thread = weight row q * 32 + lane; a warp writes 32 neighbouring floats of one activation row at a time
        float* dst = staging + (size_t)s * Cfg::STAGING_FLOATS + (q * 32 + lane);
        if (MT >= 32) {
#pragma unroll
          for (int g = 0; g < MT / 32; ++g) {
            uint32_t r[32];
            tmem_ld32(taddr + g * 32, r);
            tmem_ld_wait();
#pragma unroll
            for (int j = 0; j < 32; ++j) dst[(size_t)(g * 32 + j) * Cfg::PITCH] = __uint_as_float(r[j]);
          }
        } else {
          uint32_t r[16];
          tmem_ld16(taddr, r);
          tmem_ld_wait();
#pragma unroll
          for (int j = 0; j < 16; ++j) dst[(size_t)j * Cfg::PITCH] = __uint_as_float(r[j]);
        }
      }
      tc_fence_before();
    }
  }

  // ---- every thread of every CTA of the cluster: the staged accumulators are complete (GC_SWIGLU: every CTA's
  // MMAs are complete, so every ring is free) ----
  __syncwarp();
  cluster_sync_all();

  if (MODE == GC_RESIDUAL) {
    // Pushed like the gate+up parts below: a thread sends the MT values of its weight row w into the shared memory
    // of the CTA that finishes column w (CTA w / 16), buffer [source CTA][activation row][16 columns]; after the
    // second barrier CTA `rank` adds the eight parts of its columns [16 rank, +16) in rank order, adds the residual
    // stream in place (its old values were fetched during the exchange) and leaves the sums of squares.
    constexpr int CP = 16;
    static_assert(CS * MT * CP * 4 <= Cfg::RING_BYTES, "the parts of a CTA's columns must fit the ring");
    constexpr int ITEMS = MT * 4, PER = (ITEMS + 127) / 128;   // (row m, group of four columns c4)
    const int e = threadIdx.x - 64;
    const bool fin = warp >= 2 && n_units > 0;
    float4 xo[PER];
    bool on[PER];
    if (fin) {
#pragma unroll
      for (int k = 0; k < PER; ++k) {
        const int it = e + 128 * k, m = it >> 2, c4 = it & 3;
        const int col = t * 128 + rank * 16 + c4 * 4;
        on[k] = it < ITEMS && m < p.M && col < p.N;
        xo[k] = on[k] ? *reinterpret_cast<const float4*>(p.x + (size_t)m * p.N + col) : make_float4(0.f, 0.f, 0.f, 0.f);
      }
      const int q = warp & 3, w = q * 32 + lane;
      const uint32_t dst = dsmem_addr(smem_u32(staging), (uint32_t)(w >> 4)) + (uint32_t)((rank * MT * CP + (w & 15)) * 4);
      const uint32_t taddr = tmem_base + ((uint32_t)(q * 32) << 16);
      tc_fence_after();
      if (MT >= 32) {
#pragma unroll
        for (int g = 0; g < MT / 32; ++g) {
          uint32_t r[32];
          tmem_ld32(taddr + g * 32, r);
          tmem_ld_wait();
#pragma unroll
          for (int j = 0; j < 32; ++j) dsmem_st(dst + (uint32_t)((g * 32 + j) * CP * 4), __uint_as_float(r[j]));
        }
      } else {
        uint32_t r[16];
        tmem_ld16(taddr, r);
        tmem_ld_wait();
#pragma unroll
        for (int j = 0; j < 16; ++j) dsmem_st(dst + (uint32_t)(j * CP * 4), __uint_as_float(r[j]));
      }
      tc_fence_before();
    }
    __syncwarp();
    cluster_sync_all();                                       // the parts have arrived (release / acquire)
    if (fin) {
      float ss[PER];
#pragma unroll
      for (int k = 0; k < PER; ++k) {
        const int it = e + 128 * k, m = it >> 2, c4 = it & 3;
        float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
        if (it < ITEMS) {
          const float* src = staging + m * CP + c4 * 4;
#pragma unroll
          for (int rr = 0; rr < CS; ++rr) add4(acc, *reinterpret_cast<const float4*>(src + rr * MT * CP));   // rank order
        }
        add4(xo[k], acc);
        ss[k] = xo[k].x * xo[k].x + xo[k].y * xo[k].y + xo[k].z * xo[k].z + xo[k].w * xo[k].w;
        if (on[k]) *reinterpret_cast<float4*>(p.x + (size_t)m * p.N + t * 128 + rank * 16 + c4 * 4) = xo[k];
      }
      if (p.ss_part) {
        // the four column groups of a row sit in four neighbouring lanes
#pragma unroll
        for (int k = 0; k < PER; ++k) {
          float v = on[k] ? ss[k] : 0.f;
          v += __shfl_xor_sync(0xffffffffu, v, 1);
          v += __shfl_xor_sync(0xffffffffu, v, 2);
          const int it = e + 128 * k, m = it >> 2;
          if ((it & 3) == 0 && it < ITEMS && m < p.M)
            p.ss_part[(size_t)m * (((p.N + 127) >> 7) * CS) + t * CS + rank] = v;
        }
      }
    }
    tc_fence_before();
    __syncthreads();
    if (warp == 1) tmem_dealloc(tmem_base, TMEM_COLS);
    return;
  }

  if (MODE == GC_SWIGLU) {
    // Push instead of pull: a thread owns weight row w of its CTA's accumulators and sends its MT values
    // straight into the shared memory of the CTA that finishes column w (rows 0..43 -> CTA 0, 44..83 -> CTA 1,
    // 84..127 -> CTA 2) with remote stores, which nobody waits for; after the next barrier each CTA reads only
    // its own shared memory. Four compact buffers [MT][GLU_PITCH] per CTA: gate parts of CTA 0 and CTA 1, up
    // parts of CTA 1 and CTA 2. (Reading the parts through distributed shared memory instead took 4.4 us.)
    constexpr int CP = 48;                                    // floats per staged row (44 columns at most)
    static_assert(4 * MT * CP * 4 <= Cfg::RING_BYTES, "four compact buffers must fit the ring");
    if (warp >= 2 && n_units > 0) {
      const int q = warp & 3, w = q * 32 + lane;
      const int own = w < 44 ? 0 : (w < 84 ? 1 : 2);
      const int col = w - (own == 0 ? 0 : (own == 1 ? 44 : 84));
      const uint32_t dst0 = dsmem_addr(smem_u32(staging), (uint32_t)own);
      tc_fence_after();
      for (int s2 = 0; s2 < nseg; ++s2) {
        const int slot = seg[s2].mat == 0 ? rank : rank + 1;
        const uint32_t taddr = tmem_base + ((uint32_t)(q * 32) << 16) + (uint32_t)(s2 * MT);
        const uint32_t dst = dst0 + (uint32_t)((slot * MT * CP + col) * 4);
        if (MT >= 32) {
#pragma unroll
          for (int g = 0; g < MT / 32; ++g) {
            uint32_t r[32];
            tmem_ld32(taddr + g * 32, r);
            tmem_ld_wait();
#pragma unroll
            for (int j = 0; j < 32; ++j) dsmem_st(dst + (uint32_t)((g * 32 + j) * CP * 4), __uint_as_float(r[j]));
          }
        } else {
          uint32_t r[16];
          tmem_ld16(taddr, r);
          tmem_ld_wait();
#pragma unroll
          for (int j = 0; j < 16; ++j) dsmem_st(dst + (uint32_t)(j * CP * 4), __uint_as_float(r[j]));
        }
      }
      tc_fence_before();
    }
    __syncwarp();
    cluster_sync_all();                                       // the parts have arrived (release / acquire)
    if (warp >= 2 && n_units > 0) {
      const int e = threadIdx.x - 64;
      const int lo = rank == 0 ? 0 : (rank == 1 ? 44 : 84), hi = rank == 0 ? 44 : (rank == 1 ? 84 : 128);
      const int gpr = (hi - lo) >> 2;                        // groups of four columns per row: 11, 10, 11
      constexpr int PER = (MT * 11 + 127) / 128;
      const float* b0 = staging;
#pragma unroll
      for (int k = 0; k < PER; ++k) {
        const int it = e + 128 * k, m = it / gpr, w4 = it % gpr;
        const int col = t * 128 + lo + 4 * w4;
        if (m < MT && m < p.M && col < p.N) {
          const float* src = b0 + m * CP + 4 * w4;
          float4 ga = *reinterpret_cast<const float4*>(src), ua = *reinterpret_cast<const float4*>(src + 2 * MT * CP);
          add4(ga, *reinterpret_cast<const float4*>(src + MT * CP));
          add4(ua, *reinterpret_cast<const float4*>(src + 3 * MT * CP));
          uint2 o;
          o.x = pack_bf16x2(silu_f(ga.x) * ua.x, silu_f(ga.y) * ua.y);
          o.y = pack_bf16x2(silu_f(ga.z) * ua.z, silu_f(ga.w) * ua.w);
          *reinterpret_cast<uint2*>(p.act + (size_t)m * p.N + col) = o;
        }
      }
    }
    // nobody writes to or reads from another CTA's shared memory after the second barrier: no third one
    tc_fence_before();
    __syncthreads();
    if (warp == 1) tmem_dealloc(tmem_base, TMEM_COLS);
    return;
  }

  if (warp >= 2 && n_units > 0) {
    // Every finishing thread issues all its loads (distributed shared memory, residual stream) before it
    // uses the first one: the step costs about one round trip, not one per item.
    const int e = threadIdx.x - 64;                        // 0..127
    const uint32_t stage_local = smem_u32(staging);
    if (MODE == GC_ROPE) {
      // the tile holds 128 / D whole heads. CTA `rank` takes the activation rows rank, rank + cluster size, ...; an item is
      // (row, group of four rotation pairs): columns [lo, lo + 4) and [lo + D/2, lo + D/2 + 4) of one head
      constexpr int ITEMS = R_ITEMS, PER = R_PER;
      const int half = p.g.head_dim >> 1;
      bool (&on)[R_PER] = r_on;
      int (&mrow)[R_PER] = r_mrow, (&lo_c)[R_PER] = r_lo_c;
      float4 (&cs01)[R_PER] = r_cs01, (&cs23)[R_PER] = r_cs23;
      bf16* (&dst)[R_PER] = r_dst;
      uint32_t sb[CS];
#pragma unroll
      for (int r = 0; r < CS; ++r) sb[r] = dsmem_addr(stage_local, (uint32_t)r);
      float4 a[PER], c[PER];
#pragma unroll
      for (int k = 0; k < PER; ++k) {
        const int lo = lo_c[k] & 0xffff;
        const uint32_t o_lo = (uint32_t)((mrow[k] * Cfg::PITCH + lo) * 4), o_hi = o_lo + (uint32_t)(half * 4);
        const bool ld = (e + 128 * k) < ITEMS && mrow[k] < MT;
        a[k] = ld ? dsmem_ld4(sb[0] + o_lo) : make_float4(0.f, 0.f, 0.f, 0.f);
        c[k] = ld ? dsmem_ld4(sb[0] + o_hi) : make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
        for (int r = 1; r < CS; ++r)
          if (ld) { add4(a[k], dsmem_ld4(sb[r] + o_lo)); add4(c[k], dsmem_ld4(sb[r] + o_hi)); }
      }
#pragma unroll
      for (int k = 0; k < PER; ++k) {
        if (!on[k]) continue;
        const float4 t01 = cs01[k], t23 = cs23[k];
        uint2 lo_o, hi_o;
        if (rope_mat < 2) {
          lo_o.x = pack_bf16x2(a[k].x * t01.x - c[k].x * t01.y, a[k].y * t01.z - c[k].y * t01.w);
          lo_o.y = pack_bf16x2(a[k].z * t23.x - c[k].z * t23.y, a[k].w * t23.z - c[k].w * t23.w);
          hi_o.x = pack_bf16x2(c[k].x * t01.x + a[k].x * t01.y, c[k].y * t01.z + a[k].y * t01.w);
          hi_o.y = pack_bf16x2(c[k].z * t23.x + a[k].z * t23.y, c[k].w * t23.z + a[k].w * t23.w);
        } else {
          lo_o.x = pack_bf16x2(a[k].x, a[k].y); lo_o.y = pack_bf16x2(a[k].z, a[k].w);
          hi_o.x = pack_bf16x2(c[k].x, c[k].y); hi_o.y = pack_bf16x2(c[k].z, c[k].w);
        }
        const int up = rope_mat == 0 ? half : (lo_c[k] >> 16);
        *reinterpret_cast<uint2*>(dst[k]) = lo_o;
        *reinterpret_cast<uint2*>(dst[k] + up) = hi_o;
      }
    }
  }

  // nobody leaves (and gives up its shared memory) before every CTA of the cluster has read it
  __syncwarp();
  cluster_sync_all();
  tc_fence_before();
  __syncthreads();
  if (warp == 1) tmem_dealloc(tmem_base, TMEM_COLS);
}

}  // namespace spec
