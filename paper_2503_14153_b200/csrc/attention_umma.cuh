// Tree-masked attention on the 5th-generation tensor cores (tcgen05, accumulators in tensor memory) for
// passes of up to 64 query rows per CTA over long contexts, and for batched passes.
//
// A CTA owns one head, up to 64 query rows (a "row half": a 128-row pass takes two CTAs per head) and one
// split of the keys, and walks its keys in tiles of 128. A warp can read only the 32 tensor-memory lanes of
// its own SM quarter, and lane = MMA row, so to put all four quarters to work the 64 query rows are given
// twice to the 128-row MMA: rows 0..63 ("low stream") take care of keys 0..63 of every tile, rows 64..127
// (the same queries again, "high stream") of keys 64..127.
//   S = Q K^T      A = Q (twice), B = the tile's K slabs exactly as the cache holds them (K-major, 128-byte
//                  swizzle): both streams get the row's 128 scores, each thread reads its 64;
//   P = exp2(scale * S - ref) under the tree mask, rounded to bf16 into shared memory as a block-diagonal
//       operand: row r < 64 fills keys 0..63 and leaves 64..127 zero, row r + 64 the other way round;
//   O += P V       A = P, B = the tile's V slabs as the cache holds them (MN-major), accumulating in tensor
//                  memory: rows 0..63 collect the low keys' contribution, rows 64..127 the high keys'.
// `ref` is a stream's running reference: it is raised (and the stream's O row and sum rescaled, O by a
// load / multiply / store of its tensor-memory row) only when a tile's maximum exceeds it by more than 2^8,
// which after the first tile almost never happens. Two groups of four warps take alternate tiles, each with
// its own score buffer and O accumulator (4 x 128 = all 512 tensor-memory columns): while one group
// exponentiates, the tensor cores work for the other. A producer warp brings a tile's four 16 KB slabs
// (K / V x dims 0..63 / 64..127) with four 5-dimensional TMA loads straight out of the page pool -- the
// library places page p of sequence b at pool page p * max_batch + b and keeps the pages of a (layer, head)
// side by side, so a sequence's pages are a strided dimension of the tensor map --; one thread issues all
// MMAs. The four streams of a row (two groups x two key halves) are merged through shared memory. The key
// splits of a (sequence, row half, head) form one thread-block cluster, split s owning tiles s, s + cluster
// size, ... (which tiles does not depend on the length, so the first two can be asked for before the
// dependency wait when they lie below the host's lower bound of the committed length): each CTA leaves its
// merged partial in its own shared memory, and after a cluster barrier every CTA finishes a share of the
// rows, reading all the partials through distributed shared memory -- no partial sums in HBM, no arrival
// counter. Every mbarrier wait is bounded; a CTA whose wait ran out still joins the cluster barriers, so its
// peers do not wait for it.
#pragma once
#include <cuda.h>

#include "attention_tc.cuh"
#include "common.cuh"
#include "gemm_cluster.cuh"

namespace spec {

constexpr int AU_KT = 128;        // keys per tile
constexpr int AU_ROWS = 64;       // query rows per CTA
constexpr int AU_THREADS = 320;   // warps 0..3: softmax group 0; warps 4..7: group 1; warp 8: producer; warp 9: MMA
constexpr float AU_RESCALE_LOG2 = 8.f;   // a stream's reference is raised when a tile's maximum exceeds it by more than this
constexpr int AU_MAX_CLUSTER = 8; // most key splits (portable cluster size)
constexpr int AU_EXP = 132;       // floats per staged output row: head_dim + 4 (16-byte aligned rows, banks shifted by 4)

__host__ __device__ inline size_t attention_umma_smem() {
  return 1024 /*alignment*/ + 32768 /*Q, twice*/ + 2 * 32768 /*P*/ + 2 * 65536 /*K/V stages*/ + 256 /*barriers*/;
}

__device__ __forceinline__ void tma_load_5d(void* smem_dst, const void* tmap, int c0, int c1, int c2, int c3, int c4, uint64_t* bar) {
  asm volatile(
      "cp.async.bulk.tensor.5d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5, %6, %7}], [%2];"
      ::"r"(smem_u32(smem_dst)), "l"(tmap), "r"(smem_u32(bar)), "r"(c0), "r"(c1), "r"(c2), "r"(c3), "r"(c4)
      : "memory");
}
// 128-byte-swizzle descriptor with explicit leading / stride byte offsets (MN-major operands use both).
__device__ __forceinline__ uint64_t make_sw128_desc(uint32_t smem_addr, uint32_t lbo, uint32_t sbo) {
  uint64_t d = 0;
  d |= (uint64_t)((smem_addr & 0x3FFFFu) >> 4);
  d |= (uint64_t)(lbo >> 4) << 16;
  d |= (uint64_t)(sbo >> 4) << 32;
  d |= (uint64_t)1 << 46;
  d |= (uint64_t)2 << 61;
  return d;
}
__device__ __forceinline__ void tmem_st32(uint32_t taddr, const uint32_t (&r)[32]) {
  asm volatile(
      "tcgen05.st.sync.aligned.32x32b.x32.b32 [%0], "
      "{%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,%16,%17,%18,%19,%20,%21,%22,%23,%24,%25,%26,%27,%28,%29,%30,%31,%32};"
      ::"r"(taddr), "r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]), "r"(r[7]), "r"(r[8]), "r"(r[9]), "r"(r[10]),
        "r"(r[11]), "r"(r[12]), "r"(r[13]), "r"(r[14]), "r"(r[15]), "r"(r[16]), "r"(r[17]), "r"(r[18]), "r"(r[19]), "r"(r[20]), "r"(r[21]),
        "r"(r[22]), "r"(r[23]), "r"(r[24]), "r"(r[25]), "r"(r[26]), "r"(r[27]), "r"(r[28]), "r"(r[29]), "r"(r[30]), "r"(r[31])
      : "memory");
}
__device__ __forceinline__ void tmem_st_wait() { asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory"); }
__device__ __forceinline__ float2 dsmem_ld2(uint32_t addr) {
  float2 v;
  asm volatile("ld.shared::cluster.v2.f32 {%0, %1}, [%2];" : "=f"(v.x), "=f"(v.y) : "r"(addr) : "memory");
  return v;
}
__device__ __forceinline__ void fence_proxy_async_smem() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }

template <int HD>
__global__ void __launch_bounds__(AU_THREADS, 1)
attention_umma(const __grid_constant__ CUtensorMap tm_kv, const AttnTcArgs a, unsigned long long* tr) {
  static_assert(HD == 128, "two 64-dim slabs per row");
  KTrace kt(tr);
  extern __shared__ uint8_t smem_raw[];
  const uint32_t raw = smem_u32(smem_raw);
  uint8_t* sm = smem_raw + (((raw + 1023u) & ~1023u) - raw);
  uint8_t* q_s = sm;                          // 2 slabs x [128 rows][128 B] (rows 64.. repeat rows 0..63)
  uint8_t* p_s = sm + 32768;                  // [2 buffers] x 2 slabs x [128 rows][128 B]; slab h = keys [64 h, +64) of the tile
  uint8_t* kv_s = sm + 32768 + 65536;         // [2 stages] x (K slab 0, K slab 1, V slab 0, V slab 1) x [128 keys][128 B]
  uint64_t* bars = reinterpret_cast<uint64_t*>(kv_s + 2 * 65536);
  uint64_t* k_full = bars;                    // [2] K slabs of a stage have landed
  uint64_t* k_empty = bars + 2;               // [2] ... have been read by the tile's score MMAs
  uint64_t* v_full = bars + 4;                // [2]
  uint64_t* v_empty = bars + 6;               // [2] ... by the tile's P V MMAs
  uint64_t* s_full = bars + 8;                // [2] scores of a tile are in tensor memory
  uint64_t* p_full = bars + 10;               // [2] P operand written (the group's four warps)
  uint64_t* o_done = bars + 12;               // [2] P V of a tile has been added to the group's accumulator
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + 14);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int halves = gridDim.z / a.rows.B;
  // CTAs are handed out in grid order: with more CTAs than SMs the longest sequences go first, so that the
  // launch does not end on a long sequence started last (the host sorts by its bounds of the lengths)
  const int zb = blockIdx.z / halves;
  const int h = blockIdx.x, sp = blockIdx.y, b = a.rows.B <= ATTN_MAX_SEQS ? (int)a.order[zb] : zb, half = blockIdx.z % halves;
  const int row0 = half * AU_ROWS;
  const int H = a.H, kvh = h / (H / a.g.n_kv_heads);
  const int ncl = (int)gridDim.y;                              // key splits = the cluster; split sp owns tiles sp, sp + ncl, ...
  // ---- producer's loads: two K slabs and two V slabs per tile, K one tile ahead of V (K is released by the
  // score MMAs, long before the tile's V is released by the P V MMAs) ----
  const int lh = a.layer * a.g.n_kv_heads + kvh;             // slab rows of a page's pair: K dims 0..63, K 64..127, V, V
  auto load_k = [&](int t) -> bool {
    const int st = t & 1;
    if (t >= 2 && !mbar_wait(&k_empty[st], ((t >> 1) - 1) & 1, a.status, 50)) return false;
    uint8_t* dst = kv_s + st * 65536;
    mbar_expect_tx(&k_full[st], 32768);
    const int page0 = (sp + t * ncl) * (AU_KT / 16);
    tma_load_5d(dst, &tm_kv, 0, 0, b, page0, lh, &k_full[st]);
    tma_load_5d(dst + 16384, &tm_kv, 0, 16, b, page0, lh, &k_full[st]);
    return true;
  };
  auto load_v = [&](int t) -> bool {
    const int st = t & 1;
    if (t >= 2 && !mbar_wait(&v_empty[st], ((t >> 1) - 1) & 1, a.status, 56)) return false;
    uint8_t* dst = kv_s + st * 65536 + 32768;
    mbar_expect_tx(&v_full[st], 32768);
    const int page0 = (sp + t * ncl) * (AU_KT / 16);
    tma_load_5d(dst, &tm_kv, 0, 32, b, page0, lh, &v_full[st]);
    tma_load_5d(dst + 16384, &tm_kv, 0, 48, b, page0, lh, &v_full[st]);
    return true;
  };
  // The producer thread sets up the barriers itself and at once asks for its first two tiles where they lie
  // wholly below the host's lower bound of the committed length: those keys were written by earlier steps (no
  // kernel of this step starts before the kernels of the step before it have completed), so the loads need not
  // wait for the kernel before this one, and which tiles a split owns does not depend on the length.
  int pre = 0;                                                 // tiles whose loads went out before the dependency wait
  if (threadIdx.x == 8 * 32) {
    for (int i = 0; i < 14; ++i) mbar_init(&bars[i], (i == 10 || i == 11) ? 4 : 1);
    mbar_fence_init();
    const int n_lo = b < ATTN_MAX_SEQS ? a.n_lo[b] : 0;
    if ((sp + 1) * AU_KT <= n_lo) {
      load_k(0);
      pre = 1;
      if ((sp + ncl + 1) * AU_KT <= n_lo) { load_k(1); pre = 2; }
      load_v(0);
    }
  }
  if (warp == 9) { tmem_alloc(tmem_slot, 512); tmem_relinquish(); }
  // the P operands' off-diagonal blocks stay zero for the whole kernel
  for (int c = threadIdx.x; c < 65536 / 16; c += AU_THREADS) reinterpret_cast<uint4*>(p_s)[c] = make_uint4(0, 0, 0, 0);
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = *tmem_slot;
  // Dependents may start only now: this CTA holds all of the SM's tensor memory, and a dependent kernel's CTA
  // that took some first would wait for this grid while this CTA waited for its columns.
  pdl_launch_dependents();
  pdl_wait();
  if (threadIdx.x == 0) trace_mark_min(tr, 2);
  const int R = a.rows.R, cnt = a.rows.cnt[b], n = a.rows.n[b];
  const int S = n + cnt;
  const int total_tiles = (S + AU_KT - 1) / AU_KT;
  const int nt = sp < total_tiles ? (total_tiles - sp + ncl - 1) / ncl : 0;   // (pre <= nt: the tiles asked for lie below n)
  const bool active = row0 < cnt && nt > 0;
  if (active) {
    if (warp == 8) {
      // the first tiles are on their way while the other warps stage Q
      if (lane == 0) {
        if (pre < 1) load_k(0);
        if (pre < 2 && nt > 1) load_k(1);
        if (pre < 1) load_v(0);
      }
    } else if (warp < 8) {
      // Q rows of this CTA into the two K-major slabs, each row at r and at r + 64 (rows beyond cnt are zeros);
      // a thread fetches its four pieces before it stores the first
      uint4 v[4];
#pragma unroll
      for (int k = 0; k < 4; ++k) {
        const int c = threadIdx.x + 256 * k, qr = c / (HD / 8), ch = c % (HD / 8);
        v[k] = make_uint4(0, 0, 0, 0);
        if (row0 + qr < cnt) v[k] = *reinterpret_cast<const uint4*>(a.q + (size_t)(b * R + row0 + qr) * H * HD + h * HD + ch * 8);
      }
#pragma unroll
      for (int k = 0; k < 4; ++k) {
        const int c = threadIdx.x + 256 * k, qr = c / (HD / 8), ch = c % (HD / 8);
        uint8_t* dst = q_s + (ch >> 3) * 16384 + qr * 128 + (((ch & 7) ^ (qr & 7)) << 4);   // (qr + 64) & 7 == qr & 7
        *reinterpret_cast<uint4*>(dst) = v[k];
        *reinterpret_cast<uint4*>(dst + AU_ROWS * 128) = v[k];
      }
    }
  } else if (pre > 0 && threadIdx.x == 8 * 32) {
    // rows beyond the pass's count: nothing to do, but the loads asked for above must have landed before the
    // CTA gives up its shared memory
    mbar_wait(&k_full[0], 0, a.status, 59);
    mbar_wait(&v_full[0], 0, a.status, 59);
    if (pre > 1) mbar_wait(&k_full[1], 0, a.status, 59);
  }
  fence_proxy_async_smem();
  __syncthreads();

  const int grp = warp >> 2;                                   // softmax group of warps 0..3 / 4..7
  const int q4 = warp & 3;                                     // SM quarter = tensor-memory lanes [32 q4, +32)
  const int mrow = q4 * 32 + lane;                             // this thread's MMA row (tensor-memory lane)
  const int qrow = mrow & (AU_ROWS - 1), kh = mrow >> 6;       // its query row within the CTA and key half of every tile
  float m_ref = -INFINITY, l_run = 0.f;
  int my_tiles = 0;
  bool ok = true;

  if (active) {
    if (warp == 8) {
      if (lane == 0) {
        for (int t = 1; t < nt && ok; ++t) {
          if (t + 1 < nt && !load_k(t + 1)) { ok = false; break; }
          if (!load_v(t)) { ok = false; break; }
        }
      }
    } else if (warp == 9) {
      if (lane == 0) {
        // ---- MMA issuer. Order S(0), S(1), then PV(t), S(t + 2) for t = 0, 1, ...: the scores of the next two tiles are
        // always out before a group's probabilities are awaited, and no MMA waits behind a load it does not need ----
        const uint32_t idesc_s = make_idesc_bf16(128, AU_KT);                  // A and B K-major
        const uint32_t idesc_o = make_idesc_bf16(128, HD) | (1u << 16);        // B (V) MN-major
        const uint32_t q_addr = smem_u32(q_s);
        auto mma_s = [&](int t) -> bool {
          const int bf = t & 1, st = t & 1;
          if (!mbar_wait(&k_full[st], (t >> 1) & 1, a.status, 51)) return false;
          tc_fence_after();
          const uint32_t d_addr = tmem + (uint32_t)(bf * 128);
          const uint32_t k_addr = smem_u32(kv_s + st * 65536);
#pragma unroll
          for (int j = 0; j < HD / 16; ++j) {                                 // k-steps of 16 dims
            const uint64_t ad = make_kmajor_sw128_desc(q_addr + (j >> 2) * 16384) + 2 * (j & 3);
            const uint64_t bd = make_kmajor_sw128_desc(k_addr + (j >> 2) * 16384) + 2 * (j & 3);
            tc_mma_f16(d_addr, ad, bd, idesc_s, j > 0 ? 1u : 0u);
          }
          tc_commit(&s_full[bf]);
          tc_commit(&k_empty[st]);
          return true;
        };
        auto mma_pv = [&](int u) -> bool {
          const int bf = u & 1, st = u & 1;
          if (!mbar_wait(&p_full[bf], (u >> 1) & 1, a.status, 52)) return false;
          if (!mbar_wait(&v_full[st], (u >> 1) & 1, a.status, 57)) return false;
          tc_fence_after();
          const uint32_t d_addr = tmem + 256u + (uint32_t)(bf * 128);            // the group's accumulator
          const uint32_t p_addr = smem_u32(p_s + bf * 32768), v_addr = smem_u32(kv_s + st * 65536 + 32768);
#pragma unroll
          for (int j = 0; j < AU_KT / 16; ++j) {                              // k-steps of 16 keys
            const uint64_t ad = make_kmajor_sw128_desc(p_addr + (j >> 2) * 16384) + 2 * (j & 3);
            const uint64_t bd = make_sw128_desc(v_addr + j * 2048, 16384, 1024);
            tc_mma_f16(d_addr, ad, bd, idesc_o, (u >= 2 || j > 0) ? 1u : 0u);   // a group's first tile starts its accumulator
          }
          tc_commit(&o_done[bf]);
          tc_commit(&v_empty[st]);
          return true;
        };
        ok = mma_s(0);
        if (ok && nt > 1) ok = mma_s(1);
        if (ok) trace_mark_max(tr, 3);
        for (int t = 0; t < nt && ok; ++t) {
          if (!mma_pv(t)) { ok = false; break; }
          if (t + 2 < nt && !mma_s(t + 2)) { ok = false; break; }
        }
      }
    } else {
      // ---- softmax groups: tiles grp, grp + 2, ...; a thread = one query row x one half of every tile's keys ----
      const int i_row = row0 + qrow;
      uint32_t anc[4];
#pragma unroll
      for (int w = 0; w < 4; ++w) anc[w] = i_row < cnt ? a.rows.anc[i_row * 4 + w] : 0u;
      const uint32_t lane_base = (uint32_t)(q4 * 32) << 16;
      for (int t = grp; t < nt; t += 2) {
        const int bf = t & 1;
        if (!mbar_wait(&s_full[bf], (t >> 1) & 1, a.status, 54)) { ok = false; break; }
        tc_fence_after();
        const uint32_t s_addr = tmem + lane_base + (uint32_t)(bf * 128 + kh * 64);
        const int k0 = (sp + t * ncl) * AU_KT + kh * 64;       // first key of this thread's half
        uint32_t r0[32], r1[32];
        tmem_ld32(s_addr, r0);
        tmem_ld32(s_addr + 32, r1);
        uint32_t vis0 = 0xffffffffu, vis1 = 0xffffffffu;
        if (k0 + 64 > n) {                                      // the half reaches into the tree rows or past the end
          const unsigned long long v = attn_vis64(anc, k0, n);
          vis0 = (uint32_t)v; vis1 = (uint32_t)(v >> 32);
        }
        tmem_ld_wait();
        float tmax = -INFINITY;
        if ((vis0 & vis1) == 0xffffffffu) {
#pragma unroll
          for (int j = 0; j < 32; ++j) tmax = fmaxf(tmax, fmaxf(__uint_as_float(r0[j]), __uint_as_float(r1[j])));
        } else {
#pragma unroll
          for (int j = 0; j < 32; ++j) {
            if ((vis0 >> j) & 1u) tmax = fmaxf(tmax, __uint_as_float(r0[j]));
            if ((vis1 >> j) & 1u) tmax = fmaxf(tmax, __uint_as_float(r1[j]));
          }
        }
        tmax *= a.scale_log2;
        // raise the reference only when it is too low by more than 2^AU_RESCALE_LOG2 (or not set yet)
        const bool raise = tmax > m_ref + AU_RESCALE_LOG2 || (m_ref == -INFINITY && tmax > -INFINITY);
        const float m_new = raise ? tmax : m_ref;
        const float alpha = raise ? exp2f(m_ref - m_new) : 1.f;   // 0 the first time
        // the group's previous tile must be through the tensor cores: its P operand and accumulator are reused
        if (t >= 2 && !mbar_wait(&o_done[bf], ((t >> 1) - 1) & 1, a.status, 55)) { ok = false; break; }
        if (__any_sync(0xffffffffu, raise && my_tiles > 0)) {
          // rescale this lane's accumulator row (other lanes of the warp multiply by one)
          tc_fence_after();
          const uint32_t o_addr = tmem + lane_base + 256u + (uint32_t)(bf * 128);
#pragma unroll 1
          for (int c = 0; c < 4; ++c) {
            uint32_t r[32];
            tmem_ld32(o_addr + c * 32, r);
            tmem_ld_wait();
#pragma unroll
            for (int j = 0; j < 32; ++j) r[j] = __float_as_uint(__uint_as_float(r[j]) * alpha);
            tmem_st32(o_addr + c * 32, r);
          }
          tmem_st_wait();
        }
        l_run *= alpha;
        m_ref = m_new;
        const float base = (m_new == -INFINITY) ? 0.f : m_new;
        // probabilities of this thread's 64 keys, rounded to bf16, into row `mrow` of slab `kh` of the P operand
        float l0 = 0.f, l1 = 0.f;
        uint8_t* p_row = p_s + bf * 32768 + kh * 16384 + mrow * 128;
#pragma unroll
        for (int c = 0; c < 2; ++c) {
          const uint32_t (&r)[32] = c ? r1 : r0;
          const uint32_t vc = c ? vis1 : vis0;
          uint32_t pk[16];
#pragma unroll
          for (int j = 0; j < 32; j += 2) {
            float p0 = exp2f(fmaf(__uint_as_float(r[j]), a.scale_log2, -base));
            float p1 = exp2f(fmaf(__uint_as_float(r[j + 1]), a.scale_log2, -base));
            if (!((vc >> j) & 1u)) p0 = 0.f;
            if (!((vc >> (j + 1)) & 1u)) p1 = 0.f;
            l0 += p0; l1 += p1;
            pk[j >> 1] = pack_bf16(p0, p1);
          }
#pragma unroll
          for (int g = 0; g < 4; ++g) {
            const int ch = c * 4 + g;
            *reinterpret_cast<uint4*>(p_row + ((ch ^ (mrow & 7)) << 4)) = make_uint4(pk[4 * g], pk[4 * g + 1], pk[4 * g + 2], pk[4 * g + 3]);
          }
        }
        l_run += l0 + l1;
        ++my_tiles;
        fence_proxy_async_smem();
        tc_fence_before();
        __syncwarp();
        if (lane == 0) mbar_arrive(&p_full[bf]);
      }
      // the group's last tile must be through the tensor cores before its accumulator is read
      if (ok && my_tiles > 0) {
        const int t_last = grp + 2 * (my_tiles - 1);
        if (!mbar_wait(&o_done[t_last & 1], (t_last >> 1) & 1, a.status, 58)) ok = false;
      }
    }
  }
  ok = __syncthreads_and(ok);
  if (row0 >= cnt) {                                           // the same for every CTA of the cluster
    if (warp == 9) { tc_fence_after(); tmem_dealloc(tmem, 512); }
    return;
  }
  // ---- the four streams of a query row (two groups x two key halves), staged in shared memory ----
  float* ex = reinterpret_cast<float*>(sm);                    // [4 streams][64 rows][AU_EXP]; stream 0 becomes the CTA's partial
  float* ml = ex + 4 * AU_ROWS * AU_EXP;                       // [4 streams][64 rows] (reference, sum)
  float* cml = ml + 4 * AU_ROWS * 2;                           // [64 rows] of the CTA's partial
  const bool work = active && ok;
  if (warp < 8) {
    const int sid = grp * 2 + kh;
    float* my = ex + ((size_t)sid * AU_ROWS + qrow) * AU_EXP;
    tc_fence_after();
    if (work && my_tiles > 0) {
      const uint32_t o_addr = tmem + ((uint32_t)(q4 * 32) << 16) + 256u + (uint32_t)(grp * 128);
#pragma unroll 1
      for (int c = 0; c < 4; ++c) {
        uint32_t r[32];
        tmem_ld32(o_addr + c * 32, r);
        tmem_ld_wait();
#pragma unroll
        for (int j = 0; j < 32; j += 4)
          *reinterpret_cast<float4*>(my + c * 32 + j) =
              make_float4(__uint_as_float(r[j]), __uint_as_float(r[j + 1]), __uint_as_float(r[j + 2]), __uint_as_float(r[j + 3]));
      }
    } else {
#pragma unroll 4
      for (int j = 0; j < HD; j += 4) *reinterpret_cast<float4*>(my + j) = make_float4(0.f, 0.f, 0.f, 0.f);
    }
    *reinterpret_cast<float2*>(ml + ((size_t)sid * AU_ROWS + qrow) * 2) = work ? make_float2(m_ref, l_run) : make_float2(-INFINITY, 0.f);
    tc_fence_before();
  }
  __syncthreads();
  if (warp == 9) { tc_fence_after(); tmem_dealloc(tmem, 512); }
  if (warp < 8) {
    // thread = (row, every fourth 4-dim chunk): merge the four streams
    const int row = threadIdx.x >> 2, qd = threadIdx.x & 3;
    float ms[4], ls[4], mm = -INFINITY;
#pragma unroll
    for (int s2 = 0; s2 < 4; ++s2) {
      const float2 v = *reinterpret_cast<const float2*>(ml + ((size_t)s2 * AU_ROWS + row) * 2);
      ms[s2] = v.x; ls[s2] = v.y;
      mm = fmaxf(mm, v.x);
    }
    const float base = (mm == -INFINITY) ? 0.f : mm;
    float L = 0.f;
#pragma unroll
    for (int s2 = 0; s2 < 4; ++s2) { ms[s2] = exp2f(ms[s2] - base); L += ms[s2] * ls[s2]; }
    const float inv = 1.f / L;
    const size_t m = (size_t)b * R + row0 + row;
    const bool valid = row0 + row < cnt;
#pragma unroll
    for (int j = 0; j < HD / 16; ++j) {
      const int d = (j * 4 + qd) * 4;
      float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
      for (int s2 = 0; s2 < 4; ++s2) {
        const float4 v = *reinterpret_cast<const float4*>(ex + ((size_t)s2 * AU_ROWS + row) * AU_EXP + d);
        acc.x += ms[s2] * v.x; acc.y += ms[s2] * v.y; acc.z += ms[s2] * v.z; acc.w += ms[s2] * v.w;
      }
      if (ncl == 1) {
        if (valid) *reinterpret_cast<uint2*>(a.out + m * H * HD + h * HD + d) =
            make_uint2(pack_bf16(acc.x * inv, acc.y * inv), pack_bf16(acc.z * inv, acc.w * inv));
      } else {
        *reinterpret_cast<float4*>(ex + (size_t)row * AU_EXP + d) = acc;      // in place: only this thread touches it
      }
    }
    if (ncl > 1 && qd == 0) *reinterpret_cast<float2*>(cml + row * 2) = make_float2(mm, L);
  }
  if (ncl == 1) return;
  // ---- the cluster's partials: CTA `rank` finishes rows [rank * rpc, +rpc) from everybody's shared memory ----
  __syncwarp();
  cluster_sync_all();
  {
    const int rank = (int)cluster_ctarank();
    const int rpc = (AU_ROWS + ncl - 1) / ncl;
    const uint32_t ex_local = smem_u32(ex), cml_local = smem_u32(cml);
    uint32_t ex_r[AU_MAX_CLUSTER], cml_r[AU_MAX_CLUSTER];
#pragma unroll
    for (int s2 = 0; s2 < AU_MAX_CLUSTER; ++s2) {
      ex_r[s2] = dsmem_addr(ex_local, (uint32_t)min(s2, ncl - 1));
      cml_r[s2] = dsmem_addr(cml_local, (uint32_t)min(s2, ncl - 1));
    }
    for (int it = threadIdx.x; it < rpc * (HD / 4); it += AU_THREADS) {
      const int row = rank * rpc + it / (HD / 4), d = (it % (HD / 4)) * 4;
      if (row >= AU_ROWS || row0 + row >= cnt) continue;
      float2 mlv[AU_MAX_CLUSTER];
      float4 ov[AU_MAX_CLUSTER];
#pragma unroll
      for (int s2 = 0; s2 < AU_MAX_CLUSTER; ++s2) {
        mlv[s2] = make_float2(-INFINITY, 0.f);
        ov[s2] = make_float4(0.f, 0.f, 0.f, 0.f);
        if (s2 < ncl) {
          mlv[s2] = dsmem_ld2(cml_r[s2] + (uint32_t)(row * 8));
          ov[s2] = dsmem_ld4(ex_r[s2] + (uint32_t)((row * AU_EXP + d) * 4));
        }
      }
      float mm = -INFINITY;
#pragma unroll
      for (int s2 = 0; s2 < AU_MAX_CLUSTER; ++s2) mm = fmaxf(mm, mlv[s2].x);
      float L = 0.f;
      float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
      for (int s2 = 0; s2 < AU_MAX_CLUSTER; ++s2) {
        const float w = exp2f(mlv[s2].x - mm);                 // a valid row sees itself: mm is finite
        L += w * mlv[s2].y;
        acc.x += w * ov[s2].x; acc.y += w * ov[s2].y; acc.z += w * ov[s2].z; acc.w += w * ov[s2].w;
      }
      const float inv = 1.f / L;
      const size_t m = (size_t)b * R + row0 + row;
      *reinterpret_cast<uint2*>(a.out + m * H * HD + h * HD + d) =
          make_uint2(pack_bf16(acc.x * inv, acc.y * inv), pack_bf16(acc.z * inv, acc.w * inv));
    }
  }
  // nobody leaves while a peer may still read its shared memory
  __syncwarp();
  cluster_sync_all();
}

}  // namespace spec
