// Tree-masked attention on the 5th-generation tensor cores (tcgen05, accumulators in tensor memory) for
// passes of up to 64 query rows per CTA over long contexts, and for batched passes.
//
// A CTA owns one head, up to 64 query rows (a "row half": a 128-row pass takes two CTAs per head) and one
// split of the keys, and walks its keys in tiles of 128:
//   S   = Q K^T    one MMA group per tile: A = Q (64 rows in a 128-row operand; rows 64.. are don't-care),
//                  B = the tile's K slabs exactly as the cache holds them (K-major, 128-byte swizzle);
//   P   = exp2(scale * S - max) under the tree mask, by the threads that own the rows (tensor-memory lane =
//         query row, so a row's 128 scores sit in one thread: no shuffles), rounded to bf16 into shared memory;
//   O_t = P V      A = P (K-major), B = the tile's V slabs as the cache holds them (MN-major);
//   O   = O * alpha + O_t in the registers of the row's thread (online softmax).
// Two groups of two warps take alternate tiles, each with its own score and O_t accumulators (4 x 128 = all
// 512 tensor-memory columns) and its own running (max, sum, O): while one group exponentiates, the tensor
// cores work for the other. A producer warp brings a tile's four 16 KB slabs (K / V x dims 0..63 / 64..127)
// with four 5-dimensional TMA loads straight out of the page pool -- the library places page p of sequence b
// at pool page p * max_batch + b, so a sequence's pages are a strided dimension of the tensor map --; one
// thread issues all MMAs. The two groups' states are merged through shared memory, the key splits by the
// CTA that arrives last. Every wait is bounded.
#pragma once
#include <cuda.h>

#include "attention_tc.cuh"
#include "common.cuh"

namespace spec {

constexpr int AU_KT = 128;        // keys per tile
constexpr int AU_ROWS = 64;       // query rows per CTA
constexpr int AU_THREADS = 192;   // warps 0,1: softmax group 0; warp 2: producer; warp 3: MMA; warps 4,5: softmax group 1
constexpr int AU_SPLIT_TILES = 4; // fewest tiles worth a key split of their own

__host__ __device__ inline size_t attention_umma_smem() {
  return 1024 /*alignment*/ + 16384 /*Q*/ + 2 * 16384 /*P*/ + 2 * 65536 /*K/V stages*/ + 256 /*barriers*/;
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
__device__ __forceinline__ void fence_proxy_async_smem() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }

template <int HD>
__global__ void __launch_bounds__(AU_THREADS, 1)
attention_umma(const __grid_constant__ CUtensorMap tm_kv, const AttnTcArgs a, unsigned long long* tr) {
  static_assert(HD == 128, "two 64-dim slabs per row");
  KTrace kt(tr);
  extern __shared__ uint8_t smem_raw[];
  const uint32_t raw = smem_u32(smem_raw);
  uint8_t* sm = smem_raw + (((raw + 1023u) & ~1023u) - raw);
  uint8_t* q_s = sm;                          // 2 slabs x [64 rows][128 B]
  uint8_t* p_s = sm + 16384;                  // [2 buffers] x 2 slabs x [64 rows][128 B]
  uint8_t* kv_s = sm + 16384 + 32768;         // [2 stages] x (K slab 0, K slab 1, V slab 0, V slab 1) x [128 keys][128 B]
  uint64_t* bars = reinterpret_cast<uint64_t*>(kv_s + 2 * 65536);
  uint64_t* k_full = bars;                    // [2] K slabs of a stage have landed
  uint64_t* k_empty = bars + 2;               // [2] ... have been read by the tile's score MMAs
  uint64_t* v_full = bars + 4;                // [2]
  uint64_t* v_empty = bars + 6;               // [2] ... by the tile's P V MMAs
  uint64_t* s_full = bars + 8;                // [2] scores of a tile are in tensor memory
  uint64_t* p_full = bars + 10;               // [2] P operand written (the group's two warps)
  uint64_t* o_full = bars + 12;               // [2] P V of a tile is in tensor memory
  uint64_t* o_empty = bars + 14;              // [2] ... has been read (the group's two warps)
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + 16);
  __shared__ int last_s;

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int halves = gridDim.z / a.rows.B;
  const int h = blockIdx.x, sp = blockIdx.y, b = blockIdx.z / halves, half = blockIdx.z % halves;
  const int row0 = half * AU_ROWS;
  const int H = a.H, kvh = h / (H / a.g.n_kv_heads);
  if (threadIdx.x == 0) {
    for (int i = 0; i < 16; ++i) mbar_init(&bars[i], (i >= 10 && i < 12) || i >= 14 ? 2 : 1);
    mbar_fence_init();
    tma_prefetch_desc(&tm_kv);
  }
  if (warp == 3) { tmem_alloc(tmem_slot, 512); tmem_relinquish(); }
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
  const int S = n + cnt, M = a.rows.B * R;
  const int total_tiles = (S + AU_KT - 1) / AU_KT;
  const int nsplit = max(1, min(a.nsplit, (total_tiles + AU_SPLIT_TILES - 1) / AU_SPLIT_TILES));
  const int tps = (total_tiles + nsplit - 1) / nsplit;
  const int t0 = sp * tps, nt = min(total_tiles, t0 + tps) - t0;
  const bool active = row0 < cnt && sp < nsplit && nt > 0;
  // Q rows of this CTA into the two K-major slabs (rows beyond cnt are zeros)
  if (active) {
    for (int c = threadIdx.x; c < AU_ROWS * (HD / 8); c += AU_THREADS) {
      const int r = c / (HD / 8), ch = c % (HD / 8);
      uint4 v = make_uint4(0, 0, 0, 0);
      if (row0 + r < cnt) v = *reinterpret_cast<const uint4*>(a.q + (size_t)(b * R + row0 + r) * H * HD + h * HD + ch * 8);
      *reinterpret_cast<uint4*>(q_s + (ch >> 3) * 8192 + r * 128 + (((ch & 7) ^ (r & 7)) << 4)) = v;
    }
    fence_proxy_async_smem();
  }
  __syncthreads();

  const int grp = warp >> 2;                                   // softmax group of warps 0,1 / 4,5
  const int row = (warp & 1) * 32 + lane;                      // this thread's query row within the CTA (tensor-memory lane)
  float o_acc[HD];
  float m_run = -INFINITY, l_run = 0.f;
#pragma unroll
  for (int d = 0; d < HD; ++d) o_acc[d] = 0.f;
  bool ok = true;

  if (active) {
    if (warp == 2) {
      if (lane == 0) {
        // ---- producer: two K slabs and two V slabs per tile, K one tile ahead of V (K is released by the score
        // MMAs, long before the tile's V is released by the P V MMAs) ----
        const int blk_k = ((a.layer * a.g.n_kv_heads + kvh) * 2 + 0) * 2, blk_v = blk_k + 2;
        auto load_k = [&](int t) -> bool {
          const int st = t & 1;
          if (t >= 2 && !mbar_wait(&k_empty[st], ((t >> 1) - 1) & 1, a.status, 50)) return false;
          uint8_t* dst = kv_s + st * 65536;
          mbar_expect_tx(&k_full[st], 32768);
          const int page0 = (t0 + t) * (AU_KT / 16);
          tma_load_5d(dst, &tm_kv, 0, 0, blk_k, b, page0, &k_full[st]);
          tma_load_5d(dst + 16384, &tm_kv, 0, 0, blk_k + 1, b, page0, &k_full[st]);
          return true;
        };
        auto load_v = [&](int t) -> bool {
          const int st = t & 1;
          if (t >= 2 && !mbar_wait(&v_empty[st], ((t >> 1) - 1) & 1, a.status, 56)) return false;
          uint8_t* dst = kv_s + st * 65536 + 32768;
          mbar_expect_tx(&v_full[st], 32768);
          const int page0 = (t0 + t) * (AU_KT / 16);
          tma_load_5d(dst, &tm_kv, 0, 0, blk_v, b, page0, &v_full[st]);
          tma_load_5d(dst + 16384, &tm_kv, 0, 0, blk_v + 1, b, page0, &v_full[st]);
          return true;
        };
        ok = load_k(0);
        for (int t = 0; t < nt && ok; ++t) {
          if (t + 1 < nt && !load_k(t + 1)) { ok = false; break; }
          if (!load_v(t)) { ok = false; break; }
        }
      }
    } else if (warp == 3) {
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
            const uint64_t ad = make_kmajor_sw128_desc(q_addr + (j >> 2) * 8192) + 2 * (j & 3);
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
          if (u >= 2 && !mbar_wait(&o_empty[bf], ((u >> 1) - 1) & 1, a.status, 53)) return false;
          tc_fence_after();
          const uint32_t d_addr = tmem + 256u + (uint32_t)(bf * 128);
          const uint32_t p_addr = smem_u32(p_s + bf * 16384), v_addr = smem_u32(kv_s + st * 65536 + 32768);
#pragma unroll
          for (int j = 0; j < AU_KT / 16; ++j) {                              // k-steps of 16 keys
            const uint64_t ad = make_kmajor_sw128_desc(p_addr + (j >> 2) * 8192) + 2 * (j & 3);
            const uint64_t bd = make_sw128_desc(v_addr + j * 2048, 16384, 1024);
            tc_mma_f16(d_addr, ad, bd, idesc_o, j > 0 ? 1u : 0u);
          }
          tc_commit(&o_full[bf]);
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
      // ---- softmax groups: tiles grp, grp + 2, ... ----
      const int i_row = row0 + row;
      uint32_t anc[4];
#pragma unroll
      for (int w = 0; w < 4; ++w) anc[w] = i_row < cnt ? a.rows.anc[i_row * 4 + w] : 0u;
      const uint32_t lane_base = (uint32_t)((warp & 1) * 32) << 16;
      for (int t = grp; t < nt; t += 2) {
        const int bf = t & 1;
        if (!mbar_wait(&s_full[bf], (t >> 1) & 1, a.status, 54)) { ok = false; break; }
        tc_fence_after();
        const uint32_t s_addr = tmem + lane_base + (uint32_t)(bf * 128);
        const int k0 = (t0 + t) * AU_KT;
        const bool all_visible = k0 + AU_KT <= n;             // committed positions only (every tile but the last one or two)
        uint8_t* p_row = p_s + bf * 16384 + row * 128;
        float tmax = -INFINITY, l_tile = 0.f, m_new, base, alpha;
        if (all_visible) {
          // pass 1: the row's maximum
#pragma unroll 1
          for (int c = 0; c < 4; ++c) {
            uint32_t r[32];
            tmem_ld32(s_addr + c * 32, r);
            tmem_ld_wait();
#pragma unroll
            for (int j = 0; j < 32; ++j) tmax = fmaxf(tmax, __uint_as_float(r[j]));
          }
          tmax *= a.scale_log2;
          m_new = fmaxf(m_run, tmax);
          base = m_new;
          alpha = exp2f(m_run - base);
          // pass 2: probabilities, rounded to bf16 into the P operand (row `row`, 16-byte chunks swizzled with the row)
#pragma unroll 1
          for (int c = 0; c < 4; ++c) {
            uint32_t r[32];
            tmem_ld32(s_addr + c * 32, r);
            tmem_ld_wait();
            uint32_t pk[16];
#pragma unroll
            for (int j = 0; j < 32; j += 2) {
              const float p0 = exp2f(fmaf(__uint_as_float(r[j]), a.scale_log2, -base));
              const float p1 = exp2f(fmaf(__uint_as_float(r[j + 1]), a.scale_log2, -base));
              l_tile += p0 + p1;
              pk[j >> 1] = pack_bf16(p0, p1);
            }
#pragma unroll
            for (int q4 = 0; q4 < 4; ++q4) {
              const int ch = (c & 1) * 4 + q4;
              *reinterpret_cast<uint4*>(p_row + (c >> 1) * 8192 + ((ch ^ (row & 7)) << 4)) = make_uint4(pk[4 * q4], pk[4 * q4 + 1], pk[4 * q4 + 2], pk[4 * q4 + 3]);
            }
          }
        } else {
          // the tile reaches into the tree rows (or past the sequence's end): per-key visibility
          uint32_t vis[4];
#pragma unroll 1
          for (int c = 0; c < 4; ++c) {
            uint32_t r[32];
            tmem_ld32(s_addr + c * 32, r);
            vis[c] = (k0 + c * 32 + 32 <= n) ? 0xffffffffu : (uint32_t)attn_vis64(anc, k0 + c * 32, n);
            tmem_ld_wait();
#pragma unroll
            for (int j = 0; j < 32; ++j)
              if ((vis[c] >> j) & 1u) tmax = fmaxf(tmax, __uint_as_float(r[j]));
          }
          tmax *= a.scale_log2;
          m_new = fmaxf(m_run, tmax);
          base = (m_new == -INFINITY) ? 0.f : m_new;
          alpha = exp2f(m_run - base);
#pragma unroll 1
          for (int c = 0; c < 4; ++c) {
            uint32_t r[32];
            tmem_ld32(s_addr + c * 32, r);
            tmem_ld_wait();
            uint32_t pk[16];
            const uint32_t vc = vis[c];
#pragma unroll
            for (int j = 0; j < 32; j += 2) {
              const float p0 = ((vc >> j) & 1u) ? exp2f(fmaf(__uint_as_float(r[j]), a.scale_log2, -base)) : 0.f;
              const float p1 = ((vc >> (j + 1)) & 1u) ? exp2f(fmaf(__uint_as_float(r[j + 1]), a.scale_log2, -base)) : 0.f;
              l_tile += p0 + p1;
              pk[j >> 1] = pack_bf16(p0, p1);
            }
#pragma unroll
            for (int q4 = 0; q4 < 4; ++q4) {
              const int ch = (c & 1) * 4 + q4;
              *reinterpret_cast<uint4*>(p_row + (c >> 1) * 8192 + ((ch ^ (row & 7)) << 4)) = make_uint4(pk[4 * q4], pk[4 * q4 + 1], pk[4 * q4 + 2], pk[4 * q4 + 3]);
            }
          }
        }
        fence_proxy_async_smem();
        tc_fence_before();
        __syncwarp();
        if (lane == 0) mbar_arrive(&p_full[bf]);
        l_run = l_run * alpha + l_tile;
        m_run = m_new;
        // correction: O = O * alpha + P V of this tile
        if (!mbar_wait(&o_full[bf], (t >> 1) & 1, a.status, 55)) { ok = false; break; }
        tc_fence_after();
        const uint32_t o_addr = tmem + lane_base + 256u + (uint32_t)(bf * 128);
#pragma unroll
        for (int c = 0; c < 4; ++c) {
          uint32_t r[32];
          tmem_ld32(o_addr + c * 32, r);
          tmem_ld_wait();
#pragma unroll
          for (int j = 0; j < 32; ++j) o_acc[c * 32 + j] = o_acc[c * 32 + j] * alpha + __uint_as_float(r[j]);
        }
        tc_fence_before();
        __syncwarp();
        if (lane == 0) mbar_arrive(&o_empty[bf]);
      }
    }
  }
  // all tensor-core work of this CTA is complete or abandoned: merge the two groups through shared memory
  ok = __syncthreads_and(ok);
  if (warp == 3) {
    tc_fence_after();
    tmem_dealloc(tmem, 512);
  }
  if (!ok || !active) return;
  float* ex = reinterpret_cast<float*>(kv_s);                 // [64 rows][HD + 2]
  constexpr int EXP = HD + 2;
  if (warp >= 4) {
    float* my = ex + (size_t)row * EXP;
#pragma unroll
    for (int d = 0; d < HD; ++d) my[d] = o_acc[d];
    my[HD] = m_run; my[HD + 1] = l_run;
  }
  __syncthreads();
  const int i_row = row0 + row;
  if (warp < 2) {
    const float* th = ex + (size_t)row * EXP;
    const float m1 = th[HD], l1 = th[HD + 1];
    const float mm = fmaxf(m_run, m1);
    const float base = (mm == -INFINITY) ? 0.f : mm;
    const float w0 = exp2f(m_run - base), w1 = exp2f(m1 - base);
    m_run = mm;
    l_run = l_run * w0 + l1 * w1;
#pragma unroll
    for (int d = 0; d < HD; ++d) o_acc[d] = o_acc[d] * w0 + th[d] * w1;
    if (i_row < cnt) {
      const size_t m = (size_t)b * R + i_row;
      if (nsplit == 1) {
        const float inv = 1.f / l_run;
        bf16* po = a.out + m * H * HD + h * HD;
#pragma unroll
        for (int d = 0; d < HD; d += 8) {
          uint4 v;
          v.x = pack_bf16(o_acc[d] * inv, o_acc[d + 1] * inv); v.y = pack_bf16(o_acc[d + 2] * inv, o_acc[d + 3] * inv);
          v.z = pack_bf16(o_acc[d + 4] * inv, o_acc[d + 5] * inv); v.w = pack_bf16(o_acc[d + 6] * inv, o_acc[d + 7] * inv);
          *reinterpret_cast<uint4*>(po + d) = v;
        }
      } else {
        float* po = a.part_o + ((size_t)sp * M + m) * H * HD + h * HD;
#pragma unroll
        for (int d = 0; d < HD; d += 4) *reinterpret_cast<float4*>(po + d) = make_float4(o_acc[d], o_acc[d + 1], o_acc[d + 2], o_acc[d + 3]);
        float* ml = a.part_ml + (((size_t)sp * M + m) * H + h) * 2;
        ml[0] = m_run;
        ml[1] = l_run;
      }
    }
  }
  if (nsplit == 1) return;
  // the CTA of this (sequence, row half, head) that arrives last merges the splits
  __threadfence();
  __syncthreads();
  unsigned int* ctr = a.arrive + ((size_t)b * halves + half) * H + h;
  if (threadIdx.x == 0) {
    const unsigned int old = atomicAdd(ctr, 1u);
    const int last = (old == (unsigned int)(nsplit - 1)) ? 1 : 0;
    if (last) *ctr = 0u;
    last_s = last;
  }
  __syncthreads();
  if (!last_s) return;
  __threadfence();
  {
    // two threads per query row, each merging half of the head dimension
    const int il = threadIdx.x >> 1, d0 = (threadIdx.x & 1) * (HD / 2);
    const int i = row0 + il;
    if (il < AU_ROWS && i < cnt) {
      const size_t m = (size_t)b * R + i;
      float wgt[16];
      float mx = -INFINITY, L = 0.f;
#pragma unroll
      for (int s2 = 0; s2 < 16; ++s2) {
        wgt[s2] = -INFINITY;
        if (s2 < nsplit) wgt[s2] = __ldcg(a.part_ml + (((size_t)s2 * M + m) * H + h) * 2);
        mx = fmaxf(mx, wgt[s2]);
      }
#pragma unroll
      for (int s2 = 0; s2 < 16; ++s2)
        if (s2 < nsplit) {
          const float l2 = __ldcg(a.part_ml + (((size_t)s2 * M + m) * H + h) * 2 + 1);
          wgt[s2] = exp2f(wgt[s2] - mx);
          L += wgt[s2] * l2;
        }
      float acc[HD / 2];
#pragma unroll
      for (int e = 0; e < HD / 2; ++e) acc[e] = 0.f;
#pragma unroll
      for (int s2 = 0; s2 < 16; ++s2) {
        if (s2 >= nsplit) break;
        const float w = wgt[s2];
        const float* src = a.part_o + ((size_t)s2 * M + m) * H * HD + h * HD + d0;
        float4 v[HD / 8];
#pragma unroll
        for (int e = 0; e < HD / 8; ++e) v[e] = __ldcg(reinterpret_cast<const float4*>(src + e * 4));
#pragma unroll
        for (int e = 0; e < HD / 8; ++e) {
          acc[4 * e] += w * v[e].x; acc[4 * e + 1] += w * v[e].y; acc[4 * e + 2] += w * v[e].z; acc[4 * e + 3] += w * v[e].w;
        }
      }
      const float inv = 1.f / L;
      bf16* dst = a.out + m * H * HD + h * HD + d0;
#pragma unroll
      for (int e = 0; e < HD / 8; ++e) {
        uint2 pk;
        pk.x = pack_bf16(acc[4 * e] * inv, acc[4 * e + 1] * inv);
        pk.y = pack_bf16(acc[4 * e + 2] * inv, acc[4 * e + 3] * inv);
        *reinterpret_cast<uint2*>(dst + e * 4) = pk;
      }
    }
  }
}

}  // namespace spec
