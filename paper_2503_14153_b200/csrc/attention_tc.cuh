// Tree-masked decode attention over the paged bf16 KV cache (verification forward of
// Sec. III-B: every tree node attends to all committed positions and to its own ancestors
// in the tree). One CTA per (query head, KV split, sequence) with NW x KG warps: warp
// (rg, kg) owns query rows [16 rg, 16 rg + 16) and every KG-th tile of the split, so two
// tiles are worked on at a time; the key groups' softmax states are merged through shared
// memory at the end. KV tiles of 64 keys are brought in page by page with bulk asynchronous
// copies that complete on an mbarrier (the cache's slab layout -- 64 dims per 128-byte row, chunks
// swizzled with the row -- makes the landed tile conflict-free for ldmatrix); QK^T and PV run on mma.sync m16n8k16 with a warp-level
// online softmax; the tree mask is a 128-bit ancestor set per row applied only to keys at or
// beyond the committed length. Two kernels: attention_rows (at the end of this file) when the
// (sequence, head, 16-row block) CTAs of the pass fit the SMs, attention_tc otherwise. For
// attention_tc the host only picks the launch shape (one split per head for short contexts, or
// up to `nsplit` KV splits per head) from its bound on the context length; how many of the
// launched splits are used, and the tiles of each, follow from the
// sequence length on the device, so one launch shape (and a recorded graph) serves a whole
// range of lengths. With a single split, tiles that hold only rows of earlier steps are
// fetched before the wait on the previous kernel and the CTA writes the normalised bf16 output
// itself; otherwise each split leaves (max, sum, unnormalised output) and the CTA of a
// (sequence, head) that finishes last (arrival counter, no waiting) merges them.
#pragma once
#include "common.cuh"
#include "kernels_simple.cuh"

namespace spec {

__device__ __forceinline__ void ldmatrix_x4(uint32_t addr, uint32_t (&r)[4]) {
  asm("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(addr) : "memory");
}
__device__ __forceinline__ void ldmatrix_x4_trans(uint32_t addr, uint32_t (&r)[4]) {
  asm("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0,%1,%2,%3}, [%4];"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(addr) : "memory");
}
__device__ __forceinline__ void mma_bf16_16816(float (&c)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1) {
  asm(
      "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
      : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
      : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}
__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi) {
  __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
  return *reinterpret_cast<uint32_t*>(&v);
}

constexpr int ATTN_MAX_STAGES = 6;
constexpr int ATTN_PT_CACHE = 256;
constexpr int ATTN_MAX_SEQS = 16;

struct AttnTcArgs {
  const bf16* q;        // [M][H*HD]
  float* part_o;        // [nsplit][M][H*HD] unnormalised
  float* part_ml;       // [nsplit][M][H][2] (running max in log2 units, sum)
  const bf16* pool;
  KVGeom g;
  const int* page_table;
  Rows rows;
  int layer, H;
  int nsplit;           // KV splits launched (gridDim.y); the splits in use are min(nsplit, ceil(tiles / split_tiles))
  int split_tiles;      // fewest KV tiles worth a split of their own
  int stages;           // KV tiles in flight per CTA (2..ATTN_MAX_STAGES, at least KG); sizes the shared memory
  int n_lo[ATTN_MAX_SEQS];   // host's lower bound of each sequence's committed length: keys below it
                             // were written by earlier steps and may be fetched before the dependency wait
  unsigned char order[ATTN_MAX_SEQS];   // attention_umma: sequence taken by the z-th group of CTAs, longest first
  float scale_log2;     // log2(e) / sqrt(head_dim)
  bf16* out;            // [M][H*HD]
  unsigned int* arrive; // [B][H] arrival counters, zero between launches
  int* status;
};

__host__ __device__ inline size_t attention_tc_smem(int head_dim, int nw, int stages) {
  const size_t rowb = (size_t)head_dim * 2;
  return (size_t)nw * 16 * rowb + 2 * (size_t)stages * 64 * rowb + 8 * ATTN_MAX_STAGES + 4 * ATTN_PT_CACHE;
}

// 64 visibility bits of one query row for keys k0 .. k0+63: keys below the committed length n
// are visible, key n + u is visible iff bit u of the row's 128-bit ancestor set is set.
__device__ __forceinline__ unsigned long long attn_vis64(const uint32_t (&an)[4], int k0, int n) {
  const int u0 = k0 - n;
  const unsigned long long A0 = an[0] | ((unsigned long long)an[1] << 32), A1 = an[2] | ((unsigned long long)an[3] << 32);
  if (u0 <= -64) return ~0ull;
  if (u0 < 0) return ((1ull << (-u0)) - 1ull) | (A0 << (-u0));
  if (u0 == 0) return A0;
  if (u0 < 64) return (A0 >> u0) | (A1 << (64 - u0));
  if (u0 == 64) return A1;
  if (u0 < 128) return A1 >> (u0 - 64);
  return 0ull;
}

template <int HD, int NW, int KG>
__global__ void __launch_bounds__(NW * KG * 32)
attention_tc(const AttnTcArgs a, unsigned long long* tr) {
  KTrace kt(tr);
  constexpr int KT = 64;                      // keys per tile
  constexpr int ROWB = HD * 2;                // bytes per row
  constexpr int TILE_BYTES = KT * ROWB;
  constexpr int PAGE_BYTES = 16 * ROWB;
  constexpr int NTHR = NW * KG * 32;
  const int ST = a.stages;
  extern __shared__ __align__(128) uint8_t smem[];
  uint8_t* qs = smem;                                       // [NW*16][HD]
  uint8_t* ks = qs + NW * 16 * ROWB;                        // [ST][page][K | V][16][HD]
  uint64_t* full = reinterpret_cast<uint64_t*>(ks + ST * 2 * TILE_BYTES);   // [ATTN_MAX_STAGES]
  int* pt_s = reinterpret_cast<int*>(full + ATTN_MAX_STAGES);           // [ATTN_PT_CACHE] page-table entries of this split

  pdl_launch_dependents();
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int rg = warp % NW, kg = warp / NW;
  const int h = blockIdx.x, sp = blockIdx.y, b = blockIdx.z;
  constexpr int row0 = 0;                                        // the CTA owns all query rows of its sequence
  const int H = a.H, kvh = h / (H / a.g.n_kv_heads);
  const bool single = a.nsplit == 1;          // one split: its tiles start at 0 whatever the length
  const int* pt = a.page_table + b * a.g.pages_per_seq;
  if (threadIdx.x == 0) {
    for (int i = 0; i < ST; ++i) mbar_init(&full[i], 1);
    mbar_fence_init();
  }
  // the page table is fixed at set-up: with a single split its first entries are staged before the dependency wait
  if (single)
    for (int e = threadIdx.x; e < ATTN_PT_CACHE; e += NTHR) pt_s[e] = e < a.g.pages_per_seq ? pt[e] : 0;
  __syncthreads();   // barriers initialised, page entries staged
  int t0 = 0;
  auto issue = [&](int tile, int buf) {
    mbar_expect_tx(&full[buf], 2 * TILE_BYTES);
    for (int pg = 0; pg < KT / 16; ++pg) {
      const int e = (tile - t0) * (KT / 16) + pg;
      const int page = e < ATTN_PT_CACHE ? pt_s[e] : pt[tile * (KT / 16) + pg];
      // the K block and the V block of a (page, layer, head) are adjacent in the pool: one copy
      bulk_load_1d(ks + buf * 2 * TILE_BYTES + pg * 2 * PAGE_BYTES, a.pool + a.g.block_offset(page, a.layer, 0, kvh),
                   2 * PAGE_BYTES, &full[buf]);
    }
  };
  // tiles that lie wholly below the host's lower bound of the committed length hold rows of
  // earlier steps: start fetching them now (thread 0 keeps the count)
  int pre = 0;
  if (single && threadIdx.x == 0) {
    const int safe = (b < ATTN_MAX_SEQS ? a.n_lo[b] : 0) / KT;      // tiles [0, safe) are committed
    for (; pre < ST && pre < safe; ++pre) issue(pre, pre);
  }
  pdl_wait();
  if (threadIdx.x == 0) trace_mark_min(tr, 2);
  // sequence state, ancestor sets and the Q tile are independent loads: one trip for all of them
  const int R = a.rows.R, cnt = a.rows.cnt[b], n = a.rows.n[b];
  const int i0 = row0 + rg * 16 + (lane >> 2), i1 = i0 + 8;  // this thread's two query rows
  uint32_t anc0[4], anc1[4];
#pragma unroll
  for (int w = 0; w < 4; ++w) { anc0[w] = a.rows.anc[i0 * 4 + w]; anc1[w] = a.rows.anc[i1 * 4 + w]; }
  constexpr int QC = NW * 16 * (HD / 8);                      // 16-byte chunks of the Q tile
  constexpr int PER = (QC + NTHR - 1) / NTHR;
  uint4 qv[PER];
#pragma unroll
  for (int k = 0; k < PER; ++k) {
    const int c = threadIdx.x + k * NTHR;
    const int r = c / (HD / 8), ch = c % (HD / 8);
    qv[k] = make_uint4(0, 0, 0, 0);
    if (c < QC && row0 + r < R) qv[k] = *reinterpret_cast<const uint4*>(a.q + (size_t)(b * R + row0 + r) * H * HD + h * HD + ch * 8);
  }
  const int S = n + cnt;
  const int M = a.rows.B * R;
  const int total_tiles = (S + KT - 1) / KT;
  // the splits in use and their tiles follow from the length: split_tiles tiles or more per split
  const int nsplit = single ? 1 : max(1, min(a.nsplit, (total_tiles + a.split_tiles - 1) / a.split_tiles));
  const int tps = (total_tiles + nsplit - 1) / nsplit;
  t0 = sp * tps;
  const int t1 = min(total_tiles, t0 + tps);
  if (cnt == 0 || sp >= nsplit) {
    // inactive sequence or unused split: let the copies already in flight land before the CTA goes away
    if (threadIdx.x == 0)
      for (int i = 0; i < pre; ++i) mbar_wait(&full[i], 0, a.status, 21);
    return;
  }
  if (!single) {
    for (int e = threadIdx.x; e < tps * (KT / 16) && e < ATTN_PT_CACHE; e += NTHR) {
      const int idx = t0 * (KT / 16) + e;
      pt_s[e] = idx < a.g.pages_per_seq ? pt[idx] : 0;
    }
    __syncthreads();
  }
  // the rest of the first tiles
  if (threadIdx.x == 0)
    for (int i = pre; i < ST && t0 + i < t1; ++i) issue(t0 + i, i);
  // rows beyond cnt see nothing and hold zeros
  if (i0 >= cnt) anc0[0] = anc0[1] = anc0[2] = anc0[3] = 0u;
  if (i1 >= cnt) anc1[0] = anc1[1] = anc1[2] = anc1[3] = 0u;
#pragma unroll
  for (int k = 0; k < PER; ++k) {
    const int c = threadIdx.x + k * NTHR;
    const int r = c / (HD / 8), ch = c % (HD / 8);
    if (c < QC) *reinterpret_cast<uint4*>(qs + r * ROWB + ((ch ^ (r & 7)) << 4)) = (row0 + r < cnt) ? qv[k] : make_uint4(0, 0, 0, 0);
  }
  __syncthreads();

  // Q fragments stay in registers
  uint32_t qf[HD / 16][4];
  {
    int row = rg * 16 + (lane & 7) + ((lane >> 3) & 1) * 8;
#pragma unroll
    for (int kk = 0; kk < HD / 16; ++kk) {
      int ch = kk * 2 + (lane >> 4);
      ldmatrix_x4(smem_u32(qs + row * ROWB + ((ch ^ (row & 7)) << 4)), qf[kk]);
    }
  }

  float o[HD / 8][4];
#pragma unroll
  for (int d = 0; d < HD / 8; ++d) o[d][0] = o[d][1] = o[d][2] = o[d][3] = 0.f;
  float mrow[2] = {-INFINITY, -INFINITY}, lrow[2] = {0.f, 0.f};

  bool ok = true;
  const int ntile = t1 - t0;
  for (int it = 0; it < ntile; it += KG) {
    const int my = it + kg;                 // this warp's tile of the round, relative to t0
    const bool have = my < ntile;
    if (have && !mbar_wait(&full[my % ST], (my / ST) & 1, a.status, 20)) ok = false;
    ok = __syncthreads_and(ok);
    if (!ok) break;
    if (it == 0 && threadIdx.x == 0) trace_mark_max(tr, 3);
    if (have) {
      const int t = t0 + my;
      const uint8_t* kt = ks + (my % ST) * 2 * TILE_BYTES;   // key `key` of the tile: page key / 16, row key % 16
      const uint8_t* vt = kt + PAGE_BYTES;
      float s[KT / 8][4];
#pragma unroll
      for (int j = 0; j < KT / 8; ++j) s[j][0] = s[j][1] = s[j][2] = s[j][3] = 0.f;
      // K fragments of a 16-wide slice of the head dimension are fetched together, one slice
      // ahead of the MMAs that use them
      {
        uint32_t kf[2][KT / 16][4];
        auto load_k = [&](int kk, uint32_t (&dst)[KT / 16][4]) {
#pragma unroll
          for (int j2 = 0; j2 < KT / 16; ++j2) {
            int key = j2 * 16 + (lane & 7) + (lane >> 4) * 8;
            int ch = kk * 2 + ((lane >> 3) & 1);
            ldmatrix_x4(smem_u32(kt + (key >> 4) * 2 * PAGE_BYTES + (ch >> 3) * 2048 + (key & 15) * 128 + (((ch & 7) ^ (key & 7)) << 4)), dst[j2]);
          }
        };
        load_k(0, kf[0]);
#pragma unroll
        for (int kk = 0; kk < HD / 16; ++kk) {
          if (kk + 1 < HD / 16) load_k(kk + 1, kf[(kk + 1) & 1]);
#pragma unroll
          for (int j2 = 0; j2 < KT / 16; ++j2) {
            mma_bf16_16816(s[2 * j2], qf[kk], kf[kk & 1][j2][0], kf[kk & 1][j2][1]);
            mma_bf16_16816(s[2 * j2 + 1], qf[kk], kf[kk & 1][j2][2], kf[kk & 1][j2][3]);
          }
        }
      }
      // mask + online softmax (log2 domain)
      const int k0 = t * KT;
      const bool need_mask = (k0 + KT > n);
      unsigned long long vis0 = ~0ull, vis1 = ~0ull;
      if (need_mask) { vis0 = attn_vis64(anc0, k0, n); vis1 = attn_vis64(anc1, k0, n); }
      float tmax[2] = {-INFINITY, -INFINITY};
#pragma unroll
      for (int j = 0; j < KT / 8; ++j) {
#pragma unroll
        for (int e = 0; e < 4; ++e) {
          float v = s[j][e] * a.scale_log2;
          const int bi = j * 8 + (lane & 3) * 2 + (e & 1);
          if (!(((e < 2 ? vis0 : vis1) >> bi) & 1ull)) v = -INFINITY;
          s[j][e] = v;
          tmax[e >> 1] = fmaxf(tmax[e >> 1], v);
        }
      }
      float alpha[2], mnew[2];
#pragma unroll
      for (int r = 0; r < 2; ++r) {
        tmax[r] = fmaxf(tmax[r], __shfl_xor_sync(0xffffffffu, tmax[r], 1));
        tmax[r] = fmaxf(tmax[r], __shfl_xor_sync(0xffffffffu, tmax[r], 2));
        mnew[r] = fmaxf(mrow[r], tmax[r]);
        float base = (mnew[r] == -INFINITY) ? 0.f : mnew[r];
        alpha[r] = exp2f(mrow[r] - base);
        mrow[r] = mnew[r];
        mnew[r] = base;
        lrow[r] *= alpha[r];
      }
#pragma unroll
      for (int d = 0; d < HD / 8; ++d) { o[d][0] *= alpha[0]; o[d][1] *= alpha[0]; o[d][2] *= alpha[1]; o[d][3] *= alpha[1]; }
      uint32_t pf[KT / 16][4];
#pragma unroll
      for (int j = 0; j < KT / 8; ++j) {
        float p0 = exp2f(s[j][0] - mnew[0]), p1 = exp2f(s[j][1] - mnew[0]);
        float p2 = exp2f(s[j][2] - mnew[1]), p3 = exp2f(s[j][3] - mnew[1]);
        lrow[0] += p0 + p1;
        lrow[1] += p2 + p3;
        pf[j >> 1][(j & 1) * 2 + 0] = pack_bf16(p0, p1);
        pf[j >> 1][(j & 1) * 2 + 1] = pack_bf16(p2, p3);
      }
      // V fragments: four 16-wide slices of the head dimension at a time, one group ahead
      {
        constexpr int DG = 4, NG = (KT / 16) * (HD / 16) / DG;
        uint32_t vf[2][DG][4];
        auto load_v = [&](int g, uint32_t (&dst)[DG][4]) {
          const int j = g / (HD / 16 / DG), d0 = (g % (HD / 16 / DG)) * DG;
#pragma unroll
          for (int dd = 0; dd < DG; ++dd) {
            int key = j * 16 + (lane & 7) + ((lane >> 3) & 1) * 8;
            int ch = (d0 + dd) * 2 + (lane >> 4);
            ldmatrix_x4_trans(smem_u32(vt + (key >> 4) * 2 * PAGE_BYTES + (ch >> 3) * 2048 + (key & 15) * 128 + (((ch & 7) ^ (key & 7)) << 4)), dst[dd]);
          }
        };
        load_v(0, vf[0]);
#pragma unroll
        for (int g = 0; g < NG; ++g) {
          if (g + 1 < NG) load_v(g + 1, vf[(g + 1) & 1]);
          const int j = g / (HD / 16 / DG), d0 = (g % (HD / 16 / DG)) * DG;
#pragma unroll
          for (int dd = 0; dd < DG; ++dd) {
            mma_bf16_16816(o[2 * (d0 + dd)], pf[j], vf[g & 1][dd][0], vf[g & 1][dd][1]);
            mma_bf16_16816(o[2 * (d0 + dd) + 1], pf[j], vf[g & 1][dd][2], vf[g & 1][dd][3]);
          }
        }
      }
    }
    __syncthreads();   // the round's tiles are consumed: their buffers may be refilled
    if (threadIdx.x == 0)
      for (int g = 0; g < KG; ++g)
        if (it + g + ST < ntile) issue(t0 + it + g + ST, (it + g) % ST);
  }
  if (!ok) return;

#pragma unroll
  for (int r = 0; r < 2; ++r) {
    lrow[r] += __shfl_xor_sync(0xffffffffu, lrow[r], 1);
    lrow[r] += __shfl_xor_sync(0xffffffffu, lrow[r], 2);
  }
  if (KG > 1) {
    // merge the key groups' states through the (now idle) KV buffers: groups 1.. leave theirs,
    // group 0 adds them in group order
    float* ex = reinterpret_cast<float*>(ks);
    constexpr int GT = NW * 32;                                // threads per key group
    constexpr int SLOT = (HD / 2 + 4) * GT;                    // floats per group state
    const int gt = rg * 32 + lane;
    if (kg > 0) {
      float* my = ex + (size_t)(kg - 1) * SLOT;
#pragma unroll
      for (int d = 0; d < HD / 8; ++d)
#pragma unroll
        for (int e = 0; e < 4; ++e) my[(d * 4 + e) * GT + gt] = o[d][e];
      my[(HD / 2 + 0) * GT + gt] = mrow[0]; my[(HD / 2 + 1) * GT + gt] = mrow[1];
      my[(HD / 2 + 2) * GT + gt] = lrow[0]; my[(HD / 2 + 3) * GT + gt] = lrow[1];
    }
    __syncthreads();
    if (kg == 0) {
#pragma unroll 1
      for (int g2 = 1; g2 < KG; ++g2) {
        const float* th = ex + (size_t)(g2 - 1) * SLOT;
        float w0[2], w1[2];
#pragma unroll
        for (int r = 0; r < 2; ++r) {
          const float m1 = th[(HD / 2 + r) * GT + gt], l1 = th[(HD / 2 + 2 + r) * GT + gt];
          const float mm = fmaxf(mrow[r], m1);
          const float base = (mm == -INFINITY) ? 0.f : mm;
          w0[r] = exp2f(mrow[r] - base);
          w1[r] = exp2f(m1 - base);
          mrow[r] = mm;
          lrow[r] = lrow[r] * w0[r] + l1 * w1[r];
        }
#pragma unroll
        for (int d = 0; d < HD / 8; ++d)
#pragma unroll
          for (int e = 0; e < 4; ++e) o[d][e] = o[d][e] * w0[e >> 1] + th[(d * 4 + e) * GT + gt] * w1[e >> 1];
      }
    }
  }
  if (nsplit == 1) {
    // the only split: normalise and store the bf16 output
    if (kg == 0) {
#pragma unroll
      for (int r = 0; r < 2; ++r) {
        int i = r ? i1 : i0;
        if (i >= cnt) continue;
        const float inv = 1.f / lrow[r];
        bf16* po = a.out + ((size_t)b * R + i) * H * HD + h * HD;
#pragma unroll
        for (int d = 0; d < HD / 8; ++d)
          *reinterpret_cast<uint32_t*>(po + d * 8 + (lane & 3) * 2) = pack_bf16(o[d][2 * r] * inv, o[d][2 * r + 1] * inv);
      }
    }
    return;
  }
  if (kg == 0) {
#pragma unroll
    for (int r = 0; r < 2; ++r) {
      int i = r ? i1 : i0;
      if (i >= cnt) continue;
      size_t m = (size_t)b * R + i;
      float* po = a.part_o + ((size_t)sp * M + m) * H * HD + h * HD;
#pragma unroll
      for (int d = 0; d < HD / 8; ++d)
        *reinterpret_cast<float2*>(po + d * 8 + (lane & 3) * 2) = make_float2(o[d][2 * r], o[d][2 * r + 1]);
      if ((lane & 3) == 0) {
        float* ml = a.part_ml + (((size_t)sp * M + m) * H + h) * 2;
        ml[0] = mrow[r];
        ml[1] = lrow[r];
      }
    }
  }
  // the CTA of this (sequence, head) that arrives last merges the splits
  __shared__ int last_s;
  __threadfence();
  __syncthreads();
  if (threadIdx.x == 0) {
    const unsigned int old = atomicAdd(a.arrive + b * H + h, 1u);
    const int last = (old == (unsigned int)(nsplit - 1)) ? 1 : 0;
    if (last) a.arrive[b * H + h] = 0u;
    last_s = last;
  }
  __syncthreads();
  if (!last_s) return;
  __threadfence();
  // two threads per query row, each merging half of the head dimension
  {
    const int i = threadIdx.x >> 1, d0 = (threadIdx.x & 1) * (HD / 2);
    if (i < cnt && i < NW * 16) {
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

// ------------------------------------------------------------------ one CTA per (head, 16 query rows)
// The same attention for passes whose (sequence, head, 16-row block) count fits the GPU's SMs: a
// CTA owns 16 query rows of one head and walks the whole context, so there is nothing to merge
// across CTAs and the launch does not depend on the context length at all. Each of the W warps
// streams its own sub-tiles of 32 keys (two cache pages; sub-tile w, w + W, ...) through two
// private buffers: it waits for a buffer, works on it (QK^T, mask, online softmax, PV) and asks
// for its next-but-one sub-tile into the same buffer, without any CTA-wide barrier in the
// loop. The warps' softmax states are merged through shared memory at the end and warp 0
// writes the normalised bf16 rows. Sub-tiles below the host's lower bound of the committed
// length are requested before the wait on the previous kernel.
__host__ __device__ inline size_t attention_rows_smem(int head_dim, int warps) {
  const size_t rowb = (size_t)head_dim * 2;
  return 16 * rowb + (size_t)warps * 2 * 2 * 32 * rowb + 8 * (size_t)warps * 2 + 4 * ATTN_PT_CACHE;
}

template <int HD, int W>
__global__ void __launch_bounds__(W * 32)
attention_rows(const AttnTcArgs a, unsigned long long* tr) {
  KTrace kt(tr);
  constexpr int SK = 32;                      // keys per sub-tile
  constexpr int NB = 2;                       // buffers per warp
  constexpr int ROWB = HD * 2;                // bytes per row
  constexpr int SUB_BYTES = SK * ROWB;        // one operand of a sub-tile
  constexpr int PAGE_BYTES = 16 * ROWB;
  constexpr int NTHR = W * 32;
  extern __shared__ __align__(128) uint8_t smem[];
  uint8_t* qs = smem;                                                        // [16][HD]
  uint8_t* kv = qs + 16 * ROWB;                                              // [W][NB][page][K | V][16][HD]
  uint64_t* full = reinterpret_cast<uint64_t*>(kv + W * NB * 2 * SUB_BYTES); // [W][NB]
  int* pt_s = reinterpret_cast<int*>(full + W * NB);                         // [ATTN_PT_CACHE]

  pdl_launch_dependents();
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int h = blockIdx.x, b = blockIdx.z, row0 = blockIdx.y * 16;
  const int H = a.H, kvh = h / (H / a.g.n_kv_heads);
  const int* pt = a.page_table + b * a.g.pages_per_seq;
  if (threadIdx.x == 0) {
    for (int i = 0; i < W * NB; ++i) mbar_init(&full[i], 1);
    mbar_fence_init();
  }
  for (int e = threadIdx.x; e < ATTN_PT_CACHE; e += NTHR) pt_s[e] = e < a.g.pages_per_seq ? pt[e] : 0;
  __syncthreads();   // barriers initialised, page entries staged
  uint8_t* mine = kv + (size_t)warp * NB * 2 * SUB_BYTES;
  uint64_t* my_full = full + warp * NB;
  auto issue = [&](int st, int bf) {          // lane 0: sub-tile st of this sequence into buffer bf
    mbar_expect_tx(&my_full[bf], 2 * SUB_BYTES);
#pragma unroll
    for (int pg = 0; pg < SK / 16; ++pg) {
      const int e = st * (SK / 16) + pg;
      const int page = e < ATTN_PT_CACHE ? pt_s[e] : pt[e];
      // the K block and the V block of a (page, layer, head) are adjacent in the pool: one copy
      bulk_load_1d(mine + bf * 2 * SUB_BYTES + pg * 2 * PAGE_BYTES, a.pool + a.g.block_offset(page, a.layer, 0, kvh), 2 * PAGE_BYTES, &my_full[bf]);
    }
  };
  // own sub-tiles that lie wholly below the host's lower bound hold rows of earlier steps
  int issued = 0;                             // own sub-tiles requested so far (same in every lane)
  {
    const int safe = (b < ATTN_MAX_SEQS ? a.n_lo[b] : 0) / SK;
    while (issued < NB && warp + issued * W < safe) {
      if (lane == 0) issue(warp + issued * W, issued);
      ++issued;
    }
  }
  pdl_wait();
  if (threadIdx.x == 0) trace_mark_min(tr, 2);
  const int R = a.rows.R, cnt = a.rows.cnt[b], n = a.rows.n[b];
  const int i0 = row0 + (lane >> 2), i1 = i0 + 8;          // this thread's two query rows
  uint32_t anc0[4], anc1[4];
#pragma unroll
  for (int w = 0; w < 4; ++w) { anc0[w] = a.rows.anc[i0 * 4 + w]; anc1[w] = a.rows.anc[i1 * 4 + w]; }
  constexpr int QC = 16 * (HD / 8);                          // 16-byte chunks of the Q tile
  constexpr int PER = (QC + NTHR - 1) / NTHR;
  uint4 qv[PER];
#pragma unroll
  for (int k = 0; k < PER; ++k) {
    const int c = threadIdx.x + k * NTHR;
    const int r = c / (HD / 8), ch = c % (HD / 8);
    qv[k] = make_uint4(0, 0, 0, 0);
    if (c < QC && row0 + r < R) qv[k] = *reinterpret_cast<const uint4*>(a.q + (size_t)(b * R + row0 + r) * H * HD + h * HD + ch * 8);
  }
  const int S = n + cnt;
  const int n_sub = (S + SK - 1) / SK;
  if (row0 >= cnt) {
    // no valid row in this block: let the copies already in flight land before the CTA goes away
    if (lane == 0)
      for (int i = 0; i < issued; ++i) mbar_wait(&my_full[i], 0, a.status, 21);
    return;
  }
  while (issued < NB && warp + issued * W < n_sub) {
    if (lane == 0) issue(warp + issued * W, issued);
    ++issued;
  }
  if (i0 >= cnt) anc0[0] = anc0[1] = anc0[2] = anc0[3] = 0u;
  if (i1 >= cnt) anc1[0] = anc1[1] = anc1[2] = anc1[3] = 0u;
#pragma unroll
  for (int k = 0; k < PER; ++k) {
    const int c = threadIdx.x + k * NTHR;
    const int r = c / (HD / 8), ch = c % (HD / 8);
    if (c < QC) *reinterpret_cast<uint4*>(qs + r * ROWB + ((ch ^ (r & 7)) << 4)) = (row0 + r < cnt) ? qv[k] : make_uint4(0, 0, 0, 0);
  }
  __syncthreads();
  uint32_t qf[HD / 16][4];
  {
    const int row = (lane & 7) + ((lane >> 3) & 1) * 8;
#pragma unroll
    for (int kk = 0; kk < HD / 16; ++kk) {
      const int ch = kk * 2 + (lane >> 4);
      ldmatrix_x4(smem_u32(qs + row * ROWB + ((ch ^ (row & 7)) << 4)), qf[kk]);
    }
  }
  float o[HD / 8][4];
#pragma unroll
  for (int d = 0; d < HD / 8; ++d) o[d][0] = o[d][1] = o[d][2] = o[d][3] = 0.f;
  float mrow[2] = {-INFINITY, -INFINITY}, lrow[2] = {0.f, 0.f};

  bool ok = true;
  int k = 0;                                   // own sub-tiles done
  for (int st = warp; st < n_sub; st += W, ++k) {
    const int bf = k % NB;
    if (!mbar_wait(&my_full[bf], (k / NB) & 1, a.status, 20)) { ok = false; break; }
    if (st == 0 && lane == 0) trace_mark_max(tr, 3);
    const uint8_t* kt = mine + bf * 2 * SUB_BYTES;     // key `key` of the sub-tile: page key / 16, row key % 16
    const uint8_t* vt = kt + PAGE_BYTES;
    float s[SK / 8][4];
#pragma unroll
    for (int j = 0; j < SK / 8; ++j) s[j][0] = s[j][1] = s[j][2] = s[j][3] = 0.f;
    {
      // K fragments of a 16-wide slice of the head dimension, one slice ahead of the MMAs that use them
      uint32_t kf[2][SK / 16][4];
      auto load_k = [&](int kk, uint32_t (&dst)[SK / 16][4]) {
#pragma unroll
        for (int j2 = 0; j2 < SK / 16; ++j2) {
          const int key = j2 * 16 + (lane & 7) + (lane >> 4) * 8;
          const int ch = kk * 2 + ((lane >> 3) & 1);
          ldmatrix_x4(smem_u32(kt + (key >> 4) * 2 * PAGE_BYTES + (ch >> 3) * 2048 + (key & 15) * 128 + (((ch & 7) ^ (key & 7)) << 4)), dst[j2]);
        }
      };
      load_k(0, kf[0]);
#pragma unroll
      for (int kk = 0; kk < HD / 16; ++kk) {
        if (kk + 1 < HD / 16) load_k(kk + 1, kf[(kk + 1) & 1]);
#pragma unroll
        for (int j2 = 0; j2 < SK / 16; ++j2) {
          mma_bf16_16816(s[2 * j2], qf[kk], kf[kk & 1][j2][0], kf[kk & 1][j2][1]);
          mma_bf16_16816(s[2 * j2 + 1], qf[kk], kf[kk & 1][j2][2], kf[kk & 1][j2][3]);
        }
      }
    }
    // mask + online softmax (log2 domain)
    const int k0 = st * SK;
    float tmax[2] = {-INFINITY, -INFINITY};
    if (k0 + SK > n) {
      // the sub-tile reaches into the tree rows: per-key visibility
      const uint32_t vis0 = (uint32_t)attn_vis64(anc0, k0, n), vis1 = (uint32_t)attn_vis64(anc1, k0, n);
#pragma unroll
      for (int j = 0; j < SK / 8; ++j) {
#pragma unroll
        for (int e = 0; e < 4; ++e) {
          float v = s[j][e] * a.scale_log2;
          const int bi = j * 8 + (lane & 3) * 2 + (e & 1);
          if (!(((e < 2 ? vis0 : vis1) >> bi) & 1u)) v = -INFINITY;
          s[j][e] = v;
          tmax[e >> 1] = fmaxf(tmax[e >> 1], v);
        }
      }
    } else {
      // committed positions only: every key is visible to every row
#pragma unroll
      for (int j = 0; j < SK / 8; ++j) {
#pragma unroll
        for (int e = 0; e < 4; ++e) {
          s[j][e] *= a.scale_log2;
          tmax[e >> 1] = fmaxf(tmax[e >> 1], s[j][e]);
        }
      }
    }
    float alpha[2], mnew[2];
#pragma unroll
    for (int r = 0; r < 2; ++r) {
      tmax[r] = fmaxf(tmax[r], __shfl_xor_sync(0xffffffffu, tmax[r], 1));
      tmax[r] = fmaxf(tmax[r], __shfl_xor_sync(0xffffffffu, tmax[r], 2));
      mnew[r] = fmaxf(mrow[r], tmax[r]);
      const float base = (mnew[r] == -INFINITY) ? 0.f : mnew[r];
      alpha[r] = exp2f(mrow[r] - base);
      mrow[r] = mnew[r];
      mnew[r] = base;
      lrow[r] *= alpha[r];
    }
#pragma unroll
    for (int d = 0; d < HD / 8; ++d) { o[d][0] *= alpha[0]; o[d][1] *= alpha[0]; o[d][2] *= alpha[1]; o[d][3] *= alpha[1]; }
    uint32_t pf[SK / 16][4];
#pragma unroll
    for (int j = 0; j < SK / 8; ++j) {
      const float p0 = exp2f(s[j][0] - mnew[0]), p1 = exp2f(s[j][1] - mnew[0]);
      const float p2 = exp2f(s[j][2] - mnew[1]), p3 = exp2f(s[j][3] - mnew[1]);
      lrow[0] += p0 + p1;
      lrow[1] += p2 + p3;
      pf[j >> 1][(j & 1) * 2 + 0] = pack_bf16(p0, p1);
      pf[j >> 1][(j & 1) * 2 + 1] = pack_bf16(p2, p3);
    }
    {
      // V fragments: four 16-wide slices of the head dimension at a time, one group ahead
      constexpr int DG = 4, NG = (SK / 16) * (HD / 16) / DG;
      uint32_t vf[2][DG][4];
      auto load_v = [&](int g, uint32_t (&dst)[DG][4]) {
        const int j = g / (HD / 16 / DG), d0 = (g % (HD / 16 / DG)) * DG;
#pragma unroll
        for (int dd = 0; dd < DG; ++dd) {
          const int key = j * 16 + (lane & 7) + ((lane >> 3) & 1) * 8;
          const int ch = (d0 + dd) * 2 + (lane >> 4);
          ldmatrix_x4_trans(smem_u32(vt + (key >> 4) * 2 * PAGE_BYTES + (ch >> 3) * 2048 + (key & 15) * 128 + (((ch & 7) ^ (key & 7)) << 4)), dst[dd]);
        }
      };
      load_v(0, vf[0]);
#pragma unroll
      for (int g = 0; g < NG; ++g) {
        if (g + 1 < NG) load_v(g + 1, vf[(g + 1) & 1]);
        const int j = g / (HD / 16 / DG), d0 = (g % (HD / 16 / DG)) * DG;
#pragma unroll
        for (int dd = 0; dd < DG; ++dd) {
          mma_bf16_16816(o[2 * (d0 + dd)], pf[j], vf[g & 1][dd][0], vf[g & 1][dd][1]);
          mma_bf16_16816(o[2 * (d0 + dd) + 1], pf[j], vf[g & 1][dd][2], vf[g & 1][dd][3]);
        }
      }
    }
    __syncwarp();                              // every lane has read the buffer: it may be refilled
    const int nxt = st + NB * W;
    if (nxt < n_sub && lane == 0) issue(nxt, bf);
  }
  if (!ok && lane == 0) {
    // a wait gave up: the other copy this warp may still have in flight gets a bounded time to land
    const int st1 = warp + (k + 1) * W;
    if (st1 < n_sub) mbar_wait(&my_full[(k + 1) % NB], ((k + 1) / NB) & 1, a.status, 22);
  }
  ok = __syncthreads_and(ok);                  // all warps are done with their buffers
  if (!ok) return;

#pragma unroll
  for (int r = 0; r < 2; ++r) {
    lrow[r] += __shfl_xor_sync(0xffffffffu, lrow[r], 1);
    lrow[r] += __shfl_xor_sync(0xffffffffu, lrow[r], 2);
  }
  // merge the warps' states through the (now idle) KV buffers: warps 1.. leave theirs, warp 0 adds
  // them in warp order
  float* ex = reinterpret_cast<float*>(kv);
  constexpr int SLOT = (HD / 2 + 4) * 32;       // floats per warp state
  if (warp > 0) {
    float* my = ex + (size_t)(warp - 1) * SLOT;
#pragma unroll
    for (int d = 0; d < HD / 8; ++d)
#pragma unroll
      for (int e = 0; e < 4; ++e) my[(d * 4 + e) * 32 + lane] = o[d][e];
    my[(HD / 2 + 0) * 32 + lane] = mrow[0]; my[(HD / 2 + 1) * 32 + lane] = mrow[1];
    my[(HD / 2 + 2) * 32 + lane] = lrow[0]; my[(HD / 2 + 3) * 32 + lane] = lrow[1];
  }
  __syncthreads();
  if (warp != 0) return;
#pragma unroll 1
  for (int g2 = 1; g2 < W; ++g2) {
    const float* th = ex + (size_t)(g2 - 1) * SLOT;
    float w0[2], w1[2];
#pragma unroll
    for (int r = 0; r < 2; ++r) {
      const float m1 = th[(HD / 2 + r) * 32 + lane], l1 = th[(HD / 2 + 2 + r) * 32 + lane];
      const float mm = fmaxf(mrow[r], m1);
      const float base = (mm == -INFINITY) ? 0.f : mm;
      w0[r] = exp2f(mrow[r] - base);
      w1[r] = exp2f(m1 - base);
      mrow[r] = mm;
      lrow[r] = lrow[r] * w0[r] + l1 * w1[r];
    }
#pragma unroll
    for (int d = 0; d < HD / 8; ++d)
#pragma unroll
      for (int e = 0; e < 4; ++e) o[d][e] = o[d][e] * w0[e >> 1] + th[(d * 4 + e) * 32 + lane] * w1[e >> 1];
  }
#pragma unroll
  for (int r = 0; r < 2; ++r) {
    const int i = r ? i1 : i0;
    if (i >= cnt) continue;
    const float inv = 1.f / lrow[r];
    bf16* po = a.out + ((size_t)b * R + i) * H * HD + h * HD;
#pragma unroll
    for (int d = 0; d < HD / 8; ++d)
      *reinterpret_cast<uint32_t*>(po + d * 8 + (lane & 3) * 2) = pack_bf16(o[d][2 * r] * inv, o[d][2 * r + 1] * inv);
  }
}

// ------------------------------------------------------------------ long contexts: shared K/V tiles, split keys
// At thousands of cached positions the kernel above reads a head's K/V once per 16-row block (four
// times at 64 tree rows) and keeps only six warps on an SM. Here a CTA owns up to 64 query rows of one
// head (AS_RB blocks of 16) and one split of the keys, with AS_RB x AS_KP warps: warp (rb, kp) works on
// rows [16 rb, +16) and on every AS_KP-th sub-tile of 32 keys of the split. The AS_RB warps of a key
// phase share a ring of AS_NB sub-tile buffers (full / empty mbarriers per buffer, no CTA-wide barrier in
// the loop): lane 0 of the phase's first warp refills a buffer once all of the phase's warps have
// released it. K/V therefore reach the SM once per 64 rows, and twelve warps hide each other's MMA and
// softmax latencies. The key phases are merged through shared memory, the splits by the CTA that arrives
// last (as in attention_tc). Grid (heads, splits, sequences x row halves); the splits in use and their
// sub-tiles follow from the sequence length on the device.
constexpr int AS_RB = 4, AS_KP = 3, AS_NB = 4;
constexpr int AS_SPLIT_SUB = 16;              // fewest sub-tiles worth a split of their own

__host__ __device__ inline size_t attention_shared_smem(int head_dim) {
  const size_t rowb = (size_t)head_dim * 2;
  return AS_RB * 16 * rowb + (size_t)AS_KP * AS_NB * 2 * 32 * rowb + 8 * (size_t)(2 * AS_KP * AS_NB) + 4 * ATTN_PT_CACHE;
}

template <int HD>
__global__ void __launch_bounds__(AS_RB * AS_KP * 32, 1)
attention_shared(const AttnTcArgs a, unsigned long long* tr) {
  KTrace kt(tr);
  constexpr int SK = 32;                      // keys per sub-tile
  constexpr int ROWB = HD * 2;
  constexpr int SUB_BYTES = SK * ROWB;        // one operand of a sub-tile
  constexpr int PAGE_BYTES = 16 * ROWB;
  constexpr int NTHR = AS_RB * AS_KP * 32;
  extern __shared__ __align__(128) uint8_t smem[];
  uint8_t* qs = smem;                                                              // [AS_RB*16][HD]
  uint8_t* kv = qs + AS_RB * 16 * ROWB;                                            // [AS_KP][AS_NB][page][K | V][16][HD]
  uint64_t* full = reinterpret_cast<uint64_t*>(kv + AS_KP * AS_NB * 2 * SUB_BYTES);  // [AS_KP][AS_NB]
  uint64_t* empty = full + AS_KP * AS_NB;                                          // [AS_KP][AS_NB]
  int* pt_s = reinterpret_cast<int*>(empty + AS_KP * AS_NB);                       // [ATTN_PT_CACHE]

  pdl_launch_dependents();
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int rb = warp % AS_RB, kp = warp / AS_RB;
  const int halves = gridDim.z / a.rows.B;
  const int h = blockIdx.x, sp = blockIdx.y, b = blockIdx.z / halves, half = blockIdx.z % halves;
  const int row0 = half * (AS_RB * 16);
  const int H = a.H, kvh = h / (H / a.g.n_kv_heads);
  const int* pt = a.page_table + b * a.g.pages_per_seq;
  pdl_wait();
  if (threadIdx.x == 0) trace_mark_min(tr, 2);
  const int R = a.rows.R, cnt = a.rows.cnt[b], n = a.rows.n[b];
  const int S = n + cnt, M = a.rows.B * R;
  const int n_sub = (S + SK - 1) / SK;
  const int nsplit = max(1, min(a.nsplit, (n_sub + AS_SPLIT_SUB - 1) / AS_SPLIT_SUB));
  const int sps = (n_sub + nsplit - 1) / nsplit;
  const int st0 = sp * sps, st1 = min(n_sub, st0 + sps);
  if (row0 >= cnt || sp >= nsplit) return;                        // nothing in flight yet
  const int nrb = min(AS_RB, (cnt - row0 + 15) >> 4);              // row blocks with a valid row
  if (threadIdx.x == 0) {
    for (int i = 0; i < AS_KP * AS_NB; ++i) { mbar_init(&full[i], 1); mbar_init(&empty[i], nrb); }
    mbar_fence_init();
  }
  for (int e = threadIdx.x; e < ATTN_PT_CACHE; e += NTHR) {
    const int idx = st0 * (SK / 16) + e;
    pt_s[e] = idx < a.g.pages_per_seq ? pt[idx] : 0;
  }
  // Q tile of the CTA's rows (rows beyond cnt hold zeros)
  const int i0 = row0 + rb * 16 + (lane >> 2), i1 = i0 + 8;    // this thread's two query rows
  uint32_t anc0[4], anc1[4];
#pragma unroll
  for (int w = 0; w < 4; ++w) { anc0[w] = i0 < cnt ? a.rows.anc[i0 * 4 + w] : 0u; anc1[w] = i1 < cnt ? a.rows.anc[i1 * 4 + w] : 0u; }
  constexpr int QC = AS_RB * 16 * (HD / 8);
  for (int c = threadIdx.x; c < QC; c += NTHR) {
    const int r = c / (HD / 8), ch = c % (HD / 8);
    uint4 v = make_uint4(0, 0, 0, 0);
    if (row0 + r < cnt) v = *reinterpret_cast<const uint4*>(a.q + (size_t)(b * R + row0 + r) * H * HD + h * HD + ch * 8);
    *reinterpret_cast<uint4*>(qs + r * ROWB + ((ch ^ (r & 7)) << 4)) = v;
  }
  __syncthreads();   // barriers initialised, page entries and Q staged

  uint8_t* ring = kv + (size_t)kp * AS_NB * 2 * SUB_BYTES;
  uint64_t* my_full = full + kp * AS_NB;
  uint64_t* my_empty = empty + kp * AS_NB;
  const int my_count = st0 + kp < st1 ? (st1 - st0 - kp + AS_KP - 1) / AS_KP : 0;    // sub-tiles of this key phase
  auto issue = [&](int idx) {                                  // lane 0 of the phase's first warp
    const int st = st0 + kp + idx * AS_KP, bf = idx % AS_NB;
    mbar_expect_tx(&my_full[bf], 2 * SUB_BYTES);
#pragma unroll
    for (int pg = 0; pg < SK / 16; ++pg) {
      const int e = (st - st0) * (SK / 16) + pg;
      const int page = e < ATTN_PT_CACHE ? pt_s[e] : pt[st * (SK / 16) + pg];
      bulk_load_1d(ring + bf * 2 * SUB_BYTES + pg * 2 * PAGE_BYTES, a.pool + a.g.block_offset(page, a.layer, 0, kvh), 2 * PAGE_BYTES, &my_full[bf]);
    }
  };
  bool ok = true;
  int issued = 0;
  float o[HD / 8][4];
#pragma unroll
  for (int d = 0; d < HD / 8; ++d) o[d][0] = o[d][1] = o[d][2] = o[d][3] = 0.f;
  float mrow[2] = {-INFINITY, -INFINITY}, lrow[2] = {0.f, 0.f};
  if (rb < nrb) {
    uint32_t qf[HD / 16][4];
    {
      const int row = rb * 16 + (lane & 7) + ((lane >> 3) & 1) * 8;
#pragma unroll
      for (int kk = 0; kk < HD / 16; ++kk) {
        const int ch = kk * 2 + (lane >> 4);
        ldmatrix_x4(smem_u32(qs + row * ROWB + ((ch ^ (row & 7)) << 4)), qf[kk]);
      }
    }
    for (int j = 0; j < my_count; ++j) {
      const int bf = j % AS_NB;
      if (rb == 0) {
        // keep AS_NB sub-tiles of this phase in flight: a buffer is refilled once every warp of the phase released it
        const int upto = min(j + AS_NB, my_count);
        while (issued < upto && ok) {
          if (issued >= AS_NB && !mbar_wait(&my_empty[issued % AS_NB], ((issued / AS_NB) - 1) & 1, a.status, 23)) { ok = false; break; }
          if (lane == 0) issue(issued);
          ++issued;
        }
        if (!ok) break;
      }
      if (!mbar_wait(&my_full[bf], (j / AS_NB) & 1, a.status, 20)) { ok = false; break; }
      const int st = st0 + kp + j * AS_KP;
      if (st == 0 && rb == 0 && lane == 0) trace_mark_max(tr, 3);
      const uint8_t* ktile = ring + bf * 2 * SUB_BYTES;     // key `key` of the sub-tile: page key / 16, row key % 16
      const uint8_t* vtile = ktile + PAGE_BYTES;
      float s[SK / 8][4];
#pragma unroll
      for (int jj = 0; jj < SK / 8; ++jj) s[jj][0] = s[jj][1] = s[jj][2] = s[jj][3] = 0.f;
      {
        uint32_t kf[2][SK / 16][4];
        auto load_k = [&](int kk, uint32_t (&dst)[SK / 16][4]) {
#pragma unroll
          for (int j2 = 0; j2 < SK / 16; ++j2) {
            const int key = j2 * 16 + (lane & 7) + (lane >> 4) * 8;
            const int ch = kk * 2 + ((lane >> 3) & 1);
            ldmatrix_x4(smem_u32(ktile + (key >> 4) * 2 * PAGE_BYTES + (ch >> 3) * 2048 + (key & 15) * 128 + (((ch & 7) ^ (key & 7)) << 4)), dst[j2]);
          }
        };
        load_k(0, kf[0]);
#pragma unroll
        for (int kk = 0; kk < HD / 16; ++kk) {
          if (kk + 1 < HD / 16) load_k(kk + 1, kf[(kk + 1) & 1]);
#pragma unroll
          for (int j2 = 0; j2 < SK / 16; ++j2) {
            mma_bf16_16816(s[2 * j2], qf[kk], kf[kk & 1][j2][0], kf[kk & 1][j2][1]);
            mma_bf16_16816(s[2 * j2 + 1], qf[kk], kf[kk & 1][j2][2], kf[kk & 1][j2][3]);
          }
        }
      }
      const int k0 = st * SK;
      float tmax[2] = {-INFINITY, -INFINITY};
      if (k0 + SK > n) {
        const uint32_t vis0 = (uint32_t)attn_vis64(anc0, k0, n), vis1 = (uint32_t)attn_vis64(anc1, k0, n);
#pragma unroll
        for (int jj = 0; jj < SK / 8; ++jj) {
#pragma unroll
          for (int e = 0; e < 4; ++e) {
            float v = s[jj][e] * a.scale_log2;
            const int bi = jj * 8 + (lane & 3) * 2 + (e & 1);
            if (!(((e < 2 ? vis0 : vis1) >> bi) & 1u)) v = -INFINITY;
            s[jj][e] = v;
            tmax[e >> 1] = fmaxf(tmax[e >> 1], v);
          }
        }
      } else {
#pragma unroll
        for (int jj = 0; jj < SK / 8; ++jj) {
#pragma unroll
          for (int e = 0; e < 4; ++e) {
            s[jj][e] *= a.scale_log2;
            tmax[e >> 1] = fmaxf(tmax[e >> 1], s[jj][e]);
          }
        }
      }
      float alpha[2], mnew[2];
#pragma unroll
      for (int r = 0; r < 2; ++r) {
        tmax[r] = fmaxf(tmax[r], __shfl_xor_sync(0xffffffffu, tmax[r], 1));
        tmax[r] = fmaxf(tmax[r], __shfl_xor_sync(0xffffffffu, tmax[r], 2));
        mnew[r] = fmaxf(mrow[r], tmax[r]);
        const float base = (mnew[r] == -INFINITY) ? 0.f : mnew[r];
        alpha[r] = exp2f(mrow[r] - base);
        mrow[r] = mnew[r];
        mnew[r] = base;
        lrow[r] *= alpha[r];
      }
#pragma unroll
      for (int d = 0; d < HD / 8; ++d) { o[d][0] *= alpha[0]; o[d][1] *= alpha[0]; o[d][2] *= alpha[1]; o[d][3] *= alpha[1]; }
      uint32_t pf[SK / 16][4];
#pragma unroll
      for (int jj = 0; jj < SK / 8; ++jj) {
        const float p0 = exp2f(s[jj][0] - mnew[0]), p1 = exp2f(s[jj][1] - mnew[0]);
        const float p2 = exp2f(s[jj][2] - mnew[1]), p3 = exp2f(s[jj][3] - mnew[1]);
        lrow[0] += p0 + p1;
        lrow[1] += p2 + p3;
        pf[jj >> 1][(jj & 1) * 2 + 0] = pack_bf16(p0, p1);
        pf[jj >> 1][(jj & 1) * 2 + 1] = pack_bf16(p2, p3);
      }
      {
        constexpr int DG = 4, NG = (SK / 16) * (HD / 16) / DG;
        uint32_t vf[2][DG][4];
        auto load_v = [&](int g, uint32_t (&dst)[DG][4]) {
          const int jv = g / (HD / 16 / DG), d0 = (g % (HD / 16 / DG)) * DG;
#pragma unroll
          for (int dd = 0; dd < DG; ++dd) {
            const int key = jv * 16 + (lane & 7) + ((lane >> 3) & 1) * 8;
            const int ch = (d0 + dd) * 2 + (lane >> 4);
            ldmatrix_x4_trans(smem_u32(vtile + (key >> 4) * 2 * PAGE_BYTES + (ch >> 3) * 2048 + (key & 15) * 128 + (((ch & 7) ^ (key & 7)) << 4)), dst[dd]);
          }
        };
        load_v(0, vf[0]);
#pragma unroll
        for (int g = 0; g < NG; ++g) {
          if (g + 1 < NG) load_v(g + 1, vf[(g + 1) & 1]);
          const int jv = g / (HD / 16 / DG), d0 = (g % (HD / 16 / DG)) * DG;
#pragma unroll
          for (int dd = 0; dd < DG; ++dd) {
            mma_bf16_16816(o[2 * (d0 + dd)], pf[jv], vf[g & 1][dd][0], vf[g & 1][dd][1]);
            mma_bf16_16816(o[2 * (d0 + dd) + 1], pf[jv], vf[g & 1][dd][2], vf[g & 1][dd][3]);
          }
        }
      }
      __syncwarp();                              // every lane has read the buffer
      if (lane == 0) mbar_arrive(&my_empty[bf]);
    }
    if (!ok && rb == 0 && lane == 0) {
      // a wait gave up: copies this phase may still have in flight get a bounded time to land
      for (int i = issued > AS_NB ? issued - AS_NB : 0; i < issued; ++i) mbar_wait(&my_full[i % AS_NB], (i / AS_NB) & 1, a.status, 22);
    }
  }
  ok = __syncthreads_and(ok);                    // all warps are done with the buffers
  if (!ok) return;

#pragma unroll
  for (int r = 0; r < 2; ++r) {
    lrow[r] += __shfl_xor_sync(0xffffffffu, lrow[r], 1);
    lrow[r] += __shfl_xor_sync(0xffffffffu, lrow[r], 2);
  }
  // merge the key phases of a row block through the (now idle) K/V buffers: phases 1.. leave their state,
  // phase 0 adds them in phase order
  float* ex = reinterpret_cast<float*>(kv);
  constexpr int SLOT = (HD / 2 + 4) * 32;       // floats per warp state
  if (kp > 0 && rb < nrb) {
    float* my = ex + (size_t)((kp - 1) * AS_RB + rb) * SLOT;
#pragma unroll
    for (int d = 0; d < HD / 8; ++d)
#pragma unroll
      for (int e = 0; e < 4; ++e) my[(d * 4 + e) * 32 + lane] = o[d][e];
    my[(HD / 2 + 0) * 32 + lane] = mrow[0]; my[(HD / 2 + 1) * 32 + lane] = mrow[1];
    my[(HD / 2 + 2) * 32 + lane] = lrow[0]; my[(HD / 2 + 3) * 32 + lane] = lrow[1];
  }
  __syncthreads();
  if (kp == 0 && rb < nrb) {
#pragma unroll 1
    for (int g2 = 1; g2 < AS_KP; ++g2) {
      const float* th = ex + (size_t)((g2 - 1) * AS_RB + rb) * SLOT;
      float w0[2], w1[2];
#pragma unroll
      for (int r = 0; r < 2; ++r) {
        const float m1 = th[(HD / 2 + r) * 32 + lane], l1 = th[(HD / 2 + 2 + r) * 32 + lane];
        const float mm = fmaxf(mrow[r], m1);
        const float base = (mm == -INFINITY) ? 0.f : mm;
        w0[r] = exp2f(mrow[r] - base);
        w1[r] = exp2f(m1 - base);
        mrow[r] = mm;
        lrow[r] = lrow[r] * w0[r] + l1 * w1[r];
      }
#pragma unroll
      for (int d = 0; d < HD / 8; ++d)
#pragma unroll
        for (int e = 0; e < 4; ++e) o[d][e] = o[d][e] * w0[e >> 1] + th[(d * 4 + e) * 32 + lane] * w1[e >> 1];
    }
    if (nsplit == 1) {
#pragma unroll
      for (int r = 0; r < 2; ++r) {
        const int i = r ? i1 : i0;
        if (i >= cnt) continue;
        const float inv = 1.f / lrow[r];
        bf16* po = a.out + ((size_t)b * R + i) * H * HD + h * HD;
#pragma unroll
        for (int d = 0; d < HD / 8; ++d)
          *reinterpret_cast<uint32_t*>(po + d * 8 + (lane & 3) * 2) = pack_bf16(o[d][2 * r] * inv, o[d][2 * r + 1] * inv);
      }
    } else {
#pragma unroll
      for (int r = 0; r < 2; ++r) {
        const int i = r ? i1 : i0;
        if (i >= cnt) continue;
        const size_t m = (size_t)b * R + i;
        float* po = a.part_o + ((size_t)sp * M + m) * H * HD + h * HD;
#pragma unroll
        for (int d = 0; d < HD / 8; ++d)
          *reinterpret_cast<float2*>(po + d * 8 + (lane & 3) * 2) = make_float2(o[d][2 * r], o[d][2 * r + 1]);
        if ((lane & 3) == 0) {
          float* ml = a.part_ml + (((size_t)sp * M + m) * H + h) * 2;
          ml[0] = mrow[r];
          ml[1] = lrow[r];
        }
      }
    }
  }
  if (nsplit == 1) return;
  // the CTA of this (sequence, row half, head) that arrives last merges the splits
  __shared__ int last_s;
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
    if (il < AS_RB * 16 && i < cnt) {
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
