// Tree-masked decode attention over the paged bf16 KV cache (verification forward of
// Sec. III-B: every tree node attends to all committed positions and to its own ancestors
// in the tree). One CTA per (query head, KV split, sequence); warp w owns query rows
// [16w, 16w+16). KV tiles of 64 keys are brought in page by page with bulk asynchronous
// copies that complete on an mbarrier (the cache's in-page chunk swizzle makes the landed
// tile conflict-free for ldmatrix); QK^T and PV run on mma.sync m16n8k16 with a warp-level
// online softmax; the tree mask is a 128-bit ancestor set per row applied only to keys at or
// beyond the committed length. Each split leaves (max, sum, unnormalised output) and a
// small combine kernel merges the splits.
#pragma once
#include "common.cuh"
#include "kernels_simple.cuh"

namespace spec {

__device__ __forceinline__ void ldmatrix_x4(uint32_t addr, uint32_t (&r)[4]) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];"
               : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(addr));
}
__device__ __forceinline__ void ldmatrix_x4_trans(uint32_t addr, uint32_t (&r)[4]) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0,%1,%2,%3}, [%4];"
               : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(addr));
}
__device__ __forceinline__ void mma_bf16_16816(float (&c)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1) {
  asm volatile(
      "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
      : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
      : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}
__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi) {
  __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
  return *reinterpret_cast<uint32_t*>(&v);
}

struct AttnTcArgs {
  const bf16* q;        // [M][H*HD]
  float* part_o;        // [nsplit][M][H*HD] unnormalised
  float* part_ml;       // [nsplit][M][H][2] (running max in log2 units, sum)
  const bf16* pool;
  KVGeom g;
  const int* page_table;
  Rows rows;
  int layer, H, nsplit;
  float scale_log2;     // log2(e) / sqrt(head_dim)
  int* status;
};

template <int HD, int NW>
__global__ void __launch_bounds__(NW * 32)
attention_tc(const AttnTcArgs a, unsigned long long* tr) {
  KTrace kt(tr);
  constexpr int KT = 64;                      // keys per tile
  constexpr int ROWB = HD * 2;                // bytes per row
  constexpr int TILE_BYTES = KT * ROWB;
  constexpr int PAGE_BYTES = 16 * ROWB;
  extern __shared__ __align__(128) uint8_t smem[];
  uint8_t* qs = smem;                                       // [NW*16][HD]
  uint8_t* ks = qs + NW * 16 * ROWB;                        // [2][KT][HD]
  uint8_t* vs = ks + 2 * TILE_BYTES;                        // [2][KT][HD]
  uint64_t* full = reinterpret_cast<uint64_t*>(vs + 2 * TILE_BYTES);   // [2]

  pdl_launch_dependents();
  pdl_wait();
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int h = blockIdx.x, sp = blockIdx.y, b = blockIdx.z;
  const int R = a.rows.R, cnt = a.rows.cnt[b], n = a.rows.n[b];
  const int S = n + cnt;
  const int H = a.H, kvh = h / (H / a.g.n_kv_heads);
  const int M = a.rows.B * R;
  if (cnt == 0) return;
  const int total_tiles = (S + KT - 1) / KT;
  const int tps = (total_tiles + a.nsplit - 1) / a.nsplit;
  const int t0 = sp * tps, t1 = min(total_tiles, t0 + tps);
  const int* pt = a.page_table + b * a.g.pages_per_seq;

  const int i0 = warp * 16 + (lane >> 2), i1 = i0 + 8;      // this thread's two query rows
  if (t0 >= t1) {
    // empty split: publish a neutral partial for the valid rows
    if ((lane & 3) == 0) {
      if (i0 < cnt) { float* ml = a.part_ml + (((size_t)sp * M + b * R + i0) * H + h) * 2; ml[0] = -INFINITY; ml[1] = 0.f; }
      if (i1 < cnt) { float* ml = a.part_ml + (((size_t)sp * M + b * R + i1) * H + h) * 2; ml[0] = -INFINITY; ml[1] = 0.f; }
    }
    return;
  }

  if (threadIdx.x == 0) { mbar_init(&full[0], 1); mbar_init(&full[1], 1); mbar_fence_init(); }
  // stage Q (rows beyond cnt are zero) with the same chunk swizzle as the cache
  for (int c = threadIdx.x; c < NW * 16 * (HD / 8); c += NW * 32) {
    int r = c / (HD / 8), ch = c % (HD / 8);
    uint4 v = make_uint4(0, 0, 0, 0);
    if (r < cnt) v = *reinterpret_cast<const uint4*>(a.q + (size_t)(b * R + r) * H * HD + h * HD + ch * 8);
    *reinterpret_cast<uint4*>(qs + r * ROWB + ((ch ^ (r & 7)) << 4)) = v;
  }
  __syncthreads();

  auto issue = [&](int tile, int buf) {
    mbar_expect_tx(&full[buf], 2 * TILE_BYTES);
    for (int pg = 0; pg < KT / 16; ++pg) {
      int page = pt[tile * (KT / 16) + pg];
      bulk_load_1d(ks + buf * TILE_BYTES + pg * PAGE_BYTES, a.pool + a.g.block_offset(page, a.layer, 0, kvh),
                   PAGE_BYTES, &full[buf]);
      bulk_load_1d(vs + buf * TILE_BYTES + pg * PAGE_BYTES, a.pool + a.g.block_offset(page, a.layer, 1, kvh),
                   PAGE_BYTES, &full[buf]);
    }
  };
  if (threadIdx.x == 0) issue(t0, 0);

  // Q fragments stay in registers
  uint32_t qf[HD / 16][4];
  {
    int row = warp * 16 + (lane & 7) + ((lane >> 3) & 1) * 8;
#pragma unroll
    for (int kk = 0; kk < HD / 16; ++kk) {
      int ch = kk * 2 + (lane >> 4);
      ldmatrix_x4(smem_u32(qs + row * ROWB + ((ch ^ (row & 7)) << 4)), qf[kk]);
    }
  }
  uint32_t anc0[4] = {0, 0, 0, 0}, anc1[4] = {0, 0, 0, 0};
  if (i0 < cnt) for (int w = 0; w < 4; ++w) anc0[w] = a.rows.anc[i0 * 4 + w];
  if (i1 < cnt) for (int w = 0; w < 4; ++w) anc1[w] = a.rows.anc[i1 * 4 + w];

  float o[HD / 8][4];
#pragma unroll
  for (int d = 0; d < HD / 8; ++d) o[d][0] = o[d][1] = o[d][2] = o[d][3] = 0.f;
  float mrow[2] = {-INFINITY, -INFINITY}, lrow[2] = {0.f, 0.f};

  bool ok = true;
  for (int t = t0; t < t1; ++t) {
    const int buf = (t - t0) & 1;
    if (threadIdx.x == 0 && t + 1 < t1) issue(t + 1, buf ^ 1);
    if (!mbar_wait(&full[buf], ((t - t0) >> 1) & 1, a.status, 20)) { ok = false; }
    ok = __syncthreads_and(ok);
    if (!ok) break;
    const uint8_t* kt = ks + buf * TILE_BYTES;
    const uint8_t* vt = vs + buf * TILE_BYTES;
    float s[KT / 8][4];
#pragma unroll
    for (int j = 0; j < KT / 8; ++j) s[j][0] = s[j][1] = s[j][2] = s[j][3] = 0.f;
#pragma unroll
    for (int kk = 0; kk < HD / 16; ++kk) {
#pragma unroll
      for (int j2 = 0; j2 < KT / 16; ++j2) {
        int key = j2 * 16 + (lane & 7) + (lane >> 4) * 8;
        int ch = kk * 2 + ((lane >> 3) & 1);
        uint32_t bfr[4];
        ldmatrix_x4(smem_u32(kt + key * ROWB + ((ch ^ (key & 7)) << 4)), bfr);
        mma_bf16_16816(s[2 * j2], qf[kk], bfr[0], bfr[1]);
        mma_bf16_16816(s[2 * j2 + 1], qf[kk], bfr[2], bfr[3]);
      }
    }
    // mask + online softmax (log2 domain)
    const int k0 = t * KT;
    const bool need_mask = (k0 + KT > n);
    float tmax[2] = {-INFINITY, -INFINITY};
#pragma unroll
    for (int j = 0; j < KT / 8; ++j) {
#pragma unroll
      for (int e = 0; e < 4; ++e) {
        float v = s[j][e] * a.scale_log2;
        if (need_mask) {
          int key = k0 + j * 8 + (lane & 3) * 2 + (e & 1);
          bool vis = key < n;
          if (!vis && key < S) {
            int u = key - n;
            uint32_t w = (e < 2) ? anc0[u >> 5] : anc1[u >> 5];
            vis = (w >> (u & 31)) & 1u;
          }
          if (!vis) v = -INFINITY;
        }
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
#pragma unroll
    for (int j = 0; j < KT / 16; ++j) {
#pragma unroll
      for (int d2 = 0; d2 < HD / 16; ++d2) {
        int key = j * 16 + (lane & 7) + ((lane >> 3) & 1) * 8;
        int ch = d2 * 2 + (lane >> 4);
        uint32_t bfr[4];
        ldmatrix_x4_trans(smem_u32(vt + key * ROWB + ((ch ^ (key & 7)) << 4)), bfr);
        mma_bf16_16816(o[2 * d2], pf[j], bfr[0], bfr[1]);
        mma_bf16_16816(o[2 * d2 + 1], pf[j], bfr[2], bfr[3]);
      }
    }
    __syncthreads();   // tile consumed: its buffer may be refilled
  }

#pragma unroll
  for (int r = 0; r < 2; ++r) {
    lrow[r] += __shfl_xor_sync(0xffffffffu, lrow[r], 1);
    lrow[r] += __shfl_xor_sync(0xffffffffu, lrow[r], 2);
  }
  if (ok) {
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
}

// Merges the KV splits: out[m][h*HD + d] = bf16( sum_s w_s O_s / sum_s w_s l_s ),
// w_s = 2^(m_s - max_s m_s). One thread per (row, head, 4 dims).
__global__ void attention_combine(const float* __restrict__ part_o, const float* __restrict__ part_ml, int nsplit,
                                  Rows rows, int H, int HD, bf16* __restrict__ out, unsigned long long* tr) {
  KTrace kt(tr);
  pdl_launch_dependents();
  pdl_wait();
  if (threadIdx.x == 0) trace_mark_min(tr, 2);
  int M = rows.B * rows.R;
  size_t idx = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
  size_t per_row = (size_t)H * HD / 4;
  if (idx >= (size_t)M * per_row) return;
  int m = (int)(idx / per_row);
  int rem = (int)(idx % per_row);
  int h = rem / (HD / 4), d = (rem % (HD / 4)) * 4;
  if (m % rows.R >= rows.cnt[m / rows.R]) return;
  float mx = -INFINITY;
  for (int s = 0; s < nsplit; ++s) mx = fmaxf(mx, part_ml[(((size_t)s * M + m) * H + h) * 2]);
  float L = 0.f, acc[4] = {0.f, 0.f, 0.f, 0.f};
  for (int s = 0; s < nsplit; ++s) {
    const float* ml = part_ml + (((size_t)s * M + m) * H + h) * 2;
    if (ml[0] == -INFINITY) continue;
    float w = exp2f(ml[0] - mx);
    L += w * ml[1];
    float4 v = *reinterpret_cast<const float4*>(part_o + ((size_t)s * M + m) * H * HD + h * HD + d);
    acc[0] += w * v.x; acc[1] += w * v.y; acc[2] += w * v.z; acc[3] += w * v.w;
  }
  float inv = 1.f / L;
  bf16* o = out + (size_t)m * H * HD + h * HD + d;
  o[0] = __float2bfloat16_rn(acc[0] * inv);
  o[1] = __float2bfloat16_rn(acc[1] * inv);
  o[2] = __float2bfloat16_rn(acc[2] * inv);
  o[3] = __float2bfloat16_rn(acc[3] * inv);
}

}  // namespace spec
