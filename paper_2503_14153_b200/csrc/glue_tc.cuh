// Glue kernels of the bf16 verification forward: they consume the float32 partial sums the
// weight-streaming GEMM leaves (adding a tile's slots in CTA order), apply the element-wise
// step of the layer (residual + RMSNorm, RoPE + cache store, SwiGLU) and write the bf16
// operand of the next GEMM. All are vectorised (16-byte accesses), take part in programmatic
// dependent launch (trigger at entry, wait before the first dependent access) and keep the
// rounding points of the reference path: float32 until the operand is rounded to bf16.
#pragma once
#include "common.cuh"
#include "gemm_stream.cuh"
#include "kernels_simple.cuh"

namespace spec {

// Partial sums of one GEMM launch: part[slot][m][ld], padded column space (tile nt = columns
// [128 nt, 128 nt + 128)).
struct PartView {
  const float* part;
  size_t slot_stride;
  int ld;
  SegMap seg;                  // how the GEMM dealt its units: gives the slots of a tile
  int mt_shift;                // log2 of the activation rows per tile
  int single;                  // 1: every tile is one finished slot (the 128 x 256-tile GEMM): read it directly
};

constexpr int PV_UNROLL = 12;

// Sum over the slots of the tile that holds padded columns [colp, colp+4) of row m.
__device__ __forceinline__ float4 part_sum4(const PartView& pv, int m, int colp) {
  const int ns = pv.seg.nseg((colp >> 7) * pv.seg.m_tiles + (m >> pv.mt_shift));
  const float* src = pv.part + (size_t)m * pv.ld + colp;
  float4 v[PV_UNROLL];
#pragma unroll
  for (int s = 0; s < PV_UNROLL; ++s)
    v[s] = (s < ns) ? __ldcg(reinterpret_cast<const float4*>(src + (size_t)s * pv.slot_stride)) : make_float4(0.f, 0.f, 0.f, 0.f);
  float4 a = v[0];
#pragma unroll
  for (int s = 1; s < PV_UNROLL; ++s)
    if (s < ns) { a.x += v[s].x; a.y += v[s].y; a.z += v[s].z; a.w += v[s].w; }
  for (int s = PV_UNROLL; s < ns; ++s) {
    float4 w = __ldcg(reinterpret_cast<const float4*>(src + (size_t)s * pv.slot_stride));
    a.x += w.x; a.y += w.y; a.z += w.z; a.w += w.w;
  }
  return a;
}

// The same for a view of finished sums (pv.single).
__device__ __forceinline__ float4 part_one4(const PartView& pv, int m, int colp) {
  return __ldcg(reinterpret_cast<const float4*>(pv.part + (size_t)m * pv.ld + colp));
}

__device__ __forceinline__ uint2 pack4_bf16(float a, float b, float c, float d) {
  __nv_bfloat162 lo = __floats2bfloat162_rn(a, b), hi = __floats2bfloat162_rn(c, d);
  uint2 r;
  r.x = *reinterpret_cast<uint32_t*>(&lo);
  r.y = *reinterpret_cast<uint32_t*>(&hi);
  return r;
}

// ------------------------------------------------------------------ residual + RMSNorm
// x[m] += sum of the partial slots (when pv.part != nullptr); u[m] = bf16(x / rms(x) * g);
// optionally the unrounded normed row goes to hid. A cluster of NORM_CLUSTER CTAs (on
// neighbouring SMs) shares a row, each with its own slice of the columns, so that one SM does
// not have to pull a whole row's partial sums through its load queues; the slices' sums of
// squares are exchanged through distributed shared memory and added in rank order. Every
// thread issues all its loads at once (one trip to L2) and keeps its values in registers; the
// gains do not depend on the previous kernel and are fetched before the dependency wait.
// d % 4 == 0; grid (rows, NORM_CLUSTER).
constexpr int NORM_THREADS = 512;
constexpr int NORM_CLUSTER = 2;
constexpr int NORM_CACHE = 2;   // float4 values a thread keeps between the two passes

__global__ void __cluster_dims__(1, NORM_CLUSTER, 1) __launch_bounds__(NORM_THREADS)
norm_reduce_tc(float* __restrict__ x, const PartView pv, const float* __restrict__ gain, float eps,
               bf16* __restrict__ u, float* __restrict__ hid, int d, unsigned long long* tr) {
  KTrace kt(tr);
  pdl_launch_dependents();
  const int m = blockIdx.x, rank = blockIdx.y;
  float* xr = x + (size_t)m * d;
  const int n4 = d >> 2;
  const int per = (n4 + NORM_CLUSTER - 1) / NORM_CLUSTER;
  const int c_lo = rank * per, c_hi = min(n4, c_lo + per);
  float4 gk[NORM_CACHE];
#pragma unroll
  for (int k = 0; k < NORM_CACHE; ++k) {
    const int c4 = c_lo + threadIdx.x + k * NORM_THREADS;
    gk[k] = c4 < c_hi ? *reinterpret_cast<const float4*>(gain + c4 * 4) : make_float4(0.f, 0.f, 0.f, 0.f);
  }
  pdl_wait();
  if (threadIdx.x == 0) trace_mark_min(tr, 2);
  float4 keep[NORM_CACHE];
  float ss = 0.f;
#pragma unroll
  for (int k = 0; k < NORM_CACHE; ++k) {
    const int c4 = c_lo + threadIdx.x + k * NORM_THREADS;
    if (c4 < c_hi) {
      float4 v = *reinterpret_cast<const float4*>(xr + c4 * 4);
      if (pv.part) {
        const float4 a = part_sum4(pv, m, c4 * 4);
        v.x += a.x; v.y += a.y; v.z += a.z; v.w += a.w;
        *reinterpret_cast<float4*>(xr + c4 * 4) = v;
      }
      keep[k] = v;
      ss += v.x * v.x + v.y * v.y + v.z * v.z + v.w * v.w;
    }
  }
  for (int c4 = c_lo + threadIdx.x + NORM_CACHE * NORM_THREADS; c4 < c_hi; c4 += NORM_THREADS) {
    float4 v = *reinterpret_cast<const float4*>(xr + c4 * 4);
    if (pv.part) {
      const float4 a = part_sum4(pv, m, c4 * 4);
      v.x += a.x; v.y += a.y; v.z += a.z; v.w += a.w;
      *reinterpret_cast<float4*>(xr + c4 * 4) = v;
    }
    ss += v.x * v.x + v.y * v.y + v.z * v.z + v.w * v.w;
  }
  __shared__ float red[32];
  __shared__ float slice_ss;
  ss = warp_sum(ss);
  if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = ss;
  __syncthreads();
  if (threadIdx.x == 0) {
    float t = 0.f;
#pragma unroll
    for (int w = 0; w < (NORM_THREADS >> 5); ++w) t += red[w];
    slice_ss = t;
  }
  // exchange the slices' sums through distributed shared memory (cluster barrier: release / acquire)
  asm volatile("barrier.cluster.arrive.release.aligned;\n\tbarrier.cluster.wait.acquire.aligned;" ::: "memory");
  float tot = 0.f;
#pragma unroll
  for (int r = 0; r < NORM_CLUSTER; ++r) {
    uint32_t remote;
    asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(remote) : "r"(smem_u32(&slice_ss)), "r"(r));
    float v;
    asm volatile("ld.shared::cluster.f32 %0, [%1];" : "=f"(v) : "r"(remote) : "memory");
    tot += v;                                           // rank order: the same sum in every CTA
  }
  // nobody may leave (and give up its shared memory) before every CTA has read it
  asm volatile("barrier.cluster.arrive.release.aligned;\n\tbarrier.cluster.wait.acquire.aligned;" ::: "memory");
  const float inv = rsqrtf(tot / (float)d + eps);
  auto emit = [&](int c4, const float4& v, const float4& g) {
    const float4 o = make_float4(v.x * inv * g.x, v.y * inv * g.y, v.z * inv * g.z, v.w * inv * g.w);
    *reinterpret_cast<uint2*>(u + (size_t)m * d + c4 * 4) = pack4_bf16(o.x, o.y, o.z, o.w);
    if (hid) *reinterpret_cast<float4*>(hid + (size_t)m * d + c4 * 4) = o;
  };
#pragma unroll
  for (int k = 0; k < NORM_CACHE; ++k) {
    const int c4 = c_lo + threadIdx.x + k * NORM_THREADS;
    if (c4 < c_hi) emit(c4, keep[k], gk[k]);
  }
  for (int c4 = c_lo + threadIdx.x + NORM_CACHE * NORM_THREADS; c4 < c_hi; c4 += NORM_THREADS)
    emit(c4, *reinterpret_cast<const float4*>(xr + c4 * 4), *reinterpret_cast<const float4*>(gain + c4 * 4));
}

// RMSNorm of rows whose sums of squares already exist in pieces (the residual cluster epilogue leaves
// ss_part[m][n_ss], the sum of squares of every 16-column piece of row m): u[m] = bf16(x / rms(x) * g).
// gridDim.y plain CTAs share a row, each adding all the row's pieces itself in a fixed order (the same sum in
// every CTA), so nothing is exchanged between CTAs. One trip to L2 per thread.
__global__ void __launch_bounds__(NORM_THREADS)
norm_scaled_tc(const float* __restrict__ x, const float* __restrict__ ss_part, int n_ss, const float* __restrict__ gain,
               float eps, bf16* __restrict__ u, float* __restrict__ hid, int d, unsigned long long* tr) {
  KTrace kt(tr);
  pdl_launch_dependents();
  const int m = blockIdx.x;
  const float* xr = x + (size_t)m * d;
  const int n4 = d >> 2;
  const int per = (n4 + (int)gridDim.y - 1) / (int)gridDim.y;
  const int c_lo = blockIdx.y * per, c_hi = min(n4, c_lo + per);
  float4 gk[NORM_CACHE];
#pragma unroll
  for (int k = 0; k < NORM_CACHE; ++k) {
    const int c4 = c_lo + threadIdx.x + k * NORM_THREADS;
    gk[k] = c4 < c_hi ? *reinterpret_cast<const float4*>(gain + c4 * 4) : make_float4(0.f, 0.f, 0.f, 0.f);
  }
  pdl_wait();
  if (threadIdx.x == 0) trace_mark_min(tr, 2);
  float4 keep[NORM_CACHE];
#pragma unroll
  for (int k = 0; k < NORM_CACHE; ++k) {
    const int c4 = c_lo + threadIdx.x + k * NORM_THREADS;
    keep[k] = c4 < c_hi ? *reinterpret_cast<const float4*>(xr + c4 * 4) : make_float4(0.f, 0.f, 0.f, 0.f);
  }
  float ss = 0.f;
  for (int i = threadIdx.x; i < n_ss; i += NORM_THREADS) ss += __ldcg(ss_part + (size_t)m * n_ss + i);
  __shared__ float red[NORM_THREADS / 32];
  ss = warp_sum(ss);
  if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = ss;
  __syncthreads();
  float tot = 0.f;
#pragma unroll
  for (int w = 0; w < NORM_THREADS / 32; ++w) tot += red[w];
  const float inv = rsqrtf(tot / (float)d + eps);
  auto emit = [&](int c4, const float4& v, const float4& g) {
    const float4 o = make_float4(v.x * inv * g.x, v.y * inv * g.y, v.z * inv * g.z, v.w * inv * g.w);
    *reinterpret_cast<uint2*>(u + (size_t)m * d + c4 * 4) = pack4_bf16(o.x, o.y, o.z, o.w);
    if (hid) *reinterpret_cast<float4*>(hid + (size_t)m * d + c4 * 4) = o;
  };
#pragma unroll
  for (int k = 0; k < NORM_CACHE; ++k) {
    const int c4 = c_lo + threadIdx.x + k * NORM_THREADS;
    if (c4 < c_hi) emit(c4, keep[k], gk[k]);
  }
  for (int c4 = c_lo + threadIdx.x + NORM_CACHE * NORM_THREADS; c4 < c_hi; c4 += NORM_THREADS)
    emit(c4, *reinterpret_cast<const float4*>(xr + c4 * 4), *reinterpret_cast<const float4*>(gain + c4 * 4));
}

// The same operation for passes of many rows (batched verification, prompt processing): one CTA of
// NORMW_THREADS per row, no cluster. With hundreds of rows the kernel is bound by bandwidth, not by the
// latency of one row, so what counts is loads in flight: a thread fetches all its pieces of x and of the
// partial sums before it uses the first (NORMW_CACHE float4 each; rows longer than that loop).
constexpr int NORMW_THREADS = 256;
constexpr int NORMW_CACHE = 4;

__global__ void __launch_bounds__(NORMW_THREADS)
norm_rows_wide(float* __restrict__ x, const PartView pv, const float* __restrict__ gain, float eps,
               bf16* __restrict__ u, float* __restrict__ hid, int d, unsigned long long* tr) {
  KTrace kt(tr);
  pdl_launch_dependents();
  const int m = blockIdx.x;
  float* xr = x + (size_t)m * d;
  const int n4 = d >> 2;
  float4 gk[NORMW_CACHE];
#pragma unroll
  for (int k = 0; k < NORMW_CACHE; ++k) {
    const int c4 = threadIdx.x + k * NORMW_THREADS;
    gk[k] = c4 < n4 ? *reinterpret_cast<const float4*>(gain + c4 * 4) : make_float4(0.f, 0.f, 0.f, 0.f);
  }
  pdl_wait();
  if (threadIdx.x == 0) trace_mark_min(tr, 2);
  auto part4 = [&](int c4) { return pv.single ? part_one4(pv, m, c4 * 4) : part_sum4(pv, m, c4 * 4); };
  float4 keep[NORMW_CACHE], add[NORMW_CACHE];
#pragma unroll
  for (int k = 0; k < NORMW_CACHE; ++k) {
    const int c4 = threadIdx.x + k * NORMW_THREADS;
    keep[k] = add[k] = make_float4(0.f, 0.f, 0.f, 0.f);
    if (c4 < n4) {
      keep[k] = *reinterpret_cast<const float4*>(xr + c4 * 4);
      if (pv.part) add[k] = part4(c4);
    }
  }
  float ss = 0.f;
#pragma unroll
  for (int k = 0; k < NORMW_CACHE; ++k) {
    const int c4 = threadIdx.x + k * NORMW_THREADS;
    if (c4 < n4) {
      float4& v = keep[k];
      if (pv.part) {
        v.x += add[k].x; v.y += add[k].y; v.z += add[k].z; v.w += add[k].w;
        *reinterpret_cast<float4*>(xr + c4 * 4) = v;
      }
      ss += v.x * v.x + v.y * v.y + v.z * v.z + v.w * v.w;
    }
  }
  for (int c4 = threadIdx.x + NORMW_CACHE * NORMW_THREADS; c4 < n4; c4 += NORMW_THREADS) {
    float4 v = *reinterpret_cast<const float4*>(xr + c4 * 4);
    if (pv.part) {
      const float4 a = part4(c4);
      v.x += a.x; v.y += a.y; v.z += a.z; v.w += a.w;
      *reinterpret_cast<float4*>(xr + c4 * 4) = v;
    }
    ss += v.x * v.x + v.y * v.y + v.z * v.z + v.w * v.w;
  }
  __shared__ float red[NORMW_THREADS / 32];
  __shared__ float row_ss;
  ss = warp_sum(ss);
  if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = ss;
  __syncthreads();
  if (threadIdx.x == 0) {
    float t = 0.f;
#pragma unroll
    for (int w = 0; w < NORMW_THREADS / 32; ++w) t += red[w];
    row_ss = t;
  }
  __syncthreads();
  const float inv = rsqrtf(row_ss / (float)d + eps);
  auto emit = [&](int c4, const float4& v, const float4& g) {
    const float4 o = make_float4(v.x * inv * g.x, v.y * inv * g.y, v.z * inv * g.z, v.w * inv * g.w);
    *reinterpret_cast<uint2*>(u + (size_t)m * d + c4 * 4) = pack4_bf16(o.x, o.y, o.z, o.w);
    if (hid) *reinterpret_cast<float4*>(hid + (size_t)m * d + c4 * 4) = o;
  };
#pragma unroll
  for (int k = 0; k < NORMW_CACHE; ++k) {
    const int c4 = threadIdx.x + k * NORMW_THREADS;
    if (c4 < n4) emit(c4, keep[k], gk[k]);
  }
  for (int c4 = threadIdx.x + NORMW_CACHE * NORMW_THREADS; c4 < n4; c4 += NORMW_THREADS)
    emit(c4, *reinterpret_cast<const float4*>(xr + c4 * 4), *reinterpret_cast<const float4*>(gain + c4 * 4));
}

// ------------------------------------------------------------------ RoPE + cache store
// Sums the QKV partial slots, rotates q and k (rotate-half pairs (e, e + D/2), table
// cs[pos][e] = (cos, sin)), writes q as bf16 [M][H*D] and k, v as bf16 into the paged cache at
// the row's slot. qp0 / kp0 / vp0: first padded column of the q / k / v matrix in the partials.
// gridDim.y CTAs share a row; D % 8 == 0.
__global__ void __launch_bounds__(256)
rope_store_tc(const PartView pv, int qp0, int kp0, int vp0, Rows rows, const float2* __restrict__ cs,
              bf16* __restrict__ q, bf16* __restrict__ pool, KVGeom g, const int* __restrict__ page_table,
              int layer, int H, unsigned long long* tr) {
  KTrace kt(tr);
  pdl_launch_dependents();
  pdl_wait();
  if (threadIdx.x == 0) trace_mark_min(tr, 2);
  const int m = blockIdx.x, b = m / rows.R, i = m % rows.R;
  const int D = g.head_dim, half = D >> 1, Hkv = g.n_kv_heads;
  const int q4 = half >> 2;                       // float4 groups per half head
  const int n_rot = (H + Hkv) * q4, n_v = Hkv * (D >> 2);
  const int tid = blockIdx.y * blockDim.x + threadIdx.x, nthr = gridDim.y * blockDim.x;
  // row bookkeeping and partial sums are independent loads: issue them together
  const int cnt = rows.cnt[b], pos = rows.pos[m], slot = rows.slot[m];
  // item -> first padded column of its group of four (rotated items also take the group half a head further)
  auto item_col = [&](int it) {
    if (it < n_rot) {
      const int head = it / q4, e = (it % q4) * 4;
      return (head < H ? qp0 + head * D : kp0 + (head - H) * D) + e;
    }
    const int iv = it - n_rot;
    return vp0 + (iv / (D >> 2)) * D + (iv % (D >> 2)) * 4;
  };
  auto finish = [&](int it, const float4& a, const float4& c) {
    if (i >= cnt) return;
    if (it < n_rot) {
      const int head = it / q4, e = (it % q4) * 4;
      const float4 t01 = *reinterpret_cast<const float4*>(cs + (size_t)pos * half + e);
      const float4 t23 = *reinterpret_cast<const float4*>(cs + (size_t)pos * half + e + 2);
      const uint2 lo = pack4_bf16(a.x * t01.x - c.x * t01.y, a.y * t01.z - c.y * t01.w, a.z * t23.x - c.z * t23.y, a.w * t23.z - c.w * t23.w);
      const uint2 hi = pack4_bf16(c.x * t01.x + a.x * t01.y, c.y * t01.z + a.y * t01.w, c.z * t23.x + a.z * t23.y, c.w * t23.z + a.w * t23.w);
      if (head < H) {
        bf16* dst = q + (size_t)m * H * D + head * D + e;
        *reinterpret_cast<uint2*>(dst) = lo;
        *reinterpret_cast<uint2*>(dst + half) = hi;
      } else {
        const int page = page_table[b * g.pages_per_seq + slot / g.page_size], prow = slot % g.page_size;
        bf16* dst = pool + g.block_offset(page, layer, 0, head - H) + (size_t)prow * D;
        *reinterpret_cast<uint2*>(dst + kv_elem<bf16>(prow, e, D, g.page_size)) = lo;
        *reinterpret_cast<uint2*>(dst + kv_elem<bf16>(prow, e + half, D, g.page_size)) = hi;
      }
    } else {
      const int iv = it - n_rot;
      const int kh = iv / (D >> 2), e = (iv % (D >> 2)) * 4;
      const int page = page_table[b * g.pages_per_seq + slot / g.page_size], prow = slot % g.page_size;
      bf16* dst = pool + g.block_offset(page, layer, 1, kh) + (size_t)prow * D;
      *reinterpret_cast<uint2*>(dst + kv_elem<bf16>(prow, e, D, g.page_size)) = pack4_bf16(a.x, a.y, a.z, a.w);
    }
  };
  if (pv.single) {
    // passes of many rows (finished sums): a thread keeps the loads of four items in flight
    constexpr int U = 4;
    for (int it0 = tid; it0 < n_rot + n_v; it0 += U * nthr) {
      float4 a[U], c[U];
#pragma unroll
      for (int k = 0; k < U; ++k) {
        const int it = it0 + k * nthr;
        a[k] = c[k] = make_float4(0.f, 0.f, 0.f, 0.f);
        if (it < n_rot + n_v) {
          const int colp = item_col(it);
          a[k] = part_one4(pv, m, colp);
          if (it < n_rot) c[k] = part_one4(pv, m, colp + half);
        }
      }
#pragma unroll
      for (int k = 0; k < U; ++k) {
        const int it = it0 + k * nthr;
        if (it < n_rot + n_v) finish(it, a[k], c[k]);
      }
    }
    return;
  }
  for (int it = tid; it < n_rot + n_v; it += nthr) {
    const int colp = item_col(it);
    const float4 a = part_sum4(pv, m, colp);
    const float4 c = it < n_rot ? part_sum4(pv, m, colp + half) : make_float4(0.f, 0.f, 0.f, 0.f);
    finish(it, a, c);
  }
}

// ------------------------------------------------------------------ SwiGLU
// act[m][f] = bf16(SiLU(gate) * up), gate / up = sums of the partial slots of the gate and up
// matrices (padded columns gp0 + f and up0 + f). F % 4 == 0.
__global__ void __launch_bounds__(256)
swiglu_reduce_tc(const PartView pv, int gp0, int up0, bf16* __restrict__ act, int M, int F, unsigned long long* tr) {
  KTrace kt(tr);
  pdl_launch_dependents();
  pdl_wait();
  if (threadIdx.x == 0) trace_mark_min(tr, 2);
  const int f4 = F >> 2;
  const size_t total = (size_t)M * f4;
  if (pv.single) {
    // passes of many rows (finished sums, hundreds of MB): bandwidth-bound, so a thread keeps the loads of four
    // items in flight
    constexpr int U = 4;
    const size_t stride = (size_t)gridDim.x * blockDim.x;
    for (size_t idx0 = (size_t)blockIdx.x * blockDim.x + threadIdx.x; idx0 < total; idx0 += U * stride) {
      float4 gt[U], up[U];
#pragma unroll
      for (int k = 0; k < U; ++k) {
        const size_t idx = idx0 + k * stride;
        if (idx < total) {
          const int m = (int)(idx / f4), f = (int)(idx % f4) * 4;
          gt[k] = part_one4(pv, m, gp0 + f);
          up[k] = part_one4(pv, m, up0 + f);
        }
      }
#pragma unroll
      for (int k = 0; k < U; ++k) {
        const size_t idx = idx0 + k * stride;
        if (idx < total) {
          const int m = (int)(idx / f4), f = (int)(idx % f4) * 4;
          *reinterpret_cast<uint2*>(act + (size_t)m * F + f) =
              pack4_bf16(silu_f(gt[k].x) * up[k].x, silu_f(gt[k].y) * up[k].y, silu_f(gt[k].z) * up[k].z, silu_f(gt[k].w) * up[k].w);
        }
      }
    }
    return;
  }
  for (size_t idx = (size_t)blockIdx.x * blockDim.x + threadIdx.x; idx < total; idx += (size_t)gridDim.x * blockDim.x) {
    const int m = (int)(idx / f4), f = (int)(idx % f4) * 4;
    const float4 gt = part_sum4(pv, m, gp0 + f), up = part_sum4(pv, m, up0 + f);
    *reinterpret_cast<uint2*>(act + (size_t)m * F + f) =
        pack4_bf16(silu_f(gt.x) * up.x, silu_f(gt.y) * up.y, silu_f(gt.z) * up.z, silu_f(gt.w) * up.w);
  }
}

// ------------------------------------------------------------------ extra decoding heads
// r[b*K + k0 + kk][i] = bf16(h + SiLU(z + bias_k[i])), z = sum of the partial slots of head
// matrix kk of this launch group (padded columns kk * dpad + i), h = hq_last[b][i] (already
// bf16). grid (B * nk, CTAs per row).
__global__ void __launch_bounds__(256)
medusa_act_tc(const PartView pv, int dpad, const bf16* __restrict__ hq_last, const bf16* const* __restrict__ bias,
              bf16* __restrict__ r, int K, int k0, int nk, int d, unsigned long long* tr) {
  KTrace kt(tr);
  pdl_launch_dependents();
  pdl_wait();
  if (threadIdx.x == 0) trace_mark_min(tr, 2);
  const int b = blockIdx.x / nk, kk = blockIdx.x % nk, k = k0 + kk;
  const bf16* bk = bias[k];
  for (int c4 = blockIdx.y * blockDim.x + threadIdx.x; c4 < (d >> 2); c4 += gridDim.y * blockDim.x) {
    const int i = c4 * 4;
    const float4 z = part_sum4(pv, b, kk * dpad + i);
    const uint2 hraw = *reinterpret_cast<const uint2*>(hq_last + (size_t)b * d + i);
    const uint2 braw = *reinterpret_cast<const uint2*>(bk + i);
    const __nv_bfloat162* hp = reinterpret_cast<const __nv_bfloat162*>(&hraw);
    const __nv_bfloat162* bp = reinterpret_cast<const __nv_bfloat162*>(&braw);
    const float2 h01 = __bfloat1622float2(hp[0]), h23 = __bfloat1622float2(hp[1]);
    const float2 b01 = __bfloat1622float2(bp[0]), b23 = __bfloat1622float2(bp[1]);
    *reinterpret_cast<uint2*>(r + ((size_t)b * K + k) * d + i) =
        pack4_bf16(h01.x + silu_f(z.x + b01.x), h01.y + silu_f(z.y + b01.y), h23.x + silu_f(z.z + b23.x), h23.y + silu_f(z.w + b23.y));
  }
}

// lm_head consumers of the GEMM's partial sums. argmax_partials_tc: row m, vocabulary slice
// blockIdx.y of gridDim.y: logits = sum of the slots (written out when `logits` is given), the
// slice's best (value desc, index asc) goes to pval / pidx [m][gridDim.y]. The CTA of a row that
// arrives last (arrive[m], zero between launches) picks the row's best among the slices' and writes
// pval2[m] / pidx2[m]: the order (value desc, index asc) is total, so the result does not depend on
// who arrives last, and no finishing kernel is needed.
__global__ void __launch_bounds__(256)
argmax_partials_tc(const PartView pv, int V, float* __restrict__ logits, float* __restrict__ pval, int* __restrict__ pidx,
                   unsigned int* __restrict__ arrive, float* __restrict__ pval2, int* __restrict__ pidx2,
                   unsigned long long* tr) {
  KTrace kt(tr);
  pdl_launch_dependents();
  pdl_wait();
  if (threadIdx.x == 0) trace_mark_min(tr, 2);
  const int m = blockIdx.x, nsl = gridDim.y;
  const int v4 = (V + 3) >> 2;
  const int per = (v4 + nsl - 1) / nsl;
  const int c_lo = blockIdx.y * per, c_hi = min(v4, c_lo + per);
  float bv = -INFINITY; int bi = 0x7fffffff;
  for (int c4 = c_lo + threadIdx.x; c4 < c_hi; c4 += blockDim.x) {
    const float4 a = part_sum4(pv, m, c4 * 4);
    const float z[4] = {a.x, a.y, a.z, a.w};
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      const int n = c4 * 4 + j;
      if (n < V) {
        if (logits) logits[(size_t)m * V + n] = z[j];
        if (better(z[j], n, bv, bi)) { bv = z[j]; bi = n; }
      }
    }
  }
  __shared__ float sv[8];
  __shared__ int si[8];
  warp_argmax(bv, bi);
  if ((threadIdx.x & 31) == 0) { sv[threadIdx.x >> 5] = bv; si[threadIdx.x >> 5] = bi; }
  __syncthreads();
  __shared__ int last_s;
  if (threadIdx.x == 0) {
    for (int w = 1; w < (int)(blockDim.x >> 5); ++w) if (better(sv[w], si[w], bv, bi)) { bv = sv[w]; bi = si[w]; }
    pval[(size_t)m * nsl + blockIdx.y] = bv;
    pidx[(size_t)m * nsl + blockIdx.y] = bi;
    __threadfence();
    const unsigned int old = atomicAdd(arrive + m, 1u);
    last_s = old == (unsigned int)(nsl - 1);
    if (last_s) arrive[m] = 0u;
  }
  __syncthreads();
  if (!last_s) return;
  __threadfence();
  bv = -INFINITY; bi = 0x7fffffff;
  for (int t = threadIdx.x; t < nsl; t += blockDim.x) {
    const float v = __ldcg(pval + (size_t)m * nsl + t); const int i = __ldcg(pidx + (size_t)m * nsl + t);
    if (better(v, i, bv, bi)) { bv = v; bi = i; }
  }
  __syncthreads();                                           // sv / si are reused
  warp_argmax(bv, bi);
  if ((threadIdx.x & 31) == 0) { sv[threadIdx.x >> 5] = bv; si[threadIdx.x >> 5] = bi; }
  __syncthreads();
  if (threadIdx.x == 0) {
    for (int w = 1; w < (int)(blockDim.x >> 5); ++w) if (better(sv[w], si[w], bv, bi)) { bv = sv[w]; bi = si[w]; }
    pval2[m] = bv;
    pidx2[m] = bi;
  }
}

// Per-head top-k straight from the partial sums of the heads' lm_head GEMM (no materialised logits): each
// row's kmax best (value desc, index asc) of this block's slice of the vocabulary go to the partial lists
// pk_val / pk_idx [row][block][kmax]; grid (slices, rows). The CTA of a row that arrives last (arrive[row],
// zero between launches) merges the row's lists itself (topk_merge_row: the result does not depend on who
// that is). Dynamic shared memory: the larger of slice * 4 and gridDim.x * kmax * 8 bytes.
__global__ void __launch_bounds__(256)
topk_slices_tc(const PartView pv, int V, int rows_total, int slice, int kmax, float* pk_val, int* pk_idx,
               unsigned int* __restrict__ arrive, int K, const int* __restrict__ root_tok,
               const int* __restrict__ cand_override, int* __restrict__ cand, unsigned long long* tr) {
  KTrace kt(tr);
  pdl_launch_dependents();
  pdl_wait();
  if (threadIdx.x == 0) trace_mark_min(tr, 2);
  extern __shared__ float zs[];
  const int row = blockIdx.y, n0 = blockIdx.x * slice, n1 = min(n0 + slice, V);    // slice % 4 == 0
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31, nw = blockDim.x >> 5;
  for (int c4 = threadIdx.x; c4 * 4 < n1 - n0; c4 += blockDim.x) {
    const float4 a = part_sum4(pv, row, n0 + c4 * 4);
    zs[c4 * 4] = a.x; zs[c4 * 4 + 1] = a.y; zs[c4 * 4 + 2] = a.z; zs[c4 * 4 + 3] = a.w;
  }
  __syncthreads();
  __shared__ float sv[8];
  __shared__ int si[8];
  for (int t = 0; t < kmax; ++t) {
    float bv = -INFINITY; int bi = 0x7fffffff;
    for (int c = threadIdx.x; c < n1 - n0; c += blockDim.x) if (better(zs[c], n0 + c, bv, bi)) { bv = zs[c]; bi = n0 + c; }
    warp_argmax(bv, bi);
    if (lane == 0) { sv[warp] = bv; si[warp] = bi; }
    __syncthreads();
    if (threadIdx.x == 0) {
      for (int w = 1; w < nw; ++w) if (better(sv[w], si[w], bv, bi)) { bv = sv[w]; bi = si[w]; }
      const size_t o = ((size_t)row * gridDim.x + blockIdx.x) * kmax + t;
      pk_val[o] = bv;
      pk_idx[o] = bi;
      if (bi != 0x7fffffff) zs[bi - n0] = -INFINITY;
    }
    __syncthreads();
  }
  __shared__ int last_s;
  if (threadIdx.x == 0) {
    __threadfence();
    const unsigned int old = atomicAdd(arrive + row, 1u);
    last_s = old == gridDim.x - 1;
    if (last_s) arrive[row] = 0u;
  }
  __syncthreads();
  if (!last_s) return;
  __threadfence();
  topk_merge_row(pk_val, pk_idx, (int)gridDim.x, row, K, kmax, root_tok, cand_override, cand, zs);
}

// y[m][n] = sum of the partial slots (logical columns of a single matrix): the stand-alone linear.
__global__ void __launch_bounds__(256)
part_sum_rows(const PartView pv, float* __restrict__ y, int M, int N) {
  pdl_launch_dependents();
  pdl_wait();
  const int n4 = (N + 3) >> 2;
  const size_t total = (size_t)M * n4;
  for (size_t idx = (size_t)blockIdx.x * blockDim.x + threadIdx.x; idx < total; idx += (size_t)gridDim.x * blockDim.x) {
    const int m = (int)(idx / n4), n = (int)(idx % n4) * 4;
    const float4 a = part_sum4(pv, m, n);
    const float v[4] = {a.x, a.y, a.z, a.w};
    for (int j = 0; j < 4 && n + j < N; ++j) y[(size_t)m * N + n + j] = v[j];
  }
}

}  // namespace spec
