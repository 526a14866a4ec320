// CUDA-core kernels of the decode step: row preparation, RMSNorm, row-streaming linear
// (the float32 path and the M<=few GEMV-style projections of the extra heads), RoPE + cache
// store, plain tree attention, argmax, acceptance walk, KV compaction, per-head top-k.
// Templated on the operand type T (float or bf16): operands are rounded to T exactly where
// a tensor-core kernel would consume them; accumulation is float32.
#pragma once
#include "common.cuh"

namespace spec {

// ------------------------------------------------------------------ row preparation
// Verify pass: tree node i of sequence b carries candidate rank[i] of head depth[i]
// (head 0 = the base model's own next token) and sits at position n[b] + depth[i].
template <typename T>
__global__ void prepare_verify_rows(Rows rows, const int* __restrict__ cand, int cand_stride_b, int kmax,
                                    const int* __restrict__ depth, const int* __restrict__ rank, int capacity,
                                    const T* __restrict__ embed, float* __restrict__ x, int d, int vocab,
                                    int* status, unsigned long long* tr) {
  KTrace kt(tr);
  // This kernel lets its dependents start only after its own dependency wait, i.e. after every kernel before it
  // has completed: no kernel of the verification pass begins before the previous step's kernels (its cache
  // compaction above all) are done. The attention kernels rely on that when they fetch keys below the host's
  // lower bound of the committed length ahead of their own dependency wait.
  pdl_wait();
  pdl_launch_dependents();
  if (threadIdx.x == 0) trace_mark_min(tr, 2);
  int m = blockIdx.x, b = m / rows.R, i = m % rows.R;
  int n = rows.n[b];
  bool ok = (n + rows.R <= capacity);
  if (!ok && threadIdx.x == 0) set_status(status, ST_SEQLEN, 1, b);
  int t = cand[b * cand_stride_b + depth[i] * kmax + rank[i]];
  if (t < 0 || t >= vocab) { t = 0; if (threadIdx.x == 0 && ok) set_status(status, ST_BOUNDS, 1, m); }
  if (threadIdx.x == 0) {
    rows.tok[m] = t;
    rows.pos[m] = n + depth[i];
    rows.slot[m] = n + i;
    if (i == 0) rows.cnt[b] = ok ? rows.R : 0;
  }
  const T* e = embed + (size_t)t * d;
  if (sizeof(T) == 2 && d % 8 == 0) {
    // 16-byte loads of the embedding row, all in flight at once
    for (int c8 = threadIdx.x; c8 < (d >> 3); c8 += blockDim.x) {
      const uint4 raw = *reinterpret_cast<const uint4*>(reinterpret_cast<const bf16*>(e) + c8 * 8);
      const __nv_bfloat162* hp = reinterpret_cast<const __nv_bfloat162*>(&raw);
      const float2 f0 = __bfloat1622float2(hp[0]), f1 = __bfloat1622float2(hp[1]), f2 = __bfloat1622float2(hp[2]), f3 = __bfloat1622float2(hp[3]);
      float* dst = x + (size_t)m * d + c8 * 8;
      *reinterpret_cast<float4*>(dst) = make_float4(f0.x, f0.y, f1.x, f1.y);
      *reinterpret_cast<float4*>(dst + 4) = make_float4(f2.x, f2.y, f3.x, f3.y);
    }
  } else {
    for (int c = threadIdx.x; c < d; c += blockDim.x) x[(size_t)m * d + c] = to_f<T>(e[c]);
  }
}

// Prefill pass number `chunk`: row i of sequence b is prompt token chunk*R + i.
template <typename T>
__global__ void prepare_prefill_rows(Rows rows, const int* __restrict__ prompt, const int* __restrict__ offsets,
                                     int chunk, const T* __restrict__ embed, float* __restrict__ x, int d,
                                     int vocab, int* status) {
  int m = blockIdx.x, b = m / rows.R, i = m % rows.R;
  int len = offsets[b + 1] - offsets[b];
  int p = chunk * rows.R + i;
  int t = 0;
  if (p < len) {
    t = prompt[offsets[b] + p];
    if (t < 0 || t >= vocab) { t = 0; if (threadIdx.x == 0) set_status(status, ST_BOUNDS, 2, m); }
  }
  if (threadIdx.x == 0) {
    rows.tok[m] = t;
    rows.pos[m] = p;
    rows.slot[m] = p;
    if (i == 0) {
      int c = len - chunk * rows.R;
      rows.cnt[b] = c < 0 ? 0 : (c > rows.R ? rows.R : c);
      rows.n[b] = chunk * rows.R < len ? chunk * rows.R : len;
    }
  }
  const T* e = embed + (size_t)t * d;
  for (int c = threadIdx.x; c < d; c += blockDim.x) x[(size_t)m * d + c] = (p < len) ? to_f<T>(e[c]) : 0.f;
}

// After a prefill pass: sequences whose last prompt token is in this pass keep that row's
// final hidden state (float32 and operand type) for the first step's heads and lm_head.
template <typename T>
__global__ void prefill_keep_last(Rows rows, const int* __restrict__ offsets, int chunk,
                                  const float* __restrict__ hid, float* __restrict__ h_last,
                                  T* __restrict__ hq_last, int d) {
  int b = blockIdx.x;
  int len = offsets[b + 1] - offsets[b];
  int last = len - 1;
  if (last / rows.R != chunk) return;
  int m = b * rows.R + last % rows.R;
  for (int c = threadIdx.x; c < d; c += blockDim.x) {
    float v = hid[(size_t)m * d + c];
    h_last[(size_t)b * d + c] = v;
    hq_last[(size_t)b * d + c] = from_f<T>(v);
  }
  if (threadIdx.x == 0) rows.n[b] = len;
}

// ------------------------------------------------------------------ RMSNorm (+ residual)
// x[m] += sum_s part[s][m] (s in slice order) when nsplit > 0; u[m] = T(x / rms(x) * g);
// optionally the unrounded normed row goes to hid (final norm).
template <typename T>
__global__ void rmsnorm_rows(float* __restrict__ x, const float* __restrict__ part, int nsplit, size_t split_stride,
                             const float* __restrict__ gain, float eps, T* __restrict__ u,
                             float* __restrict__ hid, int d) {
  int m = blockIdx.x;
  float* xr = x + (size_t)m * d;
  float ss = 0.f;
  for (int c = threadIdx.x; c < d; c += blockDim.x) {
    float v = xr[c];
    for (int s = 0; s < nsplit; ++s) v += part[s * split_stride + (size_t)m * d + c];
    if (nsplit > 0) xr[c] = v;
    ss += v * v;
  }
  __shared__ float red[32];
  ss = warp_sum(ss);
  if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = ss;
  __syncthreads();
  if (threadIdx.x < 32) {
    float v = threadIdx.x < (blockDim.x >> 5) ? red[threadIdx.x] : 0.f;
    v = warp_sum(v);
    if (threadIdx.x == 0) red[0] = v;
  }
  __syncthreads();
  float inv = rsqrtf(red[0] / (float)d + eps);
  for (int c = threadIdx.x; c < d; c += blockDim.x) {
    float v = xr[c] * inv * gain[c];
    u[(size_t)m * d + c] = from_f<T>(v);
    if (hid) hid[(size_t)m * d + c] = v;
  }
}

// ------------------------------------------------------------------ row-streaming linear
// y[m][n] = sum_k x[m][k] * W[n][k] for MC rows m at a time; one warp per output n streams
// the weight row once with 16-byte loads. K % 8 == 0.
template <typename T> struct Vec16;
template <> struct Vec16<float> {
  static constexpr int N = 4;
  __device__ static void load(const float* p, float (&o)[8]) {
    float4 v = *reinterpret_cast<const float4*>(p);
    o[0] = v.x; o[1] = v.y; o[2] = v.z; o[3] = v.w;
  }
};
template <> struct Vec16<bf16> {
  static constexpr int N = 8;
  __device__ static void load(const bf16* p, float (&o)[8]) {
    uint4 v = *reinterpret_cast<const uint4*>(p);
    const __nv_bfloat162* h = reinterpret_cast<const __nv_bfloat162*>(&v);
#pragma unroll
    for (int i = 0; i < 4; ++i) { float2 f = __bfloat1622float2(h[i]); o[2 * i] = f.x; o[2 * i + 1] = f.y; }
  }
};

template <typename T, int MC>
__global__ void linear_rows(const T* __restrict__ x, int ldx, const T* __restrict__ W, float* __restrict__ y,
                            int ldy, int M, int N, int K) {
  constexpr int VN = Vec16<T>::N;
  int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  int n = blockIdx.x * (blockDim.x >> 5) + warp;
  int m0 = blockIdx.y * MC;
  if (n >= N) return;
  float acc[MC];
#pragma unroll
  for (int i = 0; i < MC; ++i) acc[i] = 0.f;
  const T* wr = W + (size_t)n * K;
  for (int k = lane * VN; k < K; k += 32 * VN) {
    float wv[8], xv[8];
    Vec16<T>::load(wr + k, wv);
#pragma unroll
    for (int i = 0; i < MC; ++i) {
      if (m0 + i < M) {
        Vec16<T>::load(x + (size_t)(m0 + i) * ldx + k, xv);
#pragma unroll
        for (int e = 0; e < VN; ++e) acc[i] = fmaf(wv[e], xv[e], acc[i]);
      }
    }
  }
#pragma unroll
  for (int i = 0; i < MC; ++i) {
    float v = warp_sum(acc[i]);
    if (lane == 0 && m0 + i < M) y[(size_t)(m0 + i) * ldy + n] = v;
  }
}

// act = T(SiLU(g) * u)
template <typename T>
__global__ void swiglu_rows(const float* __restrict__ g, const float* __restrict__ up, T* __restrict__ act,
                            size_t total) {
  size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (i < total) act[i] = from_f<T>(silu_f(g[i]) * up[i]);
}

// ------------------------------------------------------------------ RoPE + cache store
// qkv: float32 [nsplit][M][(H+2Hkv)*D] partial sums. Rotate-half RoPE (element i pairs with
// i + D/2, angle pos * base^(-2i/D), table cs[pos][i] = (cos, sin)) on q and k; q -> T
// [M][H*D]; k, v -> T into the paged cache at the row's slot.
template <typename T>
__global__ void rope_store(const float* __restrict__ qkv, int nsplit, size_t split_stride, Rows rows,
                           const float2* __restrict__ cs, T* __restrict__ q, T* __restrict__ pool, KVGeom g,
                           const int* __restrict__ page_table, int layer, int H) {
  int m = blockIdx.x, b = m / rows.R, i = m % rows.R;
  if (i >= rows.cnt[b]) return;
  int D = g.head_dim, half = D >> 1, Hkv = g.n_kv_heads;
  int nq = H * D, nk = Hkv * D, ld = nq + 2 * nk;
  int pos = rows.pos[m], slot = rows.slot[m];
  int page = page_table[b * g.pages_per_seq + slot / g.page_size], prow = slot % g.page_size;
  const float* src = qkv + (size_t)m * ld;
  // q and k pairs
  int npairs = (H + Hkv) * half;
  for (int p = threadIdx.x; p < npairs; p += blockDim.x) {
    int head = p / half, e = p % half;
    int col = head * D + e;
    float a = 0.f, c = 0.f;
    for (int s = 0; s < max(nsplit, 1); ++s) {
      a += src[s * split_stride + col];
      c += src[s * split_stride + col + half];
    }
    float2 t = cs[(size_t)pos * half + e];
    float r0 = a * t.x - c * t.y, r1 = c * t.x + a * t.y;
    if (head < H) {
      q[(size_t)m * nq + head * D + e] = from_f<T>(r0);
      q[(size_t)m * nq + head * D + e + half] = from_f<T>(r1);
    } else {
      int kh = head - H;
      T* dst = pool + g.block_offset(page, layer, 0, kh) + (size_t)prow * D;
      dst[kv_elem<T>(prow, e, D, g.page_size)] = from_f<T>(r0);
      dst[kv_elem<T>(prow, e + half, D, g.page_size)] = from_f<T>(r1);
    }
  }
  for (int p = threadIdx.x; p < nk; p += blockDim.x) {
    int kh = p / D, e = p % D;
    float a = 0.f;
    for (int s = 0; s < max(nsplit, 1); ++s) a += src[s * split_stride + nq + nk + p];
    T* dst = pool + g.block_offset(page, layer, 1, kh) + (size_t)prow * D;
    dst[kv_elem<T>(prow, e, D, g.page_size)] = from_f<T>(a);
  }
}

// ------------------------------------------------------------------ plain tree attention
// One warp per (row, head). Row i of sequence b sees every cached position < n[b] and row u
// of the same pass iff bit u of anc[i] is set. Two passes over the keys: maximum, then
// exp / sum / value accumulation with the probabilities rounded to T before the product.
template <typename T>
__global__ void attention_simple(const T* __restrict__ q, T* __restrict__ out, const T* __restrict__ pool, KVGeom g,
                                 const int* __restrict__ page_table, Rows rows, int layer, int H, float scale) {
  int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  int h = blockIdx.x, b = blockIdx.y;
  int i = blockIdx.z * (blockDim.x >> 5) + warp;
  if (i >= rows.cnt[b]) return;
  int m = b * rows.R + i;
  int D = g.head_dim, EPL = D >> 5;   // D in {32,64,128,256}
  int kvh = h / (H / g.n_kv_heads);
  int n = rows.n[b], S = n + rows.cnt[b];
  float qv[8];
  for (int e = 0; e < EPL; ++e) qv[e] = to_f<T>(q[(size_t)m * H * D + h * D + lane * EPL + e]);
  uint32_t a[4];
  for (int w = 0; w < 4; ++w) a[w] = rows.anc[i * 4 + w];
  const int* pt = page_table + b * g.pages_per_seq;

  float mx = -INFINITY;
  for (int j = 0; j < S; ++j) {
    if (j >= n && !((a[(j - n) >> 5] >> ((j - n) & 31)) & 1u)) continue;
    int prow = j % g.page_size;
    const T* kr = pool + g.block_offset(pt[j / g.page_size], layer, 0, kvh) + (size_t)prow * D;
    float s = 0.f;
    for (int e = 0; e < EPL; ++e) s = fmaf(qv[e], to_f<T>(kr[kv_elem<T>(prow, lane * EPL + e, D, g.page_size)]), s);
    s = warp_sum(s) * scale;
    mx = fmaxf(mx, s);
  }
  float l = 0.f, acc[8];
  for (int e = 0; e < EPL; ++e) acc[e] = 0.f;
  for (int j = 0; j < S; ++j) {
    if (j >= n && !((a[(j - n) >> 5] >> ((j - n) & 31)) & 1u)) continue;
    int prow = j % g.page_size;
    int page = pt[j / g.page_size];
    const T* kr = pool + g.block_offset(page, layer, 0, kvh) + (size_t)prow * D;
    const T* vr = pool + g.block_offset(page, layer, 1, kvh) + (size_t)prow * D;
    float s = 0.f;
    for (int e = 0; e < EPL; ++e) s = fmaf(qv[e], to_f<T>(kr[kv_elem<T>(prow, lane * EPL + e, D, g.page_size)]), s);
    s = warp_sum(s) * scale;
    float p = expf(s - mx);
    l += p;
    float pq = quant<T>(p);
    for (int e = 0; e < EPL; ++e) acc[e] = fmaf(pq, to_f<T>(vr[kv_elem<T>(prow, lane * EPL + e, D, g.page_size)]), acc[e]);
  }
  float inv = 1.f / l;
  for (int e = 0; e < EPL; ++e) out[(size_t)m * H * D + h * D + lane * EPL + e] = from_f<T>(acc[e] * inv);
}

// ------------------------------------------------------------------ argmax over vocabulary
// One block per row; lowest index wins ties. Writes one (value, index) partial per row.
__global__ void argmax_rows(const float* __restrict__ logits, int V, float* __restrict__ pval, int* __restrict__ pidx) {
  int m = blockIdx.x;
  const float* z = logits + (size_t)m * V;
  float bv = -INFINITY;
  int bi = 0x7fffffff;
  for (int c = threadIdx.x; c < V; c += blockDim.x) {
    float v = z[c];
    if (better(v, c, bv, bi)) { bv = v; bi = c; }
  }
  __shared__ float sv[32];
  __shared__ int si[32];
  warp_argmax(bv, bi);
  if ((threadIdx.x & 31) == 0) { sv[threadIdx.x >> 5] = bv; si[threadIdx.x >> 5] = bi; }
  __syncthreads();
  if (threadIdx.x < 32) {
    int nw = blockDim.x >> 5;
    bv = threadIdx.x < nw ? sv[threadIdx.x] : -INFINITY;
    bi = threadIdx.x < nw ? si[threadIdx.x] : 0x7fffffff;
    warp_argmax(bv, bi);
    if (threadIdx.x == 0) { pval[m] = bv; pidx[m] = bi; }
  }
}

// ------------------------------------------------------------------ typical acceptance
// Eq. 1: a node passes iff p_base(token | prefix ending at its parent) >
// min(eps, delta * exp(-H(p_base))). One block per node v; it reduces its parent's logits
// row (softmax at the given temperature, entropy in nats).
__global__ void typical_edges(const float* __restrict__ logits, int V, Rows rows, const int* __restrict__ parent,
                              float eps, float delta, float inv_temp, int* __restrict__ edge_ok) {
  int m = blockIdx.x, b = m / rows.R, v = m % rows.R;
  if (v >= rows.cnt[b]) return;
  if (v == 0) { if (threadIdx.x == 0) edge_ok[m] = 1; return; }
  const float* z = logits + (size_t)(b * rows.R + parent[v]) * V;
  __shared__ float red[32];
  __shared__ float bc[2];
  float mx = -INFINITY;
  for (int c = threadIdx.x; c < V; c += blockDim.x) mx = fmaxf(mx, z[c] * inv_temp);
  mx = warp_max(mx);
  if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = mx;
  __syncthreads();
  if (threadIdx.x < 32) {
    float t = threadIdx.x < (blockDim.x >> 5) ? red[threadIdx.x] : -INFINITY;
    t = warp_max(t);
    if (threadIdx.x == 0) bc[0] = t;
  }
  __syncthreads();
  mx = bc[0];
  float se = 0.f, sez = 0.f;   // sum e, sum e * (z - mx)
  for (int c = threadIdx.x; c < V; c += blockDim.x) {
    float t = z[c] * inv_temp - mx;
    float e = expf(t);
    se += e;
    sez += e * t;
  }
  se = warp_sum(se);
  sez = warp_sum(sez);
  __shared__ float red2[32];
  __syncthreads();
  if ((threadIdx.x & 31) == 0) { red[threadIdx.x >> 5] = se; red2[threadIdx.x >> 5] = sez; }
  __syncthreads();
  if (threadIdx.x < 32) {
    int nw = blockDim.x >> 5;
    float a = threadIdx.x < nw ? red[threadIdx.x] : 0.f, c = threadIdx.x < nw ? red2[threadIdx.x] : 0.f;
    a = warp_sum(a);
    c = warp_sum(c);
    if (threadIdx.x == 0) {
      float H = logf(a) - c / a;                 // -sum p log p with p = e / a
      float thr = fminf(eps, delta * expf(-H));
      float p = expf(z[rows.tok[m]] * inv_temp - mx) / a;
      edge_ok[m] = p > thr ? 1 : 0;
    }
  }
}

// ------------------------------------------------------------------ sampled decoding
// Philox-4x32, 10 rounds (Salmon et al., SC 2011): counter c[4], key k[2] -> four 32-bit words.
__device__ __forceinline__ void philox4x32_10(uint32_t (&c)[4], uint32_t k0, uint32_t k1) {
#pragma unroll
  for (int r = 0; r < 10; ++r) {
    if (r) { k0 += 0x9E3779B9u; k1 += 0xBB67AE85u; }
    const uint32_t hi0 = __umulhi(0xD2511F53u, c[0]), lo0 = 0xD2511F53u * c[0];
    const uint32_t hi1 = __umulhi(0xCD9E8D57u, c[2]), lo1 = 0xCD9E8D57u * c[2];
    const uint32_t n0 = hi1 ^ c[1] ^ k0, n2 = hi0 ^ c[3] ^ k1;
    c[0] = n0; c[1] = lo1; c[2] = n2; c[3] = lo0;
  }
}

// Sampled decoding at a temperature (Sec. IV-B: every prompt is also decoded by sampling): the
// token that follows the accepted span is drawn from softmax(logits / temperature) of the last
// accepted node by inverting the cumulative distribution in token order at the uniform
// u = top 24 bits of philox(counter = (draw index, sequence, 0, 0), key = seed) * 2^-24.
// One block per sequence; thread t owns a contiguous chunk of the vocabulary, the chunks' weights
// are summed in double precision, a prefix over the chunks finds the chunk that holds u * total
// and its owner scans it. prefill != 0: the row is the sequence's last prompt position (row b).
__global__ void __launch_bounds__(256)
sample_root(const float* __restrict__ logits, int V, int R, int K, const int* __restrict__ path,
            const int* __restrict__ count, float temperature, uint32_t seed_lo, uint32_t seed_hi,
            int* __restrict__ draws, int* __restrict__ root_tok, int prefill) {
  const int b = blockIdx.x;
  int row = b;
  if (!prefill) {
    const int len = count[b];
    if (len < 1) return;
    row = b * R + path[b * (K + 1) + len - 1];
  }
  const float* z = logits + (size_t)row * V;
  const double inv_t = 1.0 / (double)temperature;
  __shared__ double red[256];
  __shared__ double mx_s;
  __shared__ int chunk_s;
  __shared__ double target_s, before_s;
  const int per = (V + blockDim.x - 1) / blockDim.x;
  const int c0 = threadIdx.x * per, c1 = min(V, c0 + per);
  double mx = -INFINITY;
  for (int c = c0; c < c1; ++c) mx = fmax(mx, (double)z[c] * inv_t);
  red[threadIdx.x] = mx;
  __syncthreads();
  if (threadIdx.x == 0) {
    double m = -INFINITY;
    for (int t = 0; t < (int)blockDim.x; ++t) m = fmax(m, red[t]);
    mx_s = m;
  }
  __syncthreads();
  mx = mx_s;
  double sum = 0.0;
  for (int c = c0; c < c1; ++c) sum += exp((double)z[c] * inv_t - mx);
  __syncthreads();
  red[threadIdx.x] = sum;
  __syncthreads();
  if (threadIdx.x == 0) {
    uint32_t ctr[4] = {(uint32_t)draws[b], (uint32_t)b, 0u, 0u};
    philox4x32_10(ctr, seed_lo, seed_hi);
    const double u = (double)(ctr[0] >> 8) * (1.0 / 16777216.0);
    double total = 0.0;
    for (int t = 0; t < (int)blockDim.x; ++t) total += red[t];
    const double target = u * total;
    // total was added in this order, so the last non-empty chunk always exceeds the target (u < 1)
    double acc = 0.0;
    int chunk = 0;
    for (int t = 0; t < (int)blockDim.x; ++t) {
      chunk = t;
      if (acc + red[t] > target) break;
      acc += red[t];
    }
    chunk_s = chunk; target_s = target; before_s = acc;
    draws[b] += 1;
  }
  __syncthreads();
  if ((int)threadIdx.x == chunk_s) {
    // (the scan adds the chunk's weights one by one onto the prefix; should rounding keep it from
    // passing the target, the chunk's last token is the answer)
    double acc = before_s;
    int pick = c1 - 1;
    for (int c = c0; c < c1; ++c) {
      acc += exp((double)z[c] * inv_t - mx);
      if (acc > target_s) { pick = c; break; }
    }
    root_tok[b] = pick;
  }
}

// ------------------------------------------------------------------ bounded-wait self test
// One warp waits on an mbarrier that nothing will ever complete, with the given time limit: the wait
// gives up, records ST_TIMEOUT with where = 99 in the status word and the kernel returns normally.
__global__ void wait_probe(int* status, unsigned long long limit_ns) {
  __shared__ uint64_t bar;
  if (threadIdx.x == 0) {
    mbar_init(&bar, 1);
    mbar_fence_init();
    mbar_wait(&bar, 0, status, 99, limit_ns);
  }
}

// ------------------------------------------------------------------ acceptance walk
struct AcceptArgs {
  Rows rows;
  const float* pval;   // [row][ntile]
  const int* pidx;
  int ntile;
  const int *parent, *depth;   // tree arrays [R]
  const int* edge_ok;          // typical mode: per-row pass flag; NULL = greedy token match
  int K, frag_token, d, mode;  // mode 0 = verify step, 1 = prefill (row b is sequence b)
  const float* hid;            // [rows][d]
  int *am, *path, *count, *out_tok, *n_old, *root_tok;
  float* h_last;
  bf16* hq_last;               // optional bf16 copy of h_last (operand of the extra heads' GEMM)
  int *gen_log, *gen_cnt, gen_cap;
};

// One block per sequence: finishes the per-node argmax from the partials (pval/pidx
// [row][ntile], a warp per row), walks the tree (a node is accepted iff its parent is and its
// token is the argmax at the parent, or its Eq. 1 flag is set), takes the deepest accepted node
// (lowest index on ties), applies the fragment-integrity rule, and publishes the step's result
// and the next step's state.
__global__ void __launch_bounds__(256) accept_kernel(AcceptArgs a, unsigned long long* tr) {
  KTrace kt(tr);
  pdl_launch_dependents();
  pdl_wait();
  if (threadIdx.x == 0) trace_mark_min(tr, 2);
  const int b = blockIdx.x, R = a.rows.R;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31, nw = blockDim.x >> 5;
  __shared__ int am_s[SPEC_MAX_NODES], tok_s[SPEC_MAX_NODES], par_s[SPEC_MAX_NODES], dep_s[SPEC_MAX_NODES];
  __shared__ int last_s, len_s;
  if (a.mode == 1) {
    if (warp == 0) {
      float bv = -INFINITY; int bi = 0x7fffffff;
      for (int t = lane; t < a.ntile; t += 32) {
        float v = a.pval[(size_t)b * a.ntile + t]; int i = a.pidx[(size_t)b * a.ntile + t];
        if (better(v, i, bv, bi)) { bv = v; bi = i; }
      }
      warp_argmax(bv, bi);
      if (lane == 0) {
        a.am[b] = bi;
        a.root_tok[b] = bi;
        a.gen_cnt[b] = 0;
      }
    }
    return;
  }
  const int cnt = a.rows.cnt[b], m0 = b * R;
  if (a.ntile <= 4) {
    // few partial results per row: a thread per row, every row's loads in one trip
    for (int i = threadIdx.x; i < cnt; i += blockDim.x) {
      float bv = -INFINITY; int bi = 0x7fffffff;
      for (int t = 0; t < a.ntile; ++t) {
        const float v = a.pval[(size_t)(m0 + i) * a.ntile + t]; const int idx = a.pidx[(size_t)(m0 + i) * a.ntile + t];
        if (better(v, idx, bv, bi)) { bv = v; bi = idx; }
      }
      am_s[i] = bi; a.am[m0 + i] = bi;
    }
  } else
  for (int i = warp; i < cnt; i += nw) {
    float bv = -INFINITY; int bi = 0x7fffffff;
    const float* pv = a.pval + (size_t)(m0 + i) * a.ntile;
    const int* pi = a.pidx + (size_t)(m0 + i) * a.ntile;
    for (int t = lane; t < a.ntile; t += 32) {
      float v = pv[t]; int idx = pi[t];
      if (better(v, idx, bv, bi)) { bv = v; bi = idx; }
    }
    warp_argmax(bv, bi);
    if (lane == 0) { am_s[i] = bi; a.am[m0 + i] = bi; }
  }
  for (int i = threadIdx.x; i < cnt; i += blockDim.x) {
    tok_s[i] = a.rows.tok[m0 + i];
    par_s[i] = a.parent[i];
    dep_s[i] = a.depth[i];
  }
  __syncthreads();
  if (threadIdx.x == 0) {
    int len = 0, last = 0;
    for (int j = 0; j <= a.K; ++j) a.path[b * (a.K + 1) + j] = -1;
    if (cnt > 0) {
      // acc bits in registers: up to 128 nodes
      uint32_t acc[4] = {1u, 0u, 0u, 0u};
      int best = 0;
      for (int v = 1; v < cnt; ++v) {
        int p = par_s[v];
        bool ok = (acc[p >> 5] >> (p & 31)) & 1u;
        if (ok) ok = a.edge_ok ? (a.edge_ok[m0 + v] != 0) : (tok_s[v] == am_s[p]);
        if (ok) {
          acc[v >> 5] |= 1u << (v & 31);
          if (dep_s[v] > dep_s[best]) best = v;
        }
      }
      len = dep_s[best] + 1;
      int path[SPEC_MAX_HEADS + 1];
      for (int u = best; u >= 0; u = par_s[u]) path[dep_s[u]] = u;
      if (a.frag_token >= 0) {
        int keep = 1;
        for (int j = 0; j < len; ++j) if (tok_s[path[j]] == a.frag_token) keep = j + 1;
        len = keep;
      }
      int n = a.rows.n[b], gc = a.gen_cnt[b];
      for (int j = 0; j < len; ++j) {
        int t = tok_s[path[j]];
        a.path[b * (a.K + 1) + j] = path[j];
        a.out_tok[b * (a.K + 1) + j] = t;
        if (gc + j < a.gen_cap) a.gen_log[(size_t)b * a.gen_cap + gc + j] = t;
      }
      last = path[len - 1];
      a.n_old[b] = n;
      a.rows.n[b] = n + len;
      a.gen_cnt[b] = gc + len;
      a.root_tok[b] = am_s[last];
    }
    a.count[b] = len;
    last_s = last; len_s = len;
  }
  __syncthreads();
  if (len_s > 0) {
    // the accepted node's hidden row feeds the next step's heads (d % 4 == 0); four groups per
    // thread are loaded before the first store, so the copy is one trip to L2 for most widths
    const float4* src = reinterpret_cast<const float4*>(a.hid + (size_t)(m0 + last_s) * a.d);
    float4* dst = reinterpret_cast<float4*>(a.h_last + (size_t)b * a.d);
    const int n4 = a.d >> 2;
    for (int c0 = threadIdx.x; c0 < n4; c0 += 4 * blockDim.x) {
      float4 v[4];
#pragma unroll
      for (int k = 0; k < 4; ++k) {
        const int c = c0 + k * blockDim.x;
        v[k] = c < n4 ? src[c] : make_float4(0.f, 0.f, 0.f, 0.f);
      }
#pragma unroll
      for (int k = 0; k < 4; ++k) {
        const int c = c0 + k * blockDim.x;
        if (c >= n4) continue;
        dst[c] = v[k];
        if (a.hq_last) {
          __nv_bfloat162 lo = __floats2bfloat162_rn(v[k].x, v[k].y), hi = __floats2bfloat162_rn(v[k].z, v[k].w);
          uint2 pk;
          pk.x = *reinterpret_cast<uint32_t*>(&lo);
          pk.y = *reinterpret_cast<uint32_t*>(&hi);
          *reinterpret_cast<uint2*>(a.hq_last + (size_t)b * a.d + c * 4) = pk;
        }
      }
    }
  }
}

// ------------------------------------------------------------------ KV compaction
// Moves the accepted path's K/V rows from slot n_old + path[j] to slot n_old + j, for every
// layer and KV head. path[j] >= j and strictly increasing, so processing j in ascending
// order by the same thread never overwrites a row that is still to be read.
template <typename T>
__global__ void compact_kv(T* __restrict__ pool, KVGeom g, const int* __restrict__ page_table,
                           const int* __restrict__ path, const int* __restrict__ count,
                           const int* __restrict__ n_old, int K, unsigned long long* tr) {
  KTrace kt(tr);
  pdl_launch_dependents();
  pdl_wait();
  if (threadIdx.x == 0) trace_mark_min(tr, 2);
  int b = blockIdx.y;
  int blk = blockIdx.x;              // (layer*2 + kv) * Hkv + head
  int head = blk % g.n_kv_heads, lk = blk / g.n_kv_heads;
  int len = count[b];
  int D = g.head_dim;
  const int* pt = page_table + b * g.pages_per_seq;
  int n0 = n_old[b];
  for (int j = 0; j < len; ++j) {
    int src = n0 + path[b * (K + 1) + j], dst = n0 + j;
    if (src == dst) continue;
    int sr = src % g.page_size, dr = dst % g.page_size;
    const T* s = pool + g.block_offset(pt[src / g.page_size], lk >> 1, lk & 1, head) + (size_t)sr * D;
    T* t = pool + g.block_offset(pt[dst / g.page_size], lk >> 1, lk & 1, head) + (size_t)dr * D;
    for (int e = threadIdx.x; e < D; e += blockDim.x) t[kv_elem<T>(dr, e, D, g.page_size)] = s[kv_elem<T>(sr, e, D, g.page_size)];
  }
}

// ------------------------------------------------------------------ extra decoding heads
// r[b][k] = T(h + SiLU(W_k h + b_k)), h = T(h_last[b]). One warp per output element row i of
// head k; MC sequences at a time.
template <typename T, int MC>
__global__ void medusa_resblock(const float* __restrict__ h_last, const T* const* __restrict__ Wk,
                                const T* const* __restrict__ bk, T* __restrict__ r, int B, int K, int d,
                                unsigned long long* tr) {
  KTrace kt(tr);
  pdl_launch_dependents();
  pdl_wait();
  if (threadIdx.x == 0) trace_mark_min(tr, 2);
  constexpr int VN = Vec16<T>::N;
  int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  int row = blockIdx.x * (blockDim.x >> 5) + warp;   // k * d + i
  int b0 = blockIdx.y * MC;
  if (row >= K * d) return;
  int k = row / d, i = row % d;
  const T* wr = Wk[k] + (size_t)i * d;
  float acc[MC];
#pragma unroll
  for (int j = 0; j < MC; ++j) acc[j] = 0.f;
  for (int c = lane * VN; c < d; c += 32 * VN) {
    float wv[8];
    Vec16<T>::load(wr + c, wv);
#pragma unroll
    for (int j = 0; j < MC; ++j) {
      if (b0 + j < B) {
        const float* hr = h_last + (size_t)(b0 + j) * d + c;
#pragma unroll
        for (int e = 0; e < VN; ++e) acc[j] = fmaf(wv[e], quant<T>(hr[e]), acc[j]);
      }
    }
  }
#pragma unroll
  for (int j = 0; j < MC; ++j) {
    float v = warp_sum(acc[j]);
    if (lane == 0 && b0 + j < B) {
      float h = quant<T>(h_last[(size_t)(b0 + j) * d + i]);
      r[((size_t)(b0 + j) * K + k) * d + i] = from_f<T>(h + silu_f(v + to_f<T>(bk[k][i])));
    }
  }
}

// z[row][n] = W_lm[n] . r[row] for MC rows (row = b*K + k) over this block's slice of the
// vocabulary, kept in shared memory; then each row's kmax best (value desc, index asc) of
// the slice go to the partial lists pk_val/pk_idx [row][block][kmax].
template <typename T, int MC>
__global__ void medusa_lmhead_topk(const T* __restrict__ r, const T* __restrict__ Wlm, int rows_total, int V, int d,
                                   int slice, int kmax, float* __restrict__ pk_val, int* __restrict__ pk_idx,
                                   unsigned long long* tr) {
  KTrace kt(tr);
  pdl_launch_dependents();
  pdl_wait();
  if (threadIdx.x == 0) trace_mark_min(tr, 2);
  constexpr int VN = Vec16<T>::N;
  extern __shared__ float zs[];   // [MC][slice]
  int warp = threadIdx.x >> 5, lane = threadIdx.x & 31, nw = blockDim.x >> 5;
  int n0 = blockIdx.x * slice, r0 = blockIdx.y * MC;
  int n1 = min(n0 + slice, V);
  for (int n = n0 + warp; n < n1; n += nw) {
    const T* wr = Wlm + (size_t)n * d;
    float acc[MC];
#pragma unroll
    for (int j = 0; j < MC; ++j) acc[j] = 0.f;
    for (int c = lane * VN; c < d; c += 32 * VN) {
      float wv[8], xv[8];
      Vec16<T>::load(wr + c, wv);
#pragma unroll
      for (int j = 0; j < MC; ++j) {
        if (r0 + j < rows_total) {
          Vec16<T>::load(r + (size_t)(r0 + j) * d + c, xv);
#pragma unroll
          for (int e = 0; e < VN; ++e) acc[j] = fmaf(wv[e], xv[e], acc[j]);
        }
      }
    }
#pragma unroll
    for (int j = 0; j < MC; ++j) {
      float v = warp_sum(acc[j]);
      if (lane == 0) zs[j * slice + (n - n0)] = v;
    }
  }
  __syncthreads();
  for (int j = warp; j < MC; j += nw) {
    if (r0 + j >= rows_total) continue;
    float* z = zs + j * slice;
    for (int t = 0; t < kmax; ++t) {
      float bv = -INFINITY; int bi = 0x7fffffff;
      for (int c = lane; c < n1 - n0; c += 32) if (better(z[c], n0 + c, bv, bi)) { bv = z[c]; bi = n0 + c; }
      warp_argmax(bv, bi);
      if (lane == 0) {
        size_t o = ((size_t)(r0 + j) * gridDim.x + blockIdx.x) * kmax + t;
        pk_val[o] = bv;
        pk_idx[o] = bi;
        if (bi != 0x7fffffff) z[bi - n0] = -INFINITY;
      }
      __syncwarp();
    }
  }
}

// Merges the partial lists of one (sequence, head) row into cand[b][k+1][0..kmax) and applies
// the optional override table; the row of head 0 of each sequence also writes cand[b][0][0] = root.
// The row's nblocks * kmax candidates sit in shared memory (ms: nblocks * kmax * 8 bytes), every
// thread looking after each blockDim-th of them; kmax rounds of a block-wide argmax (value desc,
// index asc), the owner of the winner taking it out. Called by all threads of a CTA of at most 8
// warps; the lists are read around L1 (another CTA of the same launch may have written them).
__device__ __forceinline__ void topk_merge_row(const float* pk_val, const int* pk_idx, int nblocks, int row, int K, int kmax,
                                               const int* __restrict__ root_tok, const int* __restrict__ cand_override,
                                               int* __restrict__ cand, float* ms) {
  __shared__ float wv[8];
  __shared__ int wi[8], wc[8];
  const int b = row / K, k = row % K;
  const int total = nblocks * kmax;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31, nw = blockDim.x >> 5;
  float* v = ms;
  int* ix = reinterpret_cast<int*>(ms + total);
  for (int c = threadIdx.x; c < total; c += blockDim.x) {
    const size_t o = (size_t)row * total + c;          // lists of a row are contiguous: [row][block][kmax]
    v[c] = __ldcg(pk_val + o);
    ix[c] = __ldcg(pk_idx + o);
  }
  // the override entries do not depend on the lists: one load per round, issued up front
  int ovr = -1;
  if (cand_override && threadIdx.x < kmax) ovr = cand_override[((size_t)b * K + k) * kmax + threadIdx.x];
  __syncthreads();
  int* out = cand + ((size_t)b * (K + 1) + k + 1) * kmax;
  for (int t = 0; t < kmax; ++t) {
    float bv = -INFINITY; int bi = 0x7fffffff, bc = -1;
    for (int c = threadIdx.x; c < total; c += blockDim.x)
      if (better(v[c], ix[c], bv, bi)) { bv = v[c]; bi = ix[c]; bc = c; }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
      const float ov = __shfl_xor_sync(0xffffffffu, bv, o);
      const int oi = __shfl_xor_sync(0xffffffffu, bi, o), oc = __shfl_xor_sync(0xffffffffu, bc, o);
      if (better(ov, oi, bv, bi)) { bv = ov; bi = oi; bc = oc; }
    }
    if (lane == 0) { wv[warp] = bv; wi[warp] = bi; wc[warp] = bc; }
    __syncthreads();
    bv = wv[0]; bi = wi[0]; bc = wc[0];
    for (int w = 1; w < nw; ++w)
      if (better(wv[w], wi[w], bv, bi)) { bv = wv[w]; bi = wi[w]; bc = wc[w]; }
    // every thread holds the winner; its owner takes it out, thread t publishes rank t
    if (bc >= 0 && bc % (int)blockDim.x == (int)threadIdx.x) { v[bc] = -INFINITY; ix[bc] = 0x7fffffff; }
    if ((int)threadIdx.x == t) {
      const int tokv = ovr >= 0 ? ovr : bi;
      out[t] = (tokv == 0x7fffffff) ? 0 : tokv;
    }
    __syncthreads();
  }
  if (k == 0 && threadIdx.x == 0) cand[(size_t)b * (K + 1) * kmax] = root_tok[b];
}

// The merge as a kernel of its own (one CTA per row; dynamic shared memory nblocks * kmax * 8 bytes).
__global__ void __launch_bounds__(256)
topk_merge(const float* __restrict__ pk_val, const int* __restrict__ pk_idx, int nblocks,
           int rows_total, int K, int kmax, const int* __restrict__ root_tok,
           const int* __restrict__ cand_override, int* __restrict__ cand, unsigned long long* tr) {
  KTrace kt(tr);
  pdl_launch_dependents();
  pdl_wait();
  if (threadIdx.x == 0) trace_mark_min(tr, 2);
  extern __shared__ float ms[];     // values [nblocks*kmax], indices [nblocks*kmax]
  topk_merge_row(pk_val, pk_idx, nblocks, blockIdx.x, K, kmax, root_tok, cand_override, cand, ms);
}

}  // namespace spec
