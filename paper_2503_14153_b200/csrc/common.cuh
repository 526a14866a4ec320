// Shared device helpers: status word, type conversion, warp reductions and the PTX
// wrappers (mbarrier, bulk/TMA copies, tcgen05) used by the sm_100a kernels.
#pragma once
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

namespace spec {

typedef __nv_bfloat16 bf16;

// Device status word: [0] code (0 clean), [1] where, [2] detail, [3] spare.
enum { ST_OK = 0, ST_TIMEOUT = 1, ST_BOUNDS = 2, ST_SEQLEN = 3 };

__device__ __forceinline__ void set_status(int* status, int code, int where, int detail) {
  if (atomicCAS(status, 0, code) == 0) {
    status[1] = where;
    status[2] = detail;
  }
}

template <typename T> __device__ __forceinline__ float to_f(T v);
template <> __device__ __forceinline__ float to_f<float>(float v) { return v; }
template <> __device__ __forceinline__ float to_f<bf16>(bf16 v) { return __bfloat162float(v); }
template <typename T> __device__ __forceinline__ T from_f(float v);
template <> __device__ __forceinline__ float from_f<float>(float v) { return v; }
template <> __device__ __forceinline__ bf16 from_f<bf16>(float v) { return __float2bfloat16_rn(v); }
// value after a round trip through the operand type (identity for float)
template <typename T> __device__ __forceinline__ float quant(float v) { return to_f<T>(from_f<T>(v)); }

__device__ __forceinline__ float silu_f(float x) { return x / (1.0f + __expf(-x)); }

__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  return v;
}
__device__ __forceinline__ float warp_max(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, o));
  return v;
}
// (value, index) pair ordered by value descending then index ascending
__device__ __forceinline__ bool better(float v, int i, float ov, int oi) {
  return v > ov || (v == ov && i < oi);
}
__device__ __forceinline__ void warp_argmax(float& v, int& i) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) {
    float ov = __shfl_xor_sync(0xffffffffu, v, o);
    int oi = __shfl_xor_sync(0xffffffffu, i, o);
    if (better(ov, oi, v, i)) { v = ov; i = oi; }
  }
}

// ------------------------------------------------------------------ KV page layout
// Pool layout: [layer][kv_head][page][K|V][block]. The K block and the V block of a (page, layer, head) are
// adjacent, so one bulk copy brings both (a bulk copy costs about the same whether it moves 4 KB or 8 KB), and
// the pages of one (layer, head) -- what an attention CTA streams -- lie side by side: with one sequence its
// keys are one contiguous run of HBM, with several the runs interleave page by page (page p of sequence b is
// pool page p * max_batch + b).
// A float32 block is page_size rows of head_dim values. A bf16 block (head_dim % 64 == 0) holds head_dim / 64
// slabs; slab h = dims [64 h, 64 h + 64) of all page_size rows, a row of a slab being 128 bytes whose eight
// 16-byte chunks are XOR-swizzled with the row index (low 3 bits). That is the tensor cores' canonical K-major
// tile with the 128-byte swizzle: slabs of consecutive pages appended in shared memory are a valid tcgen05.mma
// operand as they are (K as the K-major B operand of Q K^T, V as the MN-major B operand of P V), and the rows are
// conflict-free for ldmatrix. kv_elem returns the element offset of (row, d) relative to the row's nominal
// base `block + row * head_dim` (it may be negative).
template <typename T> __device__ __host__ __forceinline__ int kv_elem(int row, int d, int D, int ps) { return d; }
template <> __device__ __host__ __forceinline__ int kv_elem<bf16>(int row, int d, int D, int ps) {
  const int h = d >> 6, dd = d & 63;
  return h * ps * 64 + row * 64 + ((((dd >> 3) ^ (row & 7)) << 3) | (dd & 7)) - row * D;
}

struct KVGeom {
  int n_layers, n_kv_heads, head_dim, page_size, pages_per_seq, max_batch;
  // elements
  __device__ __host__ __forceinline__ size_t block_elems() const { return (size_t)page_size * head_dim; }
  __device__ __host__ __forceinline__ size_t page_elems() const {
    return (size_t)n_layers * 2 * n_kv_heads * block_elems();
  }
  __device__ __host__ __forceinline__ size_t pool_pages() const { return (size_t)pages_per_seq * max_batch; }
  __device__ __host__ __forceinline__ size_t block_offset(int page, int layer, int kv, int head) const {
    return ((((size_t)layer * n_kv_heads + head) * pool_pages() + page) * 2 + kv) * block_elems();
  }
};

// Per-pass row bookkeeping. Row m = b * R + i belongs to sequence b; it is valid iff
// i < cnt[b]. n[b] cached positions precede the pass's rows of sequence b.
struct Rows {
  int R, B;
  int *tok, *pos, *slot;  // [B*R]
  int *n, *cnt;           // [B]
  const uint32_t* anc;    // [R][4] ancestor bitsets (bit u of anc[i]: row i sees row u)
};

// ------------------------------------------------------------------ PTX wrappers
__device__ __forceinline__ uint32_t smem_u32(const void* p) {
  return static_cast<uint32_t>(__cvta_generic_to_shared(p));
}
__device__ __forceinline__ uint64_t global_timer_ns() {
  uint64_t t;
  asm volatile("mov.u64 %0, %globaltimer;" : "=l"(t));
  return t;
}
__device__ __forceinline__ void mbar_init(uint64_t* bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(bar)), "r"(count));
}
__device__ __forceinline__ void mbar_fence_init() {
  asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint64_t* bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_u32(bar)), "r"(bytes)
               : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint64_t* bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_u32(bar)) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint64_t* bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(ok)
      : "r"(smem_u32(bar)), "r"(parity)
      : "memory");
  return ok != 0;
}
// Bounded wait: gives up after limit_ns (2 s unless the caller says otherwise), records where in the
// status word and returns false.
#define SPEC_WAIT_LIMIT_NS 2000000000ull
__device__ __forceinline__ bool mbar_wait(uint64_t* bar, uint32_t parity, int* status, int where,
                                          uint64_t limit_ns = SPEC_WAIT_LIMIT_NS) {
  if (mbar_try_wait(bar, parity)) return true;
  uint64_t t0 = global_timer_ns();
  uint32_t spins = 0;
  while (!mbar_try_wait(bar, parity)) {
    if ((++spins & 0x3f) == 0 && global_timer_ns() - t0 > limit_ns) {
      set_status(status, ST_TIMEOUT, where, (int)parity);
      return false;
    }
  }
  return true;
}

// 2D tiled TMA load: coordinates {x (innermost), y}; completes on the mbarrier.
__device__ __forceinline__ void tma_load_2d(void* smem_dst, const void* tmap, int x, int y, uint64_t* bar) {
  asm volatile(
      "cp.async.bulk.tensor.2d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4}], [%2];"
      ::"r"(smem_u32(smem_dst)), "l"(tmap), "r"(smem_u32(bar)), "r"(x), "r"(y)
      : "memory");
}
// L2 policy for data that is read once (the weight stream): first in line for eviction, so that
// it does not push activations, partial sums and the KV cache out of L2.
__device__ __forceinline__ uint64_t l2_policy_evict_first() {
  uint64_t pol;
  asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(pol));
  return pol;
}
__device__ __forceinline__ void tma_load_2d_hint(void* smem_dst, const void* tmap, int x, int y, uint64_t* bar, uint64_t policy) {
  asm volatile(
      "cp.async.bulk.tensor.2d.shared::cluster.global.tile.mbarrier::complete_tx::bytes.L2::cache_hint [%0], [%1, {%3, %4}], [%2], %5;"
      ::"r"(smem_u32(smem_dst)), "l"(tmap), "r"(smem_u32(bar)), "r"(x), "r"(y), "l"(policy)
      : "memory");
}
__device__ __forceinline__ void tma_prefetch_desc(const void* tmap) {
  asm volatile("prefetch.tensormap [%0];" ::"l"(tmap) : "memory");
}
// 1D bulk copy global -> shared (both 16-byte aligned, size multiple of 16).
__device__ __forceinline__ void bulk_load_1d(void* smem_dst, const void* gsrc, uint32_t bytes, uint64_t* bar) {
  asm volatile(
      "cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
      ::"r"(smem_u32(smem_dst)), "l"(gsrc), "r"(bytes), "r"(smem_u32(bar))
      : "memory");
}

__device__ __forceinline__ void bulk_load_1d_hint(void* smem_dst, const void* gsrc, uint32_t bytes, uint64_t* bar, uint64_t policy) {
  asm volatile(
      "cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes.L2::cache_hint [%0], [%1], %2, [%3], %4;"
      ::"r"(smem_u32(smem_dst)), "l"(gsrc), "r"(bytes), "r"(smem_u32(bar)), "l"(policy)
      : "memory");
}

// ---- tcgen05 (5th-gen tensor cores, accumulators in tensor memory) ----
__device__ __forceinline__ void tmem_alloc(uint32_t* smem_dst, uint32_t ncols) {
  asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(smem_dst)),
               "r"(ncols)
               : "memory");
}
__device__ __forceinline__ void tmem_relinquish() {
  asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_dealloc(uint32_t taddr, uint32_t ncols) {
  asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(taddr), "r"(ncols) : "memory");
}
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
// D[tmem] (+)= A[smem] * B[smem]; bf16 inputs, float32 accumulate.
__device__ __forceinline__ void tc_mma_f16(uint32_t tmem_d, uint64_t adesc, uint64_t bdesc, uint32_t idesc,
                                           uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
      ::"r"(tmem_d), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate)
      : "memory");
}
// mbarrier arrives once all tcgen05 operations issued so far by this thread are complete.
__device__ __forceinline__ void tc_commit(uint64_t* bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(smem_u32(bar))
               : "memory");
}
// 32 lanes x 16 consecutive 32-bit columns: thread i of the warp reads lane (base+i).
__device__ __forceinline__ void tmem_ld16(uint32_t taddr, uint32_t (&r)[16]) {
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x16.b32 {%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15}, [%16];"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
        "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15])
      : "r"(taddr)
      : "memory");
}
// 32 lanes x N consecutive 32-bit columns in one instruction (N = 32 or 64).
__device__ __forceinline__ void tmem_ld32(uint32_t taddr, uint32_t (&r)[32]) {
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
      "{%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,%16,%17,%18,%19,%20,%21,%22,%23,%24,%25,%26,%27,%28,%29,%30,%31}, [%32];"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
        "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]),
        "=r"(r[16]), "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]),
        "=r"(r[24]), "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
      : "r"(taddr)
      : "memory");
}
__device__ __forceinline__ void tmem_ld_wait() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }

// Shared-memory matrix descriptor for a K-major bf16 tile stored as rows of 128 bytes with
// the 128-byte swizzle (8-row groups are 1024 bytes apart). Fields: start address >> 4 in
// bits [0,14), stride byte offset >> 4 in bits [32,46), descriptor version 1 in bits
// [46,48), layout type 2 (128-byte swizzle) in bits [61,64).
__device__ __forceinline__ uint64_t make_kmajor_sw128_desc(uint32_t smem_addr) {
  uint64_t d = 0;
  d |= (uint64_t)((smem_addr & 0x3FFFFu) >> 4);
  d |= (uint64_t)(1024u >> 4) << 32;
  d |= (uint64_t)1 << 46;
  d |= (uint64_t)2 << 61;
  return d;
}
// Instruction descriptor, kind::f16: float32 accumulator (bits [4,6) = 1), bf16 A and B
// (bits [7,10) and [10,13) = 1), both K-major, N >> 3 in bits [17,23), M >> 4 in bits [24,29).
__device__ __host__ __forceinline__ uint32_t make_idesc_bf16(int M, int N) {
  return (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(N >> 3) << 17) | ((uint32_t)(M >> 4) << 24);
}

// programmatic dependent launch
__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ void pdl_launch_dependents() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }

// Optional per-launch timeline: t[0] = earliest block start, t[1] = latest block end,
// t[2] / t[3] = kernel-specific marks (earliest / latest), all in globaltimer nanoseconds.
// The host presets t[0] and t[2] to all-ones and t[1], t[3] to zero. t == nullptr: off.
struct KTrace {
  unsigned long long* t;
  __device__ __forceinline__ explicit KTrace(unsigned long long* p) : t(p) {
    if (t && threadIdx.x == 0) atomicMin(t, (unsigned long long)global_timer_ns());
  }
  __device__ __forceinline__ ~KTrace() {
    if (t && threadIdx.x == 0) atomicMax(t + 1, (unsigned long long)global_timer_ns());
  }
};
__device__ __forceinline__ void trace_mark_min(unsigned long long* t, int i) {
  if (t) atomicMin(t + i, (unsigned long long)global_timer_ns());
}
__device__ __forceinline__ void trace_mark_max(unsigned long long* t, int i) {
  if (t) atomicMax(t + i, (unsigned long long)global_timer_ns());
}

}  // namespace spec
