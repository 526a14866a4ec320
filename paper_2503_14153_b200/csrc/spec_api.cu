// C ABI of the draft-and-verify decode loop: context set-up, workspace carving, the
// per-step kernel schedule and the debug taps. All device work is enqueued on the caller's
// stream (a step is recorded once on a stream of the library's own and replayed on the caller's);
// every device buffer lies in the caller's workspace.
#include "../../include/spec_decode.h"

#include <cuda.h>
#include <cuda_runtime.h>
#include <math.h>
#include <stdio.h>
#include <stdlib.h>
#include <string.h>

#include <algorithm>
#include <map>
#include <string>
#include <tuple>
#include <vector>

#include "attention_tc.cuh"
#include "attention_umma.cuh"
#include "common.cuh"
#include "gemm_cluster.cuh"
#include "gemm_stream.cuh"
#include "gemm_wide.cuh"
#include "glue_tc.cuh"
#include "kernels_simple.cuh"
#include "labels.cuh"

using namespace spec;

namespace {

thread_local std::string g_create_error = "no error";

constexpr int PREFILL_ROWS = 128;   // rows per sequence in one prefill pass
constexpr int TRACE_CAP = 1024;     // launches of one step the timeline can hold
constexpr int SM_SLOTS = 296;       // 148 SMs x 2 co-resident GEMM CTAs
constexpr int N_COPY_EVERY = 4;         // enqueue-only steps between two copies of the committed lengths to the host
constexpr int MAX_STEPS_AHEAD = 8;      // enqueue-only steps the host may run ahead of the device
constexpr int ATTN_ROWS_WARPS = 6;      // warps of the CTA-per-16-rows attention kernel
constexpr int ATTN_SPLIT_TILES = 8;       // fewest KV tiles a split of attention_tc gets (2..8 measured alike)
constexpr int ATTN_SINGLE_TILES = 12;   // contexts of at most this many 64-key tiles use one KV split
constexpr int ATTN_LONG_KEYS = 2048;    // default context length from which passes of more than 32 rows use the shared-K/V kernel

inline size_t round_up(size_t v, size_t a) { return (v + a - 1) / a * a; }

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn get_encode_fn() {
  static EncodeTiledFn fn = nullptr;
  if (!fn) {
    void* p = nullptr;
    cudaDriverEntryPointQueryResult q;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) == cudaSuccess &&
        q == cudaDriverEntryPointSuccess)
      fn = reinterpret_cast<EncodeTiledFn>(p);
  }
  return fn;
}

// bf16 row-major [rows][cols] matrix, box = box_rows x 64 columns (128 bytes), 128-byte swizzle.
bool make_tmap(CUtensorMap* tm, const void* ptr, uint64_t rows, uint64_t cols, uint32_t box_rows) {
  EncodeTiledFn fn = get_encode_fn();
  if (!fn) return false;
  cuuint64_t dims[2] = {cols, rows};
  cuuint64_t strides[1] = {cols * 2};
  cuuint32_t box[2] = {64, box_rows};
  cuuint32_t estr[2] = {1, 1};
  CUresult r = fn(tm, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(ptr), dims, strides, box, estr,
                  CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                  CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  return r == CUDA_SUCCESS;
}

struct Bump {
  uint8_t* base;
  size_t off = 0;
  explicit Bump(void* b) : base(static_cast<uint8_t*>(b)) {}
  template <typename T> T* take(size_t count, size_t align = 256) {
    off = round_up(off, align);
    T* p = base ? reinterpret_cast<T*>(base + off) : nullptr;
    off += count * sizeof(T);
    return p;
  }
};

int mt_for_rows(int M) {
  if (M <= 16) return 16;
  if (M <= 32) return 32;
  if (M <= 64) return 64;
  return 128;
}

// Launch with or without the programmatic-dependent-launch attribute.
template <typename... Params, typename... Args>
cudaError_t launch_k(bool pdl, void (*kernel)(Params...), dim3 grid, dim3 block, size_t smem, cudaStream_t st, Args&&... args) {
  cudaLaunchConfig_t cfg{};
  cfg.gridDim = grid; cfg.blockDim = block; cfg.dynamicSmemBytes = smem; cfg.stream = st;
  cudaLaunchAttribute at[1];
  at[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  at[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = at;
  cfg.numAttrs = pdl ? 1 : 0;
  return cudaLaunchKernelEx(&cfg, kernel, std::forward<Args>(args)...);
}

// One launch of the weight-streaming GEMM: shapes, the dealing of units to CTAs and the view
// of its partial sums.
struct GemmPlan {
  StreamGemmParams p;
  int MT, grid;
};

bool plan_gemm(int M, int K, int n_mats, const int* rows, int g_max, GemmPlan* out) {
  if (M < 1 || K < 64 || K % 64 || n_mats < 1 || n_mats > GS_MAX_MATS || g_max < 1) return false;
  GemmPlan& g = *out;
  g = GemmPlan{};
  StreamGemmParams& p = g.p;
  g.MT = mt_for_rows(M);
  p.M = M; p.K = K; p.n_mats = n_mats;
  int tiles = 0, col = 0;
  for (int i = 0; i < n_mats; ++i) {
    if (rows[i] < 1) return false;
    p.mat_tile0[i] = tiles; p.mat_rows[i] = rows[i]; p.mat_col0[i] = col;
    tiles += (rows[i] + 127) / 128;
    col += rows[i];
  }
  for (int i = n_mats; i <= GS_MAX_MATS; ++i) p.mat_tile0[i] = tiles;
  p.n_tiles = tiles;
  p.seg.KC = K / 64;
  p.seg.m_tiles = (M + g.MT - 1) / g.MT;
  long long total = (long long)tiles * p.seg.m_tiles * p.seg.KC;
  if (total > 0x3fffffff || (total + 1) * (long long)g_max >= 0x7fffffffLL) return false;
  p.seg.total = (int)total;
  g.grid = (int)std::min<long long>(g_max, total);
  p.seg.G = g.grid;
  return true;
}

// Upper bound of the partial-sum slots a tile can have when the units go to at most g_max CTAs.
int plan_slot_bound(const GemmPlan& g) {
  const SegMap& s = g.p.seg;
  return (int)(((long long)s.KC * s.G) / s.total) + 2;
}

size_t plan_part_floats(const GemmPlan& g) { return (size_t)plan_slot_bound(g) * g.p.M * g.p.n_tiles * 128; }

// The shared-memory attribute of a kernel is per device: it is set on every launch's device the first time
// that device is seen (indexed by the device ordinal), not once per process.
constexpr int kAttrDevices = 64;
inline bool* attr_flag(bool (&flags)[kAttrDevices]) {
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kAttrDevices) dev = 0;
  return &flags[dev];
}

template <int MT, int DEEP>
cudaError_t launch_gs_mt(cudaStream_t st, bool pdl, int grid, const StreamTmaps& tm, const StreamGemmParams& p) {
  static bool attr_set_dev[kAttrDevices] = {};
  bool& attr_set = *attr_flag(attr_set_dev);
  if (!attr_set) {
    cudaError_t e = cudaFuncSetAttribute(gemm_stream<MT, DEEP>, cudaFuncAttributeMaxDynamicSharedMemorySize, StreamCfg<MT, DEEP>::SMEM_BYTES);
    if (e != cudaSuccess) return e;
    attr_set = true;
  }
  return launch_k(pdl, gemm_stream<MT, DEEP>, dim3(grid), dim3(192), (size_t)StreamCfg<MT, DEEP>::SMEM_BYTES, st, tm, p);
}
// Grids of at most one CTA per SM get the deep ring (one resident CTA must keep the SM's share
// of the memory pipe full by itself).
cudaError_t launch_gs(cudaStream_t st, bool pdl, const GemmPlan& g, const StreamTmaps& tm) {
  const bool deep = g.grid <= SM_SLOTS / 2;
  switch (g.MT) {
    case 16: return deep ? launch_gs_mt<16, 1>(st, pdl, g.grid, tm, g.p) : launch_gs_mt<16, 0>(st, pdl, g.grid, tm, g.p);
    case 32: return deep ? launch_gs_mt<32, 1>(st, pdl, g.grid, tm, g.p) : launch_gs_mt<32, 0>(st, pdl, g.grid, tm, g.p);
    case 64: return deep ? launch_gs_mt<64, 1>(st, pdl, g.grid, tm, g.p) : launch_gs_mt<64, 0>(st, pdl, g.grid, tm, g.p);
    default: return deep ? launch_gs_mt<128, 1>(st, pdl, g.grid, tm, g.p) : launch_gs_mt<128, 0>(st, pdl, g.grid, tm, g.p);
  }
}

PartView plan_view(const GemmPlan& g) {
  PartView v{};
  v.part = g.p.part; v.slot_stride = g.p.slot_stride; v.ld = g.p.n_tiles * 128; v.seg = g.p.seg;
  v.mt_shift = g.MT == 16 ? 4 : (g.MT == 32 ? 5 : (g.MT == 64 ? 6 : 7));
  return v;
}

}  // namespace

struct spec_ctx {
  spec_config cfg;
  cudaStream_t stream;
  int T, K, kmax, B;                   // tree nodes, heads, candidates per head, current batch
  bool tc;                             // bf16 tensor-core path
  size_t esz;                          // operand element size
  int Mcap, cap, pages_per_seq, gen_cap, nsplit_attn, Nqkv, ntile_lm, topk_slice, topk_blocks;
  bool qkv_fused, keep_logits;
  bool packed = false;                 // linear weights are pre-tiled images (SPEC_FLAG_PACKED_WEIGHTS)
  bool pdl = true;                     // programmatic dependent launch between the kernels of a step
  int gemm_ctas = 288;                 // persistent CTAs of the weight-streaming GEMM (measured best; at most SM_SLOTS)
  int l2_prefetch = 0;
  bool gc_attr_set[12] = {};            // per context (and so per device): shared-memory attribute of each gemm_cluster instance set
  int long_attn_keys = ATTN_LONG_KEYS; // SPEC_OPT_LONG_ATTN_KEYS (0 = never)
  bool attn_umma = true;               // SPEC_OPT_ATTN_UMMA: the long-context kernel is the tcgen05 one (head_dim 128)
  CUtensorMap tm_kv;                   // 5-D view of the page pool for its TMA loads
  bool tm_kv_ok = false;
  bool wide_gemm = true;               // SPEC_OPT_WIDE_GEMM: passes of more than 128 rows use the 128 x 256-tile kernel
  int cluster_epilogue = 7;            // SPEC_OPT_CLUSTER_EPILOGUE: which projections finish their split-K sums inside a cluster
                                       // (bits: 1 output/down, 2 gate+up, 4 q/k/v; measured on the 7B shape: only gate+up pays)
  int small_gemm_ctas = 288;           // CTAs of GEMMs with at most 48 weight tiles (Wo, down); 288 since the weights are pre-tiled (192 before)
  std::vector<int> h_parent, h_depth, h_rank;
  std::vector<int> n_hi, n_lo;         // host upper / lower bounds of the committed lengths
  std::vector<const void*> wq, wk, wv, wo, wg, wu, wd, mw, mb;
  std::vector<const float*> an, fn;
  const void *embed, *lm_head;
  const float* final_norm;
  KVGeom geom;
  // device buffers (workspace)
  int *d_n, *d_cnt, *d_n_old, *d_root, *d_count, *d_path, *d_out_tok, *d_gen_cnt, *d_gen_log, *d_cand, *d_cand_ov;
  int *d_tok, *d_pos, *d_slot, *d_am, *d_edge, *d_parent, *d_depth, *d_rank, *d_page_table, *d_prompt, *d_offsets;
  int *d_status, *d_pidx, *d_pk_idx, *d_draws;
  uint32_t *d_anc_tree, *d_anc_chain;
  const void **d_mw, **d_mb;
  float *d_x, *d_hid, *d_h_last, *d_part, *d_logits, *d_pval, *d_part_o, *d_part_ml, *d_pk_val;
  float* d_ss_part = nullptr;          // [128 rows][d / 128 tiles x 8]: sums of squares the residual cluster epilogue leaves
  float2* d_rope;
  void *d_u, *d_q, *d_attn, *d_act, *d_hq, *d_hq_last, *d_r, *d_pool;
  size_t part_floats;
  std::map<std::tuple<const void*, uint64_t, uint64_t, uint32_t>, CUtensorMap> tmaps;
  long long launches = 0;
  // optional device timeline of the last step: four stamps per launch (see KTrace)
  bool trace_on = false;
  unsigned long long* d_trace = nullptr;
  unsigned int* d_attn_arrive = nullptr;
  unsigned int* d_row_arrive = nullptr;   // [Mcap] arrival counters of the per-row finishing steps, zero between launches
  float* d_pval2 = nullptr;            // finished per-row argmax (tensor-core path)
  int* d_pidx2 = nullptr;
  int trace_n = 0;
  std::vector<std::string> trace_names;
  std::vector<unsigned long long> trace_init;
  unsigned long long* next_trace(const char* name) {
    if (!trace_on || trace_n >= TRACE_CAP) return nullptr;
    trace_names.push_back(name);
    return d_trace + 4 * (size_t)(trace_n++);
  }
  // CUDA-graph replay of the step's kernel sequence: one instantiated graph per (override given?)
  // variant, valid while the sequences stay below the length bound its attention launches were
  // planned for and no option changed (epoch)
  bool graph_on = true;
  bool capturing = false;
  cudaStream_t cap_stream = nullptr;
  struct StepGraph {
    cudaGraphExec_t exec = nullptr;
    unsigned long long epoch = 0;
    int B = 0;
    long long n_launches = 0;
    std::vector<int> n_hi_plan, n_lo_plan;
  };
  StepGraph step_graph[2];
  unsigned long long graph_epoch = 1;
  long long graph_captures = 0;
  bool prefilled = false;
  // timing: phase boundaries of the last step; optional per-launch timing of one kernel kind
  cudaEvent_t phase_ev[6] = {nullptr, nullptr, nullptr, nullptr, nullptr, nullptr};
  // enqueue-only steps: the committed lengths are copied to pinned host memory now and then, so
  // the host's bounds on them stay tight without a synchronisation
  int* h_n_pinned = nullptr;           // [max_batch], cudaHostAlloc
  cudaEvent_t n_ev = nullptr;
  bool n_copy_pending = false;
  int n_copy_steps_after = 0;          // steps enqueued after the pending copy
  int steps_since_n_copy = 0;          // enqueue-only steps since the last copy was issued
  bool phase_valid = false;
  bool phase_timing = false;           // SPEC_OPT_PHASE_TIMING
  int profile_kind = 0;                 // SPEC_PROFILE_*
  std::vector<cudaEvent_t> prof_ev;     // pairs, reused every step
  int prof_used = 0;
  double prof_ms = 0.0;
  long long prof_launches = 0;
  std::string err = "no error";

  int fail(int code, const std::string& msg) { err = msg; return code; }
  const CUtensorMap* tmap(const void* p, uint64_t rows, uint64_t cols, uint32_t box_rows) {
    auto key = std::make_tuple(p, rows, cols, box_rows);
    auto it = tmaps.find(key);
    if (it != tmaps.end()) return &it->second;
    CUtensorMap tm;
    if (!make_tmap(&tm, p, rows, cols, box_rows)) return nullptr;
    return &tmaps.emplace(key, tm).first->second;
  }
};

namespace {

bool validate_tree(const spec_config* cfg, const spec_tree* tree, int* kmax_out, std::string* why) {
  int T = tree->n_nodes;
  if (T < 1 || T > SPEC_MAX_NODES || !tree->parent || !tree->depth || !tree->rank) { *why = "n_nodes out of range or null arrays"; return false; }
  if (tree->parent[0] != -1 || tree->depth[0] != 0 || tree->rank[0] != 0) { *why = "node 0 must be the root"; return false; }
  int kmax = 1;
  for (int v = 1; v < T; ++v) {
    int p = tree->parent[v];
    if (p < 0 || p >= v) { *why = "parent must precede child"; return false; }
    if (tree->depth[v] != tree->depth[p] + 1 || tree->depth[v] > cfg->n_medusa) { *why = "bad depth"; return false; }
    if (tree->rank[v] < 0 || tree->rank[v] >= SPEC_MAX_TOPK) { *why = "bad rank"; return false; }
    for (int u = 1; u < v; ++u)
      if (tree->parent[u] == p && tree->rank[u] == tree->rank[v]) { *why = "siblings share a rank"; return false; }
    if (tree->rank[v] + 1 > kmax) kmax = tree->rank[v] + 1;
  }
  *kmax_out = kmax;
  return true;
}

bool validate_config(const spec_config* c, std::string* why) {
  if (c->n_layers < 1 || c->d_model < 8 || c->n_heads < 1 || c->n_kv_heads < 1 || c->head_dim < 32 ||
      c->d_ffn < 8 || c->vocab < 2 || c->max_batch < 1 || c->max_seq < 1 || c->page_size < 1) { *why = "non-positive size"; return false; }
  if (c->dtype != 0 && c->dtype != 1) { *why = "dtype must be 0 or 1"; return false; }
  if (c->n_heads % c->n_kv_heads) { *why = "n_heads must be a multiple of n_kv_heads"; return false; }
  if (c->head_dim % 32 || c->head_dim > 256) { *why = "head_dim must be a multiple of 32, <= 256"; return false; }
  if (c->d_model % 8 || c->d_ffn % 8 || (c->n_heads * c->head_dim) % 8) { *why = "widths must be multiples of 8"; return false; }
  if (c->n_medusa < 0 || c->n_medusa > SPEC_MAX_HEADS) { *why = "n_medusa out of range"; return false; }
  if (c->accept_mode != 0 && c->accept_mode != 1) { *why = "accept_mode must be 0 or 1"; return false; }
  if (c->sampling != 0 && c->sampling != 1) { *why = "sampling must be 0 or 1"; return false; }
  if (c->sampling && (c->accept_mode != 1 || !(c->temperature > 0.f))) { *why = "sampled decoding needs accept_mode 1 and a positive temperature"; return false; }
  bool tc = c->dtype == 1 && !(c->flags & SPEC_FLAG_SIMPLE_KERNELS);
  if ((c->flags & SPEC_FLAG_PACKED_WEIGHTS) && !tc) { *why = "pre-tiled weights need the bf16 tensor-core path"; return false; }
  if (tc) {
    if (c->d_model % 64 || c->d_ffn % 64 || (c->n_heads * c->head_dim) % 64) { *why = "bf16 path needs widths that are multiples of 64"; return false; }
    if (c->head_dim != 64 && c->head_dim != 128) { *why = "bf16 path needs head_dim 64 or 128"; return false; }
    if (c->page_size != 16) { *why = "bf16 path needs page_size 16"; return false; }
    if (c->d_model < 128 || c->d_ffn < 128 || c->vocab < 128 || c->n_kv_heads * c->head_dim < 128) { *why = "bf16 path needs every weight matrix to have at least 128 rows"; return false; }
  } else if (c->dtype == 1 && c->head_dim % 64) { *why = "bf16 cache needs head_dim multiple of 64"; return false; }
  return true;
}

// Lays the workspace out; with base == nullptr only measures it.
size_t carve(spec_ctx* c, void* base) {
  const spec_config& f = c->cfg;
  Bump b(base);
  int B = f.max_batch, T = c->T, K = c->K, d = f.d_model, F = f.d_ffn, V = f.vocab;
  int HD = f.n_heads * f.head_dim;
  c->Nqkv = HD + 2 * f.n_kv_heads * f.head_dim;
  c->Mcap = (int)round_up((size_t)B * (T > PREFILL_ROWS ? T : PREFILL_ROWS), 128);
  c->cap = (int)round_up((size_t)f.max_seq + T, f.page_size);
  if (64 % f.page_size == 0) c->cap = (int)round_up(c->cap, 64);   // whole 64-key attention tiles
  c->pages_per_seq = c->cap / f.page_size;
  c->gen_cap = f.max_seq + K + 1;
  c->ntile_lm = c->tc ? 8 : 1;   // argmax partials per row (vocabulary slices)
  c->topk_slice = ((V + SM_SLOTS - 1) / SM_SLOTS + 3) / 4 * 4;
  c->topk_blocks = (V + c->topk_slice - 1) / c->topk_slice;
  c->nsplit_attn = c->tc ? std::max(1, std::min(16, (SM_SLOTS / 2) / (f.n_heads * B))) : 1;   // most KV splits a launch may use
  int Mlog = (int)round_up((size_t)B * T, 16);
  c->keep_logits = !c->tc || (f.flags & SPEC_FLAG_KEEP_LOGITS) || f.accept_mode == 1;
  size_t M = c->Mcap;

  c->d_status = b.take<int>(4);
  c->d_trace = b.take<unsigned long long>((size_t)TRACE_CAP * 4);
  c->d_attn_arrive = b.take<unsigned int>((size_t)B * f.n_heads * 2);
  c->d_row_arrive = b.take<unsigned int>(c->Mcap);
  c->d_pval2 = b.take<float>(c->Mcap); c->d_pidx2 = b.take<int>(c->Mcap);
  c->d_draws = b.take<int>(B);
  c->d_n = b.take<int>(B); c->d_cnt = b.take<int>(B); c->d_n_old = b.take<int>(B); c->d_root = b.take<int>(B);
  c->d_count = b.take<int>(B); c->d_path = b.take<int>((size_t)B * (K + 1)); c->d_out_tok = b.take<int>((size_t)B * (K + 1));
  c->d_gen_cnt = b.take<int>(B); c->d_gen_log = b.take<int>((size_t)B * c->gen_cap);
  c->d_cand = b.take<int>((size_t)B * (K + 1) * c->kmax); c->d_cand_ov = b.take<int>((size_t)B * (K ? K : 1) * c->kmax);
  c->d_tok = b.take<int>(M); c->d_pos = b.take<int>(M); c->d_slot = b.take<int>(M); c->d_am = b.take<int>(M);
  c->d_edge = b.take<int>(M);
  c->d_parent = b.take<int>(SPEC_MAX_NODES); c->d_depth = b.take<int>(SPEC_MAX_NODES); c->d_rank = b.take<int>(SPEC_MAX_NODES);
  c->d_anc_tree = b.take<uint32_t>(SPEC_MAX_NODES * 4); c->d_anc_chain = b.take<uint32_t>(PREFILL_ROWS * 4);
  c->d_page_table = b.take<int>((size_t)B * c->pages_per_seq);
  c->d_prompt = b.take<int>((size_t)B * f.max_seq); c->d_offsets = b.take<int>(B + 1);
  c->d_mw = b.take<const void*>(SPEC_MAX_HEADS); c->d_mb = b.take<const void*>(SPEC_MAX_HEADS);
  c->d_x = b.take<float>(M * d, 1024); c->d_hid = b.take<float>(M * d, 1024); c->d_h_last = b.take<float>((size_t)B * d);
  // split-K / plain projection outputs
  size_t pf = 0;
  {
    int Ms[3] = {B * T, B * PREFILL_ROWS, B};
    for (int i = 0; i < 3; ++i) {
      size_t m = Ms[i];
      if (c->tc) {
        int KD = f.n_kv_heads * f.head_dim;
        int r_qkv[3] = {HD, KD, KD}, r_o[1] = {d}, r_gu[2] = {F, F}, r_dn[1] = {d};
        GemmPlan g;
        if (plan_gemm((int)m, d, 3, r_qkv, SM_SLOTS, &g)) pf = std::max(pf, plan_part_floats(g));
        if (plan_gemm((int)m, HD, 1, r_o, SM_SLOTS, &g)) pf = std::max(pf, plan_part_floats(g));
        if (plan_gemm((int)m, d, 2, r_gu, SM_SLOTS, &g)) pf = std::max(pf, plan_part_floats(g));
        if (plan_gemm((int)m, F, 1, r_dn, SM_SLOTS, &g)) pf = std::max(pf, plan_part_floats(g));
        int r_lm[1] = {V};
        if (plan_gemm((int)m, d, 1, r_lm, SM_SLOTS, &g)) pf = std::max(pf, plan_part_floats(g));
        int r_hd[GS_MAX_MATS] = {d, d, d, d};
        if (plan_gemm((int)m, d, GS_MAX_MATS, r_hd, SM_SLOTS, &g)) pf = std::max(pf, plan_part_floats(g));
      } else {
        pf = std::max(pf, std::max(m * (size_t)c->Nqkv, 2 * m * (size_t)F));
      }
    }
  }
  c->part_floats = pf;
  c->d_part = b.take<float>(pf, 1024);
  c->d_logits = c->keep_logits ? b.take<float>((size_t)Mlog * V, 1024) : nullptr;
  c->d_pval = b.take<float>((size_t)c->ntile_lm * M, 1024); c->d_pidx = b.take<int>((size_t)c->ntile_lm * M, 1024);
  c->d_part_o = c->tc ? b.take<float>((size_t)c->nsplit_attn * M * HD, 1024) : nullptr;
  c->d_part_ml = c->tc ? b.take<float>((size_t)c->nsplit_attn * M * f.n_heads * 2) : nullptr;
  c->d_ss_part = c->tc ? b.take<float>((size_t)128 * ((d + 127) / 128) * GC_RES_CLUSTER) : nullptr;
  c->d_pk_val = b.take<float>((size_t)c->topk_blocks * B * (K ? K : 1) * c->kmax);
  c->d_pk_idx = b.take<int>((size_t)c->topk_blocks * B * (K ? K : 1) * c->kmax);
  c->d_rope = b.take<float2>((size_t)c->cap * (f.head_dim / 2));
  size_t e = c->esz;
  c->d_u = b.take<uint8_t>(M * d * e, 1024); c->d_q = b.take<uint8_t>(M * HD * e, 1024);
  c->d_attn = b.take<uint8_t>(M * HD * e, 1024); c->d_act = b.take<uint8_t>(M * F * e, 1024);
  c->d_hq = b.take<uint8_t>(M * d * e, 1024); c->d_hq_last = b.take<uint8_t>(round_up((size_t)B, 16) * d * e, 1024);
  c->d_r = b.take<uint8_t>(round_up((size_t)B * (K ? K : 1), 16) * d * e, 1024);
  c->geom = KVGeom{f.n_layers, f.n_kv_heads, f.head_dim, f.page_size, c->pages_per_seq, B};
  size_t pool_elems = (size_t)B * c->pages_per_seq * c->geom.page_elems();
  c->d_pool = b.take<uint8_t>(pool_elems * e, 1024);
  return round_up(b.off, 1024);
}

#define CUDA_OK(call)                                                                          \
  do {                                                                                         \
    cudaError_t e_ = (call);                                                                   \
    if (e_ != cudaSuccess) return c->fail(SPEC_E_CUDA, std::string(#call) + ": " + cudaGetErrorString(e_)); \
  } while (0)

#define LAUNCH_CHECK(name)                                                                     \
  do {                                                                                         \
    c->launches++;                                                                             \
    cudaError_t e_ = cudaGetLastError();                                                       \
    if (e_ != cudaSuccess) return c->fail(SPEC_E_CUDA, std::string(name) + ": " + cudaGetErrorString(e_)); \
  } while (0)

// Brackets one launch with events when that kernel kind is being profiled.
struct ProfScope {
  spec_ctx* c;
  bool on;
  ProfScope(spec_ctx* ctx, int kind) : c(ctx), on(ctx->profile_kind == kind && kind != 0) {
    if (!on) return;
    if ((size_t)c->prof_used + 2 > c->prof_ev.size()) {
      cudaEvent_t a, b;
      if (cudaEventCreate(&a) != cudaSuccess || cudaEventCreate(&b) != cudaSuccess) { on = false; return; }
      c->prof_ev.push_back(a); c->prof_ev.push_back(b);
    }
    cudaEventRecord(c->prof_ev[c->prof_used], c->stream);
  }
  ~ProfScope() {
    if (!on) return;
    cudaEventRecord(c->prof_ev[c->prof_used + 1], c->stream);
    c->prof_used += 2;
  }
};

Rows make_rows(spec_ctx* c, int R, bool chain) {
  Rows r;
  r.R = R; r.B = c->B;
  r.tok = c->d_tok; r.pos = c->d_pos; r.slot = c->d_slot; r.n = c->d_n; r.cnt = c->d_cnt;
  r.anc = chain ? c->d_anc_chain : c->d_anc_tree;
  return r;
}

const char* gemm_kind_name(int kind) {
  switch (kind) {
    case SPEC_PROFILE_GATE_UP: return "gemm_gate_up";
    case SPEC_PROFILE_QKV: return "gemm_qkv";
    case SPEC_PROFILE_WO: return "gemm_wo";
    case SPEC_PROFILE_DOWN: return "gemm_down";
    default: return "gemm";
  }
}

// CTA count for a GEMM of n_tiles weight tiles, at most cap: one that lets the CTAs' runs end on tile
// boundaries (p CTAs per q tiles, q as small as possible), so that a tile's partial sums come from as few
// CTAs as possible and the consumers read fewer slots; within 15% of cap, else cap itself.
int aligned_ctas(int n_tiles, int cap) {
  for (int q = 1; q <= 4; ++q) {
    long long p = (long long)cap * q / n_tiles;
    while (p >= 1 && (n_tiles * p) % q) --p;
    if (p < 1) continue;
    const int G = (int)(n_tiles * p / q);
    if (G * 100 >= cap * 85) return G;
  }
  return cap;
}

// ---- tensor-core linear (bf16): partial sums of x[M,K] * [mats]^T ----
// kind: SPEC_PROFILE_* of the call site. On success *view describes the partial sums.
int run_gemm(spec_ctx* c, const void* x, int M, int K, int n_mats, const void* const* mats, const int* rows, int kind,
             PartView* view) {
  GemmPlan g;
  int tiles_all = 0;
  for (int i = 0; i < n_mats; ++i) tiles_all += (rows[i] + 127) / 128;
  if (M > 128 && c->wide_gemm && K % 64 == 0 && n_mats <= GS_MAX_MATS) {
    // many rows: the compute-bound kernel, whole tiles (one "slot" of finished sums)
    WideGemmParams w{};
    w.M = M; w.K = K; w.KC = K / 64; w.n_mats = n_mats;
    int t0 = 0;
    StreamTmaps tmw{};
    for (int i = 0; i < n_mats; ++i) {
      w.mat_tile0[i] = t0;
      t0 += (rows[i] + 127) / 128;
      if (c->packed) { w.packed[i] = static_cast<const uint8_t*>(mats[i]); continue; }
      const CUtensorMap* t = c->tmap(mats[i], rows[i], K, 128);
      if (!t) return c->fail(SPEC_E_CUDA, "cuTensorMapEncodeTiled failed (weights)");
      tmw.a[i] = *t;
    }
    for (int i = n_mats; i <= GS_MAX_MATS; ++i) w.mat_tile0[i] = t0;
    w.n_tiles = tiles_all; w.m_tiles = (M + GW_NT - 1) / GW_NT;
    const long long total = (long long)w.n_tiles * w.m_tiles * w.KC;
    if ((size_t)M * tiles_all * 128 > c->part_floats) return c->fail(SPEC_E_NOMEM, "partial-sum scratch too small");
    if (total > 0x3fffffff || (total + 1) * (long long)(w.n_tiles * w.m_tiles) >= 0x7fffffffLL) return c->fail(SPEC_E_BADARG, "unsupported linear shape");
    const CUtensorMap* tb = c->tmap(x, std::max<size_t>(round_up(M, 16), GW_NT), K, GW_NT);
    if (!tb) return c->fail(SPEC_E_CUDA, "cuTensorMapEncodeTiled failed (activations)");
    tmw.b = *tb;
    w.part = c->d_part; w.status = c->d_status; w.trace = c->next_trace(gemm_kind_name(kind));
    const int grid = std::min(w.n_tiles * w.m_tiles, SM_SLOTS / 2);
    {
      ProfScope ps(c, kind);
      static bool set_dev[kAttrDevices] = {};
      bool& set_ = *attr_flag(set_dev);
      if (!set_) { CUDA_OK(cudaFuncSetAttribute(gemm_wide, cudaFuncAttributeMaxDynamicSharedMemorySize, WideCfg::SMEM_BYTES)); set_ = true; }
      cudaError_t e = launch_k(c->pdl, gemm_wide, dim3(grid), dim3(GW_THREADS), (size_t)WideCfg::SMEM_BYTES, c->stream, tmw, w);
      c->launches++;
      if (e != cudaSuccess) return c->fail(SPEC_E_CUDA, std::string("gemm_wide launch: ") + cudaGetErrorString(e));
    }
    // the consumers see one finished slot per tile: a dealing of the units with one CTA per (weight tile, 256-row tile)
    PartView v{};
    v.part = c->d_part; v.slot_stride = (size_t)M * tiles_all * 128; v.ld = tiles_all * 128;
    v.seg.KC = w.KC; v.seg.m_tiles = w.m_tiles; v.seg.G = w.n_tiles * w.m_tiles; v.seg.total = (int)total;
    v.mt_shift = 8;
    v.single = 1;
    *view = v;
    return SPEC_OK;
  }
  const int g_cap = aligned_ctas(tiles_all, tiles_all <= 48 ? std::min(c->gemm_ctas, c->small_gemm_ctas) : c->gemm_ctas);
  if (!plan_gemm(M, K, n_mats, rows, g_cap, &g))
    return c->fail(SPEC_E_BADARG, "unsupported linear shape");
  if (plan_part_floats(g) > c->part_floats) return c->fail(SPEC_E_NOMEM, "partial-sum scratch too small");
  StreamTmaps tm{};
  for (int i = 0; i < n_mats; ++i) {
    if (c->packed) { g.p.packed[i] = static_cast<const uint8_t*>(mats[i]); continue; }
    const CUtensorMap* t = c->tmap(mats[i], rows[i], K, 128);
    if (!t) return c->fail(SPEC_E_CUDA, "cuTensorMapEncodeTiled failed (weights)");
    tm.a[i] = *t;
  }
  const CUtensorMap* tb = c->tmap(x, std::max<size_t>(round_up(M, 16), g.MT), K, g.MT);
  if (!tb) return c->fail(SPEC_E_CUDA, "cuTensorMapEncodeTiled failed (activations)");
  tm.b = *tb;
  g.p.part = c->d_part;
  g.p.slot_stride = (size_t)M * g.p.n_tiles * 128;
  g.p.l2_prefetch = c->l2_prefetch;
  g.p.status = c->d_status;
  g.p.trace = c->next_trace(gemm_kind_name(kind));
  {
    ProfScope ps(c, kind);
    cudaError_t e = launch_gs(c->stream, c->pdl, g, tm);
    c->launches++;
    if (e != cudaSuccess) return c->fail(SPEC_E_CUDA, std::string("gemm_stream launch: ") + cudaGetErrorString(e));
  }
  *view = plan_view(g);
  return SPEC_OK;
}

// Can the cluster-reduced GEMM take this shape? One activation tile, and enough K chunks for every CTA
// of the cluster to get a run (GC_SWIGLU also needs both accumulators of the middle CTA staged at once).
bool cluster_gemm_ok(const spec_ctx* c, int mode, int M, int K) {
  const int bit = mode == GC_RESIDUAL ? 1 : (mode == GC_SWIGLU ? 2 : 4);
  if (!(c->cluster_epilogue & bit) || M < 1 || M > 128 || K % 64) return false;
  const int KC = K / 64;
  if (mode == GC_RESIDUAL) return KC >= GC_RES_CLUSTER;
  if (mode == GC_SWIGLU) return KC >= 3 && M <= 64;
  return KC >= GC_ROPE_CLUSTER && (c->cfg.head_dim == 64 || c->cfg.head_dim == 128);
}

template <int MT, int MODE>
cudaError_t launch_gc_mt(cudaStream_t st, bool pdl, int grid, const StreamTmaps& tm, const ClusterGemmParams& p, bool* attr_set) {
  if (!*attr_set) {
    cudaError_t e = cudaFuncSetAttribute(gemm_cluster<MT, MODE>, cudaFuncAttributeMaxDynamicSharedMemorySize, ClusterCfg<MT>::SMEM_BYTES);
    if (e != cudaSuccess) return e;
    *attr_set = true;
  }
  cudaLaunchConfig_t cfg{};
  cfg.gridDim = dim3(grid); cfg.blockDim = dim3(192); cfg.dynamicSmemBytes = (size_t)ClusterCfg<MT>::SMEM_BYTES; cfg.stream = st;
  cudaLaunchAttribute at[2];
  at[0].id = cudaLaunchAttributeClusterDimension;
  at[0].val.clusterDim.x = MODE == GC_RESIDUAL ? GC_RES_CLUSTER : (MODE == GC_SWIGLU ? GC_GLU_CLUSTER : GC_ROPE_CLUSTER);
  at[0].val.clusterDim.y = 1; at[0].val.clusterDim.z = 1;
  at[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  at[1].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = at;
  cfg.numAttrs = pdl ? 2 : 1;
  return cudaLaunchKernelEx(&cfg, gemm_cluster<MT, MODE>, tm, p);
}

// x[M,N] += in[M,K] * W^T (GC_RESIDUAL, mats[0] = W), act_out[M,N] = bf16(SiLU(in W_g^T) * in W_u^T)
// (GC_SWIGLU, mats = gate, up) or q / cache rows of layer `layer` = RoPE(in [W_q; W_k; W_v]^T) (GC_ROPE, mats =
// q, k, v; rows = the pass's row bookkeeping), finished inside the kernel. Caller checked cluster_gemm_ok.
int run_gemm_cluster(spec_ctx* c, int mode, const void* in, int M, int K, const void* const* mats, int N, float* x,
                     bf16* act_out, int kind, int layer = -1, const Rows* rows = nullptr) {
  const spec_config& f = c->cfg;
  const int MT = mt_for_rows(M), n_mats = mode == GC_RESIDUAL ? 1 : (mode == GC_SWIGLU ? 2 : 3);
  ClusterGemmParams p{};
  p.M = M; p.K = K; p.KC = K / 64; p.N = N;
  const int HD = f.n_heads * f.head_dim, KD = f.n_kv_heads * f.head_dim;
  StreamTmaps tm{};
  for (int i = 0; i < n_mats; ++i) {
    if (c->packed) { p.packed[i] = static_cast<const uint8_t*>(mats[i]); continue; }
    const int rws = mode == GC_ROPE ? (i == 0 ? HD : KD) : N;
    const CUtensorMap* t = c->tmap(mats[i], rws, K, 128);
    if (!t) return c->fail(SPEC_E_CUDA, "cuTensorMapEncodeTiled failed (weights)");
    tm.a[i] = *t;
  }
  const CUtensorMap* tb = c->tmap(in, std::max<size_t>(round_up(M, 16), MT), K, MT);
  if (!tb) return c->fail(SPEC_E_CUDA, "cuTensorMapEncodeTiled failed (activations)");
  tm.b = *tb;
  p.x = x; p.ss_part = mode == GC_RESIDUAL ? c->d_ss_part : nullptr; p.act = act_out; p.status = c->d_status;
  int n_tiles = (N + 127) / 128;
  if (mode == GC_ROPE) {
    const int tq = (HD + 127) / 128, tk = (KD + 127) / 128;
    p.tile0[0] = 0; p.tile0[1] = tq; p.tile0[2] = tq + tk;
    n_tiles = tq + 2 * tk;
    p.H = f.n_heads; p.layer = layer; p.rows = *rows; p.cs = c->d_rope; p.q = static_cast<bf16*>(c->d_q);
    p.pool = static_cast<bf16*>(c->d_pool); p.g = c->geom; p.page_table = c->d_page_table;
  }
  p.trace = c->next_trace(gemm_kind_name(kind));
  const int grid = n_tiles * (mode == GC_RESIDUAL ? GC_RES_CLUSTER : (mode == GC_SWIGLU ? GC_GLU_CLUSTER : GC_ROPE_CLUSTER));
  cudaError_t e = cudaErrorInvalidValue;
  {
    ProfScope ps(c, kind);
    bool* as = c->gc_attr_set;
    if (mode == GC_RESIDUAL) {
      switch (MT) {
        case 16: e = launch_gc_mt<16, GC_RESIDUAL>(c->stream, c->pdl, grid, tm, p, as + 0); break;
        case 32: e = launch_gc_mt<32, GC_RESIDUAL>(c->stream, c->pdl, grid, tm, p, as + 1); break;
        case 64: e = launch_gc_mt<64, GC_RESIDUAL>(c->stream, c->pdl, grid, tm, p, as + 2); break;
        default: e = launch_gc_mt<128, GC_RESIDUAL>(c->stream, c->pdl, grid, tm, p, as + 3); break;
      }
    } else if (mode == GC_SWIGLU) {
      switch (MT) {
        case 16: e = launch_gc_mt<16, GC_SWIGLU>(c->stream, c->pdl, grid, tm, p, as + 4); break;
        case 32: e = launch_gc_mt<32, GC_SWIGLU>(c->stream, c->pdl, grid, tm, p, as + 5); break;
        default: e = launch_gc_mt<64, GC_SWIGLU>(c->stream, c->pdl, grid, tm, p, as + 6); break;
      }
    } else {
      switch (MT) {
        case 16: e = launch_gc_mt<16, GC_ROPE>(c->stream, c->pdl, grid, tm, p, as + 7); break;
        case 32: e = launch_gc_mt<32, GC_ROPE>(c->stream, c->pdl, grid, tm, p, as + 8); break;
        case 64: e = launch_gc_mt<64, GC_ROPE>(c->stream, c->pdl, grid, tm, p, as + 9); break;
        default: e = launch_gc_mt<128, GC_ROPE>(c->stream, c->pdl, grid, tm, p, as + 10); break;
      }
    }
    c->launches++;
  }
  if (e != cudaSuccess) return c->fail(SPEC_E_CUDA, std::string("gemm_cluster launch: ") + cudaGetErrorString(e));
  return SPEC_OK;
}

template <typename T>
int linear_simple(spec_ctx* c, const T* x, int ldx, const T* W, float* y, int ldy, int M, int N, int K) {
  constexpr int MC = 8;
  dim3 grid((N + 7) / 8, (M + MC - 1) / MC);
  linear_rows<T, MC><<<grid, 256, 0, c->stream>>>(x, ldx, W, y, ldy, M, N, K);
  LAUNCH_CHECK("linear_rows");
  return SPEC_OK;
}

#define KLAUNCH(name, kernel, grid, block, smem, ...)                                            \
  do {                                                                                         \
    cudaError_t e_ = launch_k(c->pdl, kernel, grid, block, smem, c->stream, __VA_ARGS__, c->next_trace(name)); \
    c->launches++;                                                                             \
    if (e_ != cudaSuccess) return c->fail(SPEC_E_CUDA, std::string(name) + ": " + cudaGetErrorString(e_)); \
  } while (0)

// Passes with several 16-row blocks whose (sequence, head, row block) CTAs fit the SMs in one wave
// use the kernel that needs no merge across CTAs and no length-dependent launch shape.
bool attn_rows_mode(const spec_ctx* c, int R) {
  const int nw = (R + 15) / 16;
  return nw > 1 && c->cfg.n_heads * c->B * nw <= SM_SLOTS / 2;
}

// Context length from which a pass of R rows goes to the long-context kernels: the option's value, but at most
// ATTN_WAVES_KEYS for passes of more than 32 rows whose (sequence, head, 16-row block) CTAs do not fit one wave
// (batched verification): there the tcgen05 kernel, one CTA per (sequence, head, 64 rows), already wins.
constexpr int ATTN_WAVES_KEYS = 512;
int attn_long_threshold(const spec_ctx* c, int R) {
  const bool umma = c->attn_umma && c->tm_kv_ok && c->cfg.head_dim == 128;
  if (c->long_attn_keys > 0 && umma && R > 32 && !attn_rows_mode(c, R)) return std::min(c->long_attn_keys, ATTN_WAVES_KEYS);
  return c->long_attn_keys;
}
// Passes of more than 32 rows (any pass with the tcgen05 kernel) over a context that may exceed that length.
bool attn_long_mode(const spec_ctx* c, int R, int keys_hi) {
  const bool umma = c->attn_umma && c->tm_kv_ok && c->cfg.head_dim == 128;
  const int thr = attn_long_threshold(c, R);
  return thr > 0 && (R > 32 || umma) && keys_hi > thr;
}

// n_hi_pass / n_lo_pass: host bounds of the cached length the pass's rows sit on, per sequence
// (n_lo_pass may be null: nothing is fetched before the dependency wait).
int launch_attention_tc(spec_ctx* c, const Rows& rows, int R, int l, const int* n_hi_pass, const int* n_lo_pass) {
  const spec_config& f = c->cfg;
  int H = f.n_heads, D = f.head_dim;
  AttnTcArgs a{};
  a.q = static_cast<const bf16*>(c->d_q); a.part_o = c->d_part_o; a.part_ml = c->d_part_ml;
  a.pool = static_cast<const bf16*>(c->d_pool); a.g = c->geom; a.page_table = c->d_page_table; a.rows = rows;
  a.layer = l; a.H = H; a.scale_log2 = 1.4426950408889634f / sqrtf((float)D);
  a.out = static_cast<bf16*>(c->d_attn); a.arrive = c->d_attn_arrive;
  a.status = c->d_status;
  int tiles_hi = 1;
  for (int b = 0; b < c->B; ++b) {
    tiles_hi = std::max(tiles_hi, (n_hi_pass[b] + R + 63) / 64);
    if (b < ATTN_MAX_SEQS) a.n_lo[b] = n_lo_pass ? n_lo_pass[b] : 0;
  }
  const int nw = (R + 15) / 16;
  if (attn_long_mode(c, R, tiles_hi * 64) && c->attn_umma && c->tm_kv_ok && D == 128) {
    // long contexts: scores and P V on tcgen05, a CTA per (head, 64 rows, key split)
    const int halves = (R + AU_ROWS - 1) / AU_ROWS;
    if (c->B <= ATTN_MAX_SEQS) {
      int idx[ATTN_MAX_SEQS];
      for (int b = 0; b < c->B; ++b) idx[b] = b;
      // (the host's current bounds, not the bounds the launch is planned for: those are the same for all)
      const int* len = (int)c->n_hi.size() >= c->B ? c->n_hi.data() : n_hi_pass;
      std::stable_sort(idx, idx + c->B, [&](int x, int y) { return len[x] > len[y]; });
      for (int b = 0; b < c->B; ++b) a.order[b] = (unsigned char)idx[b];
    }
    // the key splits of a (sequence, row half, head) are one cluster: one CTA per SM, at most a wave of them
    a.nsplit = std::max(1, std::min(std::min(c->nsplit_attn, AU_MAX_CLUSTER), (SM_SLOTS / 2) / (H * c->B * halves)));
    dim3 grid(H, a.nsplit, c->B * halves);
    ProfScope ps_attn(c, SPEC_PROFILE_ATTENTION);
    static bool set_dev[kAttrDevices] = {};
    bool& set_ = *attr_flag(set_dev);
    if (!set_) { CUDA_OK(cudaFuncSetAttribute(attention_umma<128>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)attention_umma_smem())); set_ = true; }
    cudaLaunchConfig_t cfg{};
    cfg.gridDim = grid; cfg.blockDim = dim3(AU_THREADS); cfg.dynamicSmemBytes = attention_umma_smem(); cfg.stream = c->stream;
    cudaLaunchAttribute at[2];
    int n_at = 0;
    if (a.nsplit > 1) {
      at[n_at].id = cudaLaunchAttributeClusterDimension;
      at[n_at].val.clusterDim.x = 1; at[n_at].val.clusterDim.y = (unsigned)a.nsplit; at[n_at].val.clusterDim.z = 1;
      ++n_at;
    }
    if (c->pdl) {
      at[n_at].id = cudaLaunchAttributeProgrammaticStreamSerialization;
      at[n_at].val.programmaticStreamSerializationAllowed = 1;
      ++n_at;
    }
    cfg.attrs = at; cfg.numAttrs = (unsigned)n_at;
    cudaError_t e_ = cudaLaunchKernelEx(&cfg, attention_umma<128>, c->tm_kv, a, c->next_trace("attention_tc"));
    c->launches++;
    if (e_ != cudaSuccess) return c->fail(SPEC_E_CUDA, std::string("attention_umma: ") + cudaGetErrorString(e_));
    return SPEC_OK;
  }
  if (attn_long_mode(c, R, tiles_hi * 64) && R > 32) {
    // long contexts, more than 32 rows: K/V tiles shared by the row blocks of a CTA, keys split across CTAs
    const int halves = (R + AS_RB * 16 - 1) / (AS_RB * 16);
    a.nsplit = std::max(1, std::min(c->nsplit_attn, (SM_SLOTS / 2) / (H * c->B * halves)));
    a.stages = AS_NB; a.split_tiles = AS_SPLIT_SUB;
    dim3 grid(H, a.nsplit, c->B * halves);
    ProfScope ps_attn(c, SPEC_PROFILE_ATTENTION);
    static bool set_dev[2][kAttrDevices] = {};
    bool& set_ = *attr_flag(set_dev[D == 128 ? 0 : 1]);
    if (D == 128) {
      if (!set_) { CUDA_OK(cudaFuncSetAttribute(attention_shared<128>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)attention_shared_smem(128))); set_ = true; }
      KLAUNCH("attention_tc", (attention_shared<128>), grid, dim3(AS_RB * AS_KP * 32), attention_shared_smem(128), a);
    } else {
      if (!set_) { CUDA_OK(cudaFuncSetAttribute(attention_shared<64>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)attention_shared_smem(64))); set_ = true; }
      KLAUNCH("attention_tc", (attention_shared<64>), grid, dim3(AS_RB * AS_KP * 32), attention_shared_smem(64), a);
    }
    return SPEC_OK;
  }
  if (attn_rows_mode(c, R)) {
    // few sequences: a CTA per (head, 16 query rows) walks the whole context, whatever its length
    a.nsplit = 1; a.stages = 2; a.split_tiles = 1;
    dim3 grid(H, nw, c->B);
    ProfScope ps_attn(c, SPEC_PROFILE_ATTENTION);
    if (D == 128) {
      static bool set_dev[kAttrDevices] = {};
      bool& set_ = *attr_flag(set_dev);
      if (!set_) { CUDA_OK(cudaFuncSetAttribute(attention_rows<128, ATTN_ROWS_WARPS>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)attention_rows_smem(128, ATTN_ROWS_WARPS))); set_ = true; }
      KLAUNCH("attention_tc", (attention_rows<128, ATTN_ROWS_WARPS>), grid, dim3(ATTN_ROWS_WARPS * 32), attention_rows_smem(128, ATTN_ROWS_WARPS), a);
    } else {
      static bool set_dev[kAttrDevices] = {};
      bool& set_ = *attr_flag(set_dev);
      if (!set_) { CUDA_OK(cudaFuncSetAttribute(attention_rows<64, ATTN_ROWS_WARPS>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)attention_rows_smem(64, ATTN_ROWS_WARPS))); set_ = true; }
      KLAUNCH("attention_tc", (attention_rows<64, ATTN_ROWS_WARPS>), grid, dim3(ATTN_ROWS_WARPS * 32), attention_rows_smem(64, ATTN_ROWS_WARPS), a);
    }
    return SPEC_OK;
  }
  // more sequences: one CTA per (sequence, head) and KV split, all query rows. Short contexts (host
  // bound of at most ATTN_SINGLE_TILES tiles) get one split and no merge step; longer ones as many
  // split CTAs as fit beside each other, of which the kernel uses min(that, tiles / split_tiles)
  const int slots1 = std::max(1, std::min(c->nsplit_attn, (SM_SLOTS / 2) / (H * c->B)));
  a.nsplit = tiles_hi <= ATTN_SINGLE_TILES ? 1 : slots1;
  a.split_tiles = ATTN_SPLIT_TILES;
  a.stages = 4;
  dim3 grid(H, a.nsplit, c->B);
#define ATTN_CASE(HDV, NWV, KGV)                                                                         \
  {                                                                                                    \
    size_t sm = attention_tc_smem(HDV, NWV, a.stages);                                                 \
    static bool set_dev[kAttrDevices] = {};                                                            \
    bool& set_ = *attr_flag(set_dev);                                                                  \
    if (!set_) { CUDA_OK(cudaFuncSetAttribute(attention_tc<HDV, NWV, KGV>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)attention_tc_smem(HDV, NWV, ATTN_MAX_STAGES))); set_ = true; } \
    KLAUNCH("attention_tc", (attention_tc<HDV, NWV, KGV>), grid, dim3(NWV * KGV * 32), sm, a);         \
  }
  {
    // up to 64 rows: two key groups of warps per CTA; more rows: one
    ProfScope ps_attn(c, SPEC_PROFILE_ATTENTION);
    if (D == 128) {
      if (nw <= 1) ATTN_CASE(128, 1, 2) else if (nw <= 2) ATTN_CASE(128, 2, 2) else if (nw <= 4) ATTN_CASE(128, 4, 2) else ATTN_CASE(128, 8, 1)
    } else {
      if (nw <= 1) ATTN_CASE(64, 1, 2) else if (nw <= 2) ATTN_CASE(64, 2, 2) else if (nw <= 4) ATTN_CASE(64, 4, 2) else ATTN_CASE(64, 8, 1)
    }
  }
#undef ATTN_CASE
  return SPEC_OK;
}

// One pass of the base model over M = B*R rows whose tokens/positions/slots are prepared and
// whose embeddings are in d_x: bf16 tensor-core path. Leaves the final hidden state in d_hid
// (float32) and d_hq (bf16).
int forward_layers_tc(spec_ctx* c, int R, bool chain, const int* n_hi_pass, const int* n_lo_pass) {
  const spec_config& f = c->cfg;
  Rows rows = make_rows(c, R, chain);
  const int M = c->B * R, d = f.d_model, F = f.d_ffn, H = f.n_heads, D = f.head_dim, HD = H * D, KD = f.n_kv_heads * D;
  bf16* u = static_cast<bf16*>(c->d_u);
  bf16* act = static_cast<bf16*>(c->d_act);
  const int kp0 = (HD + 127) / 128 * 128, vp0 = kp0 + (KD + 127) / 128 * 128;   // padded columns of k and v in the QKV partials
  const int up0 = (F + 127) / 128 * 128;                                        // and of the up projection
  // (passes of more than 128 rows are bound by bandwidth, not by a row's latency: one plain CTA per row)
  // (after a residual cluster epilogue the pieces' sums of squares exist already: ss_ready)
  bool ss_ready = false;
  const int n_ss = ((d + 127) / 128) * GC_RES_CLUSTER;
#define NORM_LAUNCH(pv, gain, uq, hid)                                                                   \
  if (ss_ready && M <= 128) {                                                                            \
    KLAUNCH("norm_reduce_tc", norm_scaled_tc, dim3(M, NORM_CLUSTER), dim3(NORM_THREADS), 0, (const float*)c->d_x, (const float*)c->d_ss_part, n_ss, gain, f.rms_eps, uq, hid, d); \
  } else if (M > 128) {                                                                                         \
    KLAUNCH("norm_reduce_tc", norm_rows_wide, dim3(M), dim3(NORMW_THREADS), 0, c->d_x, pv, gain, f.rms_eps, uq, hid, d); \
  } else {                                                                                               \
    KLAUNCH("norm_reduce_tc", norm_reduce_tc, dim3(M, NORM_CLUSTER), dim3(NORM_THREADS), 0, c->d_x, pv, gain, f.rms_eps, uq, hid, d); \
  }
  PartView pend{};              // partial sums of the previous down-projection still to be added to x
  for (int l = 0; l < f.n_layers; ++l) {
    NORM_LAUNCH(pend, c->an[l], u, (float*)nullptr);
    int r;
    {
      const void* mats[3] = {c->wq[l], c->wk[l], c->wv[l]};
      int rws[3] = {HD, KD, KD};
      if (cluster_gemm_ok(c, GC_ROPE, M, d)) {
        // the clusters rotate q and k and store q and the cache rows themselves
        if ((r = run_gemm_cluster(c, GC_ROPE, u, M, d, mats, 0, nullptr, nullptr, SPEC_PROFILE_QKV, l, &rows))) return r;
      } else {
        PartView vq{};
        if ((r = run_gemm(c, u, M, d, 3, mats, rws, SPEC_PROFILE_QKV, &vq))) return r;
        KLAUNCH("rope_store_tc", rope_store_tc, dim3(M, M <= 128 ? 8 : 2), dim3(256), 0, vq, 0, kp0, vp0, rows, c->d_rope,
                static_cast<bf16*>(c->d_q), static_cast<bf16*>(c->d_pool), c->geom, c->d_page_table, l, H);
      }
    }
    if ((r = launch_attention_tc(c, rows, R, l, n_hi_pass, n_lo_pass))) return r;
    PartView vo{};
    {
      const void* mats[1] = {c->wo[l]};
      int rws[1] = {d};
      if (cluster_gemm_ok(c, GC_RESIDUAL, M, HD)) {
        // the cluster adds its split-K sums and the residual stream itself: nothing left for the norm kernel to add
        if ((r = run_gemm_cluster(c, GC_RESIDUAL, c->d_attn, M, HD, mats, d, c->d_x, nullptr, SPEC_PROFILE_WO))) return r;
        ss_ready = true;
      } else {
        ss_ready = false;
        if ((r = run_gemm(c, c->d_attn, M, HD, 1, mats, rws, SPEC_PROFILE_WO, &vo))) return r;
      }
    }
    NORM_LAUNCH(vo, c->fn[l], u, (float*)nullptr);
    {
      const void* mats[2] = {c->wg[l], c->wu[l]};
      int rws[2] = {F, F};
      if (cluster_gemm_ok(c, GC_SWIGLU, M, d)) {
        if ((r = run_gemm_cluster(c, GC_SWIGLU, u, M, d, mats, F, nullptr, act, SPEC_PROFILE_GATE_UP))) return r;
      } else {
        PartView vg{};
        if ((r = run_gemm(c, u, M, d, 2, mats, rws, SPEC_PROFILE_GATE_UP, &vg))) return r;
        size_t total = (size_t)M * (F / 4);
        unsigned blocks = (unsigned)std::min<size_t>((total + 255) / 256, 2 * SM_SLOTS);
        KLAUNCH("swiglu_reduce_tc", swiglu_reduce_tc, dim3(blocks), dim3(256), 0, vg, 0, up0, act, M, F);
      }
    }
    {
      const void* mats[1] = {c->wd[l]};
      int rws[1] = {d};
      pend = PartView{};
      if (cluster_gemm_ok(c, GC_RESIDUAL, M, F)) {
        if ((r = run_gemm_cluster(c, GC_RESIDUAL, act, M, F, mats, d, c->d_x, nullptr, SPEC_PROFILE_DOWN))) return r;
        ss_ready = true;
      } else {
        ss_ready = false;
        if ((r = run_gemm(c, act, M, F, 1, mats, rws, SPEC_PROFILE_DOWN, &pend))) return r;
      }
    }
  }
  NORM_LAUNCH(pend, c->final_norm, static_cast<bf16*>(c->d_hq), c->d_hid);
#undef NORM_LAUNCH
  return SPEC_OK;
}

// The same pass with the plain CUDA-core kernels (float32 configurations and the bf16 debug mode).
template <typename T>
int forward_layers(spec_ctx* c, int R, bool chain, const int* n_hi_pass, const int* n_lo_pass) {
  if (c->tc) return forward_layers_tc(c, R, chain, n_hi_pass, n_lo_pass);
  const spec_config& f = c->cfg;
  Rows rows = make_rows(c, R, chain);
  int M = c->B * R, d = f.d_model, F = f.d_ffn, H = f.n_heads, D = f.head_dim, HD = H * D;
  T* u = static_cast<T*>(c->d_u);
  T* q = static_cast<T*>(c->d_q);
  T* attn = static_cast<T*>(c->d_attn);
  T* act = static_cast<T*>(c->d_act);
  T* pool = static_cast<T*>(c->d_pool);
  int pending = 0;              // 1: the previous down-projection output is still to be added to x
  for (int l = 0; l < f.n_layers; ++l) {
    rmsnorm_rows<T><<<M, 256, 0, c->stream>>>(c->d_x, c->d_part, pending, (size_t)M * d, c->an[l], f.rms_eps, u, nullptr, d);
    LAUNCH_CHECK("rmsnorm_rows");
    int nk = f.n_kv_heads * D, r;
    if ((r = linear_simple<T>(c, u, d, static_cast<const T*>(c->wq[l]), c->d_part, c->Nqkv, M, HD, d))) return r;
    if ((r = linear_simple<T>(c, u, d, static_cast<const T*>(c->wk[l]), c->d_part + HD, c->Nqkv, M, nk, d))) return r;
    if ((r = linear_simple<T>(c, u, d, static_cast<const T*>(c->wv[l]), c->d_part + HD + nk, c->Nqkv, M, nk, d))) return r;
    rope_store<T><<<M, 256, 0, c->stream>>>(c->d_part, 1, (size_t)M * c->Nqkv, rows, c->d_rope, q, pool, c->geom, c->d_page_table, l, H);
    LAUNCH_CHECK("rope_store");
    {
      dim3 grid(H, c->B, (R + 3) / 4);
      attention_simple<T><<<grid, 128, 0, c->stream>>>(q, attn, pool, c->geom, c->d_page_table, rows, l, H, 1.0f / sqrtf((float)D));
      LAUNCH_CHECK("attention_simple");
    }
    if ((r = linear_simple<T>(c, attn, HD, static_cast<const T*>(c->wo[l]), c->d_part, d, M, d, HD))) return r;
    rmsnorm_rows<T><<<M, 256, 0, c->stream>>>(c->d_x, c->d_part, 1, (size_t)M * d, c->fn[l], f.rms_eps, u, nullptr, d);
    LAUNCH_CHECK("rmsnorm_rows");
    {
      float* g = c->d_part;
      float* up = c->d_part + (size_t)M * F;
      if ((r = linear_simple<T>(c, u, d, static_cast<const T*>(c->wg[l]), g, F, M, F, d))) return r;
      if ((r = linear_simple<T>(c, u, d, static_cast<const T*>(c->wu[l]), up, F, M, F, d))) return r;
      size_t total = (size_t)M * F;
      swiglu_rows<T><<<(unsigned)((total + 255) / 256), 256, 0, c->stream>>>(g, up, act, total);
      LAUNCH_CHECK("swiglu_rows");
    }
    if ((r = linear_simple<T>(c, act, F, static_cast<const T*>(c->wd[l]), c->d_part, d, M, d, F))) return r;
    pending = 1;
  }
  // final norm: hidden (float32) and its operand-typed copy
  rmsnorm_rows<T><<<M, 256, 0, c->stream>>>(c->d_x, c->d_part, pending, (size_t)M * d, c->final_norm, f.rms_eps,
                                            static_cast<T*>(c->d_hq), c->d_hid, d);
  LAUNCH_CHECK("rmsnorm_rows");
  return SPEC_OK;
}

// Extra decoding heads on the tensor cores: residual blocks (head matrices stacked along the
// output dimension, up to four per launch), shared lm_head, per-head top-k.
int heads_tc(spec_ctx* c, const int* ov) {
  const spec_config& f = c->cfg;
  const int B = c->B, K = c->K, d = f.d_model, kmax = c->kmax, rows_total = B * K;
  const int dpad = (d + 127) / 128 * 128;
  for (int k0 = 0; k0 < K; k0 += GS_MAX_MATS) {
    const int nk = std::min(GS_MAX_MATS, K - k0);
    const void* mats[GS_MAX_MATS];
    int rws[GS_MAX_MATS];
    for (int i = 0; i < nk; ++i) { mats[i] = c->mw[k0 + i]; rws[i] = d; }
    PartView pv{};
    int r = run_gemm(c, c->d_hq_last, B, d, nk, mats, rws, SPEC_PROFILE_OFF, &pv);
    if (r) return r;
    KLAUNCH("medusa_act_tc", medusa_act_tc, dim3(B * nk, 4), dim3(256), 0, pv, dpad, (const bf16*)c->d_hq_last,
            reinterpret_cast<const bf16* const*>(c->d_mb), static_cast<bf16*>(c->d_r), K, k0, nk, d);
  }
  PartView pl{};
  {
    const void* mats[1] = {c->lm_head};
    int rws[1] = {f.vocab};
    int r = run_gemm(c, c->d_r, rows_total, d, 1, mats, rws, SPEC_PROFILE_OFF, &pl);
    if (r) return r;
  }
  // the row's last-arriving CTA merges the slices' lists: no merge kernel
  const size_t sm_topk = std::max((size_t)c->topk_slice * sizeof(float), (size_t)c->topk_blocks * kmax * 8);
  if (sm_topk > 48 * 1024) return c->fail(SPEC_E_BADARG, "top-k lists do not fit the merge's shared memory");
  KLAUNCH("topk_slices_tc", topk_slices_tc, dim3(c->topk_blocks, rows_total), dim3(256), sm_topk,
          pl, f.vocab, rows_total, c->topk_slice, kmax, c->d_pk_val, c->d_pk_idx, c->d_row_arrive, K, (const int*)c->d_root, ov, c->d_cand);
  return SPEC_OK;
}

// lm_head over `M` operand rows at `src`, leaving per-row argmax partials (and logits).
template <typename T>
int lm_head_argmax(spec_ctx* c, const T* src, int M) {
  const spec_config& f = c->cfg;
  if (c->tc) {
    PartView pl{};
    const void* mats[1] = {c->lm_head};
    int rws[1] = {f.vocab};
    int r = run_gemm(c, src, M, f.d_model, 1, mats, rws, SPEC_PROFILE_OFF, &pl);
    if (r) return r;
    const int NSL = c->ntile_lm;
    KLAUNCH("argmax_partials_tc", argmax_partials_tc, dim3(M, NSL), dim3(256), 0, pl, f.vocab,
            c->keep_logits ? c->d_logits : (float*)nullptr, c->d_pval, c->d_pidx, c->d_row_arrive, c->d_pval2, c->d_pidx2);
  } else {
    int r = linear_simple<T>(c, src, f.d_model, static_cast<const T*>(c->lm_head), c->d_logits, f.vocab, M, f.vocab, f.d_model);
    if (r) return r;
    argmax_rows<<<M, 256, 0, c->stream>>>(c->d_logits, f.vocab, c->d_pval, c->d_pidx);
    LAUNCH_CHECK("argmax_rows");
  }
  return SPEC_OK;
}

AcceptArgs make_accept(spec_ctx* c, int R, int mode) {
  AcceptArgs a{};
  a.rows = make_rows(c, R, false);
  a.pval = c->tc ? c->d_pval2 : c->d_pval; a.pidx = c->tc ? c->d_pidx2 : c->d_pidx; a.ntile = 1;
  a.hq_last = c->tc ? static_cast<bf16*>(c->d_hq_last) : nullptr;
  a.parent = c->d_parent; a.depth = c->d_depth; a.edge_ok = nullptr;
  a.K = c->K; a.frag_token = c->cfg.frag_token; a.d = c->cfg.d_model; a.mode = mode;
  a.hid = c->d_hid; a.am = c->d_am; a.path = c->d_path; a.count = c->d_count; a.out_tok = c->d_out_tok;
  a.n_old = c->d_n_old; a.root_tok = c->d_root; a.h_last = c->d_h_last;
  a.gen_log = c->d_gen_log; a.gen_cnt = c->d_gen_cnt; a.gen_cap = c->gen_cap;
  return a;
}

int check_status(spec_ctx* c) {
  int st[4];
  cudaError_t e = cudaMemcpyAsync(st, c->d_status, sizeof(st), cudaMemcpyDeviceToHost, c->stream);
  if (e == cudaSuccess) e = cudaStreamSynchronize(c->stream);
  if (e != cudaSuccess) return c->fail(SPEC_E_CUDA, std::string("status read: ") + cudaGetErrorString(e));
  if (st[0] == ST_OK) return SPEC_OK;
  char buf[128];
  snprintf(buf, sizeof(buf), "device status %d at %d (detail %d)", st[0], st[1], st[2]);
  return c->fail(st[0] == ST_TIMEOUT ? SPEC_E_TIMEOUT : (st[0] == ST_SEQLEN ? SPEC_E_SEQLEN : SPEC_E_BADARG), buf);
}

template <typename T>
int prefill_t(spec_ctx* c, int batch, const int32_t* tokens, const int32_t* offsets) {
  const spec_config& f = c->cfg;
  int maxlen = 0;
  for (int b = 0; b < batch; ++b) {
    int len = offsets[b + 1] - offsets[b];
    if (len < 1) return c->fail(SPEC_E_BADARG, "empty prompt");
    if (len + c->K + 1 > f.max_seq) return c->fail(SPEC_E_SEQLEN, "prompt leaves no room to generate within max_seq");
    if (offsets[b + 1] - offsets[0] > batch * f.max_seq) return c->fail(SPEC_E_SEQLEN, "prompts exceed the prompt buffer");
    maxlen = std::max(maxlen, len);
  }
  c->B = batch;
  c->prefilled = false;
  c->graph_epoch++;   // recorded steps were planned for the previous sequences
  std::vector<int> off(batch + 1);
  for (int b = 0; b <= batch; ++b) off[b] = offsets[b] - offsets[0];
  CUDA_OK(cudaMemsetAsync(c->d_status, 0, 4 * sizeof(int), c->stream));
  CUDA_OK(cudaMemsetAsync(c->d_pool, 0, (size_t)f.max_batch * c->pages_per_seq * c->geom.page_elems() * c->esz, c->stream));
  CUDA_OK(cudaMemcpyAsync(c->d_prompt, tokens + offsets[0], (size_t)off[batch] * sizeof(int), cudaMemcpyHostToDevice, c->stream));
  CUDA_OK(cudaMemcpyAsync(c->d_offsets, off.data(), (batch + 1) * sizeof(int), cudaMemcpyHostToDevice, c->stream));
  CUDA_OK(cudaMemsetAsync(c->d_gen_cnt, 0, batch * sizeof(int), c->stream));
  CUDA_OK(cudaMemsetAsync(c->d_draws, 0, batch * sizeof(int), c->stream));
  CUDA_OK(cudaStreamSynchronize(c->stream));   // host staging vector goes out of scope below
  int R = PREFILL_ROWS, M = batch * R;
  Rows rows = make_rows(c, R, true);
  int chunks = (maxlen + R - 1) / R;
  for (int ch = 0; ch < chunks; ++ch) {
    prepare_prefill_rows<T><<<M, 128, 0, c->stream>>>(rows, c->d_prompt, c->d_offsets, ch, static_cast<const T*>(c->embed), c->d_x,
                                                    f.d_model, f.vocab, c->d_status);
    LAUNCH_CHECK("prepare_prefill_rows");
    std::vector<int> n_pass(batch);
    for (int b = 0; b < batch; ++b) n_pass[b] = std::min(offsets[b + 1] - offsets[b], ch * R);
    int r = forward_layers<T>(c, R, true, n_pass.data(), nullptr);
    if (r) return r;
    prefill_keep_last<T><<<batch, 256, 0, c->stream>>>(rows, c->d_offsets, ch, c->d_hid, c->d_h_last, static_cast<T*>(c->d_hq_last), f.d_model);
    LAUNCH_CHECK("prefill_keep_last");
  }
  int r = lm_head_argmax<T>(c, static_cast<const T*>(c->d_hq_last), batch);
  if (r) return r;
  AcceptArgs a = make_accept(c, 1, 1);
  KLAUNCH("accept_kernel", accept_kernel, dim3(batch), dim3(256), 0, a);
  if (f.sampling) {
    sample_root<<<batch, 256, 0, c->stream>>>(c->d_logits, f.vocab, 1, c->K, c->d_path, c->d_count, f.temperature, f.seed_lo,
                                              f.seed_hi, c->d_draws, c->d_root, 1);
    LAUNCH_CHECK("sample_root");
  }
  r = check_status(c);
  if (r) return r;
  c->n_hi.assign(batch, 0);
  for (int b = 0; b < batch; ++b) c->n_hi[b] = offsets[b + 1] - offsets[b];
  c->n_lo = c->n_hi;
  c->n_copy_pending = false;
  c->prefilled = true;
  return SPEC_OK;
}

// Phase boundary i of the step (only with SPEC_OPT_PHASE_TIMING: an event between two kernels costs the
// programmatic overlap of that pair): an event record, an external-event node while the step is captured.
void step_event(spec_ctx* c, int i) {
  if (!c->phase_timing) return;
  if (c->capturing) cudaEventRecordWithFlags(c->phase_ev[i], c->stream, cudaEventRecordExternal);
  else cudaEventRecord(c->phase_ev[i], c->stream);
}

// Enqueues the kernels of one step (or records them, when the stream is capturing). ov: device
// candidate overrides or null; n_hi_plan / n_lo_plan: the length bounds the attention launches are planned for.
template <typename T>
int step_body(spec_ctx* c, const int* ov, const int* n_hi_plan, const int* n_lo_plan) {
  const spec_config& f = c->cfg;
  int B = c->B, K = c->K, T_ = c->T, d = f.d_model, kmax = c->kmax;
  step_event(c, 0);
  // (1) extra heads -> shared lm_head -> per-head top-k -> candidate table
  if (K > 0 && c->tc) {
    int r = heads_tc(c, ov);
    if (r) return r;
  } else if (K > 0) {
    constexpr int MC = 4;
    dim3 g1((K * d + 7) / 8, (B + MC - 1) / MC);
    KLAUNCH("medusa_resblock", (medusa_resblock<T, MC>), g1, dim3(256), 0, (const float*)c->d_h_last,
            reinterpret_cast<const T* const*>(c->d_mw), reinterpret_cast<const T* const*>(c->d_mb), static_cast<T*>(c->d_r), B, K, d);
    int rows_total = B * K;
    dim3 g2(c->topk_blocks, (rows_total + MC - 1) / MC);
    size_t sm = (size_t)MC * c->topk_slice * sizeof(float);
    KLAUNCH("medusa_lmhead_topk", (medusa_lmhead_topk<T, MC>), g2, dim3(256), sm, static_cast<const T*>(c->d_r),
            static_cast<const T*>(c->lm_head), rows_total, f.vocab, d, c->topk_slice, kmax, c->d_pk_val, c->d_pk_idx);
    // partial lists of the row chunks are laid out per block over all rows
    size_t sm2 = (size_t)c->topk_blocks * kmax * 8 + (size_t)c->topk_blocks * 4;
    KLAUNCH("topk_merge", topk_merge, dim3(rows_total), dim3(256), sm2, (const float*)c->d_pk_val, (const int*)c->d_pk_idx,
            c->topk_blocks, rows_total, K, kmax, (const int*)c->d_root, ov, c->d_cand);
  } else {
    CUDA_OK(cudaMemcpyAsync(c->d_cand, c->d_root, B * sizeof(int), cudaMemcpyDeviceToDevice, c->stream));
  }
  step_event(c, 1);
  // (2) candidate tree -> rows
  int M = B * T_;
  Rows rows = make_rows(c, T_, false);
  KLAUNCH("prepare_verify_rows", prepare_verify_rows<T>, dim3(M), dim3(128), 0, rows, (const int*)c->d_cand, (K + 1) * kmax, kmax,
          (const int*)c->d_depth, (const int*)c->d_rank, c->cap, static_cast<const T*>(c->embed), c->d_x, d, f.vocab, c->d_status);
  step_event(c, 2);
  // (3) verification forward
  int r = forward_layers<T>(c, T_, false, n_hi_plan, n_lo_plan);
  if (r) return r;
  r = lm_head_argmax<T>(c, static_cast<const T*>(c->d_hq), M);
  if (r) return r;
  step_event(c, 3);
  // (4) acceptance
  AcceptArgs a = make_accept(c, T_, 0);
  if (f.accept_mode == 1) {
    typical_edges<<<M, 256, 0, c->stream>>>(c->d_logits, f.vocab, rows, c->d_parent, f.typ_eps, f.typ_delta,
                                            1.0f / (f.temperature > 0.f ? f.temperature : 1.0f), c->d_edge);
    LAUNCH_CHECK("typical_edges");
    a.edge_ok = c->d_edge;
  }
  KLAUNCH("accept_kernel", accept_kernel, dim3(B), dim3(256), 0, a);
  if (f.sampling) {
    sample_root<<<B, 256, 0, c->stream>>>(c->d_logits, f.vocab, T_, K, c->d_path, c->d_count, f.temperature, f.seed_lo,
                                          f.seed_hi, c->d_draws, c->d_root, 0);
    LAUNCH_CHECK("sample_root");
  }
  step_event(c, 4);
  // (5) KV compaction
  dim3 gc(f.n_layers * 2 * f.n_kv_heads, B);
  KLAUNCH("compact_kv", compact_kv<T>, gc, dim3(64), 0, static_cast<T*>(c->d_pool), c->geom, (const int*)c->d_page_table,
          (const int*)c->d_path, (const int*)c->d_count, (const int*)c->d_n_old, K);
  step_event(c, 5);
  return SPEC_OK;
}

template <typename T>
int step_t(spec_ctx* c, int32_t* out_tokens, int32_t* out_counts, const int32_t* cand_override) {
  const spec_config& f = c->cfg;
  int B = c->B, K = c->K, T_ = c->T, d = f.d_model, kmax = c->kmax;
  for (int b = 0; b < B; ++b)
    if (c->n_hi[b] + K + 1 > f.max_seq) return c->fail(SPEC_E_SEQLEN, "sequence would exceed max_seq");
  for (int i = 0; i < 6; ++i)
    if (!c->phase_ev[i]) CUDA_OK(cudaEventCreate(&c->phase_ev[i]));
  c->prof_used = 0;
  if (c->trace_on) {
    c->trace_n = 0;
    c->trace_names.clear();
    CUDA_OK(cudaMemcpyAsync(c->d_trace, c->trace_init.data(), c->trace_init.size() * 8, cudaMemcpyHostToDevice, c->stream));
  }
  const int* ov = nullptr;
  if (cand_override && K > 0) {
    CUDA_OK(cudaMemcpyAsync(c->d_cand_ov, cand_override, (size_t)B * K * kmax * sizeof(int), cudaMemcpyHostToDevice, c->stream));
    ov = c->d_cand_ov;
  }
  // the attention launch shape depends only on whether the context fits ATTN_SINGLE_TILES tiles (the
  // kernel takes the lengths themselves from the device), so the launches are planned for one of two
  // length bounds and a recorded step serves every length below its bound
  std::vector<int> n_hi_plan(B), n_lo_plan(B);
  for (int b = 0; b < B; ++b) {
    // three launch shapes: contexts that may reach the long-context kernel's threshold are planned for any length;
    // below it the CTA-per-16-rows kernel serves every length up to the threshold, and the split kernel is planned
    // for at most ATTN_SINGLE_TILES tiles or for any length
    int bound;
    if (attn_long_mode(c, T_, c->n_hi[b] + T_)) bound = c->cap;
    else if (attn_rows_mode(c, T_)) bound = attn_long_mode(c, T_, 1 << 30) ? std::min(attn_long_threshold(c, T_) / 64 * 64, c->cap) : c->cap;
    else if (c->n_hi[b] + T_ > ATTN_SINGLE_TILES * 64) bound = attn_long_mode(c, T_, 1 << 30) ? std::min(std::max(attn_long_threshold(c, T_) / 64 * 64, ATTN_SINGLE_TILES * 64), c->cap) : c->cap;
    else bound = std::min(ATTN_SINGLE_TILES * 64, c->cap);
    n_hi_plan[b] = bound - T_;
    n_lo_plan[b] = c->n_lo[b];
  }
  const bool use_graph = c->graph_on && !c->trace_on && c->profile_kind == 0;
  if (!use_graph) {
    int r = step_body<T>(c, ov, n_hi_plan.data(), n_lo_plan.data());
    if (r) return r;
  } else {
    spec_ctx::StepGraph& g = c->step_graph[ov ? 1 : 0];
    bool valid = g.exec && g.epoch == c->graph_epoch && g.B == B;
    for (int b = 0; valid && b < B; ++b) valid = c->n_hi[b] <= g.n_hi_plan[b] && c->n_lo[b] >= g.n_lo_plan[b];
    if (!valid) {
      // record the step once, then replay it until a sequence outgrows the planned bound
      cudaGraph_t graph = nullptr;
      const long long l0 = c->launches;
      // recorded on a stream of the library's own (the caller's may be the legacy default stream,
      // which cannot be captured); the graph is then launched on the caller's stream
      if (!c->cap_stream) CUDA_OK(cudaStreamCreateWithFlags(&c->cap_stream, cudaStreamNonBlocking));
      CUDA_OK(cudaStreamBeginCapture(c->cap_stream, cudaStreamCaptureModeThreadLocal));
      cudaStream_t user_stream = c->stream;
      c->stream = c->cap_stream;
      c->capturing = true;
      int r = step_body<T>(c, ov, n_hi_plan.data(), n_lo_plan.data());
      c->capturing = false;
      c->stream = user_stream;
      cudaError_t e = cudaStreamEndCapture(c->cap_stream, &graph);
      if (r) { if (graph) cudaGraphDestroy(graph); c->launches = l0; return r; }
      if (e != cudaSuccess || !graph) { c->launches = l0; return c->fail(SPEC_E_CUDA, std::string("step capture: ") + cudaGetErrorString(e)); }
      if (g.exec) { cudaGraphExecDestroy(g.exec); g.exec = nullptr; }
      e = cudaGraphInstantiate(&g.exec, graph, 0);
      cudaGraphDestroy(graph);
      if (e != cudaSuccess) { g.exec = nullptr; c->launches = l0; return c->fail(SPEC_E_CUDA, std::string("step graph instantiate: ") + cudaGetErrorString(e)); }
      g.epoch = c->graph_epoch; g.B = B; g.n_launches = c->launches - l0;
      g.n_hi_plan = n_hi_plan; g.n_lo_plan = n_lo_plan;
      c->launches = l0;
      c->graph_captures++;
    }
    CUDA_OK(cudaGraphLaunch(g.exec, c->stream));
    c->launches += g.n_launches;
  }
  c->phase_valid = c->phase_timing;
  if (c->profile_kind) {
    CUDA_OK(cudaStreamSynchronize(c->stream));
    for (int i = 0; i + 1 < c->prof_used; i += 2) {
      float ms = 0.f;
      if (cudaEventElapsedTime(&ms, c->prof_ev[i], c->prof_ev[i + 1]) == cudaSuccess) { c->prof_ms += ms; c->prof_launches++; }
    }
  }
  if (out_tokens || out_counts) {
    if (out_tokens) CUDA_OK(cudaMemcpyAsync(out_tokens, c->d_out_tok, (size_t)B * (K + 1) * sizeof(int), cudaMemcpyDeviceToHost, c->stream));
    if (out_counts) CUDA_OK(cudaMemcpyAsync(out_counts, c->d_count, (size_t)B * sizeof(int), cudaMemcpyDeviceToHost, c->stream));
    std::vector<int> nn(B);
    CUDA_OK(cudaMemcpyAsync(nn.data(), c->d_n, B * sizeof(int), cudaMemcpyDeviceToHost, c->stream));
    int r = check_status(c);   // synchronises
    if (r) return r;
    for (int b = 0; b < B; ++b) c->n_hi[b] = c->n_lo[b] = nn[b];
    c->n_copy_pending = false;
  } else {
    for (int b = 0; b < B; ++b) { c->n_hi[b] += K + 1; c->n_lo[b] += 1; }
    if (c->h_n_pinned && c->n_ev) {
      if (c->n_copy_pending) {
        c->n_copy_steps_after++;
        // the host stays at most MAX_STEPS_AHEAD steps ahead of the device, so that its bounds stay close
        if (c->n_copy_steps_after >= MAX_STEPS_AHEAD) cudaEventSynchronize(c->n_ev);
        if (cudaEventQuery(c->n_ev) == cudaSuccess) {
          // the copy shows the lengths after an earlier step; every step since added 1..K+1 tokens
          for (int b = 0; b < B; ++b) {
            c->n_lo[b] = std::max(c->n_lo[b], c->h_n_pinned[b] + c->n_copy_steps_after);
            c->n_hi[b] = std::min(c->n_hi[b], c->h_n_pinned[b] + c->n_copy_steps_after * (K + 1));
          }
          c->n_copy_pending = false;
        }
      }
      // a copy between two steps costs the overlap of the step's last kernel with the next step's first:
      // one every N_COPY_EVERY steps keeps the bounds tight enough
      if (!c->n_copy_pending && ++c->steps_since_n_copy >= N_COPY_EVERY && (c->steps_since_n_copy = 0, true) &&
          cudaMemcpyAsync(c->h_n_pinned, c->d_n, (size_t)B * sizeof(int), cudaMemcpyDeviceToHost, c->stream) == cudaSuccess &&
          cudaEventRecord(c->n_ev, c->stream) == cudaSuccess) {
        c->n_copy_pending = true;
        c->n_copy_steps_after = 0;
      }
    }
  }
  return SPEC_OK;
}

}  // namespace

extern "C" {

size_t spec_workspace_bytes(const spec_config* cfg, const spec_tree* tree) {
  std::string why;
  if (!cfg || !tree || !validate_config(cfg, &why)) return 0;
  spec_ctx tmp{};
  tmp.cfg = *cfg;
  if (!validate_tree(cfg, tree, &tmp.kmax, &why)) return 0;
  tmp.T = tree->n_nodes; tmp.K = cfg->n_medusa;
  tmp.tc = cfg->dtype == 1 && !(cfg->flags & SPEC_FLAG_SIMPLE_KERNELS);
  tmp.esz = cfg->dtype == 1 ? 2 : 4;
  return carve(&tmp, nullptr);
}

int spec_create(const spec_config* cfg, const spec_weights* w, const spec_tree* tree, void* workspace,
                size_t workspace_bytes, void* cuda_stream, spec_ctx** out) {
  std::string why;
  if (!cfg || !w || !tree || !workspace || !out) { g_create_error = "null argument"; return SPEC_E_BADARG; }
  if (!validate_config(cfg, &why)) { g_create_error = why; return SPEC_E_BADARG; }
  int kmax = 1;
  if (!validate_tree(cfg, tree, &kmax, &why)) { g_create_error = why; return SPEC_E_BADTREE; }
  if (!w->embed || !w->lm_head || !w->final_norm || !w->attn_norm || !w->wq || !w->wk || !w->wv || !w->wo ||
      !w->ffn_norm || !w->w_gate || !w->w_up || !w->w_down || (cfg->n_medusa > 0 && (!w->medusa_w || !w->medusa_b))) {
    g_create_error = "null weight pointer"; return SPEC_E_BADARG;
  }
  if (reinterpret_cast<uintptr_t>(workspace) % 1024) { g_create_error = "workspace must be 1024-byte aligned"; return SPEC_E_BADARG; }
  spec_ctx* c = new spec_ctx();
  c->cfg = *cfg;
  c->stream = static_cast<cudaStream_t>(cuda_stream);
  c->T = tree->n_nodes; c->K = cfg->n_medusa; c->kmax = kmax; c->B = cfg->max_batch;
  c->tc = cfg->dtype == 1 && !(cfg->flags & SPEC_FLAG_SIMPLE_KERNELS);
  c->packed = (cfg->flags & SPEC_FLAG_PACKED_WEIGHTS) != 0;
  c->esz = cfg->dtype == 1 ? 2 : 4;
  size_t need = carve(c, workspace);
  if (need > workspace_bytes) { g_create_error = "workspace too small"; delete c; return SPEC_E_NOMEM; }
  c->h_parent.assign(tree->parent, tree->parent + c->T);
  c->h_depth.assign(tree->depth, tree->depth + c->T);
  c->h_rank.assign(tree->rank, tree->rank + c->T);
  int L = cfg->n_layers;
  c->embed = w->embed; c->lm_head = w->lm_head; c->final_norm = w->final_norm;
  c->qkv_fused = true;
  size_t qn = (size_t)cfg->n_heads * cfg->head_dim * cfg->d_model * c->esz, kn = (size_t)cfg->n_kv_heads * cfg->head_dim * cfg->d_model * c->esz;
  for (int l = 0; l < L; ++l) {
    if (!w->attn_norm[l] || !w->wq[l] || !w->wk[l] || !w->wv[l] || !w->wo[l] || !w->ffn_norm[l] || !w->w_gate[l] || !w->w_up[l] || !w->w_down[l]) {
      g_create_error = "null layer weight pointer"; delete c; return SPEC_E_BADARG;
    }
    c->an.push_back(w->attn_norm[l]); c->fn.push_back(w->ffn_norm[l]);
    c->wq.push_back(w->wq[l]); c->wk.push_back(w->wk[l]); c->wv.push_back(w->wv[l]); c->wo.push_back(w->wo[l]);
    c->wg.push_back(w->w_gate[l]); c->wu.push_back(w->w_up[l]); c->wd.push_back(w->w_down[l]);
    const uint8_t* q0 = static_cast<const uint8_t*>(w->wq[l]);
    if (static_cast<const uint8_t*>(w->wk[l]) != q0 + qn || static_cast<const uint8_t*>(w->wv[l]) != q0 + qn + kn) c->qkv_fused = false;
  }
  for (int k = 0; k < c->K; ++k) { c->mw.push_back(w->medusa_w[k]); c->mb.push_back(w->medusa_b[k]); }
  if (c->tc && !get_encode_fn()) { g_create_error = "cuTensorMapEncodeTiled entry point unavailable"; delete c; return SPEC_E_CUDA; }

  // host-made tables: tree arrays, ancestor bitsets (tree and chain), page table, RoPE table
  std::vector<uint32_t> anc_tree(SPEC_MAX_NODES * 4, 0), anc_chain(PREFILL_ROWS * 4, 0);
  for (int v = 0; v < c->T; ++v) {
    if (v > 0) for (int wd = 0; wd < 4; ++wd) anc_tree[v * 4 + wd] = anc_tree[c->h_parent[v] * 4 + wd];
    anc_tree[v * 4 + (v >> 5)] |= 1u << (v & 31);
  }
  for (int v = 0; v < PREFILL_ROWS; ++v)
    for (int u = 0; u <= v; ++u) anc_chain[v * 4 + (u >> 5)] |= 1u << (u & 31);
  std::vector<int> pt((size_t)cfg->max_batch * c->pages_per_seq);
  for (int b = 0; b < cfg->max_batch; ++b)
    for (int p = 0; p < c->pages_per_seq; ++p) pt[(size_t)b * c->pages_per_seq + p] = p * cfg->max_batch + b;
  int half = cfg->head_dim / 2;
  std::vector<float2> rope((size_t)c->cap * half);
  for (int i = 0; i < half; ++i) {
    double inv = pow((double)cfg->rope_base, -2.0 * i / cfg->head_dim);
    for (int p = 0; p < c->cap; ++p) {
      double ang = (double)p * inv;
      rope[(size_t)p * half + i] = make_float2((float)cos(ang), (float)sin(ang));
    }
  }
  cudaError_t e = cudaSuccess;
  auto up = [&](void* dst, const void* src, size_t bytes) {
    if (e == cudaSuccess && bytes) e = cudaMemcpyAsync(dst, src, bytes, cudaMemcpyHostToDevice, c->stream);
  };
  up(c->d_parent, c->h_parent.data(), c->T * sizeof(int));
  up(c->d_depth, c->h_depth.data(), c->T * sizeof(int));
  up(c->d_rank, c->h_rank.data(), c->T * sizeof(int));
  up(c->d_anc_tree, anc_tree.data(), anc_tree.size() * 4);
  up(c->d_anc_chain, anc_chain.data(), anc_chain.size() * 4);
  up(c->d_page_table, pt.data(), pt.size() * sizeof(int));
  up(c->d_rope, rope.data(), rope.size() * sizeof(float2));
  up(c->d_mw, c->mw.data(), c->mw.size() * sizeof(void*));
  up(c->d_mb, c->mb.data(), c->mb.size() * sizeof(void*));
  if (e == cudaSuccess) e = cudaMemsetAsync(c->d_status, 0, 4 * sizeof(int), c->stream);
  if (e == cudaSuccess) e = cudaMemsetAsync(c->d_attn_arrive, 0, (size_t)cfg->max_batch * cfg->n_heads * 2 * sizeof(unsigned int), c->stream);
  if (e == cudaSuccess) e = cudaMemsetAsync(c->d_row_arrive, 0, (size_t)c->Mcap * sizeof(unsigned int), c->stream);
  if (e == cudaSuccess) e = cudaMemsetAsync(c->d_cand, 0, (size_t)cfg->max_batch * (c->K + 1) * c->kmax * sizeof(int), c->stream);
  if (e == cudaSuccess) e = cudaStreamSynchronize(c->stream);
  if (e != cudaSuccess) { g_create_error = std::string("set-up copies: ") + cudaGetErrorString(e); delete c; return SPEC_E_CUDA; }
  if (cudaHostAlloc(reinterpret_cast<void**>(&c->h_n_pinned), (size_t)cfg->max_batch * sizeof(int), cudaHostAllocDefault) != cudaSuccess) c->h_n_pinned = nullptr;
  if (cudaEventCreateWithFlags(&c->n_ev, cudaEventDisableTiming) != cudaSuccess) c->n_ev = nullptr;
  cudaGetLastError();
  if (c->tc && cfg->head_dim == 128 && cfg->page_size == 16) {
    // 5-D view of the page pool for the tcgen05 attention: (64 dims of a slab row, the 64 slab rows of a page's
    // K|V pair = 4 slabs x 16 rows, sequence, page, layer * kv_heads + head); page p of sequence b is pool
    // page p * max_batch + b (the table written above), so both are strided dimensions
    EncodeTiledFn fn = get_encode_fn();
    const cuuint64_t pair_bytes = (cuuint64_t)c->geom.block_elems() * 2 * 2;
    cuuint64_t dims[5] = {64, 64, (cuuint64_t)cfg->max_batch, (cuuint64_t)c->pages_per_seq, (cuuint64_t)cfg->n_layers * cfg->n_kv_heads};
    cuuint64_t strides[4] = {128, pair_bytes, pair_bytes * (cuuint64_t)cfg->max_batch, pair_bytes * (cuuint64_t)c->geom.pool_pages()};
    cuuint32_t box[5] = {64, 16, 1, AU_KT / 16, 1};
    cuuint32_t estr[5] = {1, 1, 1, 1, 1};
    c->tm_kv_ok = fn && fn(&c->tm_kv, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 5, c->d_pool, dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
                           CU_TENSOR_MAP_SWIZZLE_NONE, CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
  }
  *out = c;
  return SPEC_OK;
}

int spec_prefill(spec_ctx* c, int32_t batch, const int32_t* tokens, const int32_t* offsets) {
  if (!c) return SPEC_E_BADARG;
  if (!tokens || !offsets) return c->fail(SPEC_E_BADARG, "null argument");
  if (batch < 1 || batch > c->cfg.max_batch) return c->fail(SPEC_E_BADARG, "batch out of range");
  return c->cfg.dtype == 1 ? prefill_t<bf16>(c, batch, tokens, offsets) : prefill_t<float>(c, batch, tokens, offsets);
}

int spec_step(spec_ctx* c, int32_t* out_tokens, int32_t* out_counts, const int32_t* cand_override) {
  if (!c) return SPEC_E_BADARG;
  if (!c->prefilled) return c->fail(SPEC_E_STATE, "spec_step before spec_prefill");
  return c->cfg.dtype == 1 ? step_t<bf16>(c, out_tokens, out_counts, cand_override)
                           : step_t<float>(c, out_tokens, out_counts, cand_override);
}

int spec_read_generated(spec_ctx* c, int32_t seq, int32_t* out, int32_t max_tokens, int32_t* n_generated) {
  if (!c) return SPEC_E_BADARG;
  if (!c->prefilled) return c->fail(SPEC_E_STATE, "nothing generated yet");
  if (seq < 0 || seq >= c->B || !n_generated || max_tokens < 0) return c->fail(SPEC_E_BADARG, "bad argument");
  int r = check_status(c);
  if (r) return r;
  int cnt = 0;
  CUDA_OK(cudaMemcpyAsync(&cnt, c->d_gen_cnt + seq, sizeof(int), cudaMemcpyDeviceToHost, c->stream));
  CUDA_OK(cudaStreamSynchronize(c->stream));
  int stored = cnt < c->gen_cap ? cnt : c->gen_cap;
  int ncopy = stored < max_tokens ? stored : max_tokens;
  if (out && ncopy > 0) {
    CUDA_OK(cudaMemcpyAsync(out, c->d_gen_log + (size_t)seq * c->gen_cap, ncopy * sizeof(int), cudaMemcpyDeviceToHost, c->stream));
    CUDA_OK(cudaStreamSynchronize(c->stream));
  }
  *n_generated = cnt;
  std::vector<int> nn(c->B);
  CUDA_OK(cudaMemcpyAsync(nn.data(), c->d_n, c->B * sizeof(int), cudaMemcpyDeviceToHost, c->stream));
  CUDA_OK(cudaStreamSynchronize(c->stream));
  for (int b = 0; b < c->B; ++b) c->n_hi[b] = c->n_lo[b] = nn[b];
  return SPEC_OK;
}

int spec_destroy(spec_ctx* c) {
  if (!c) return SPEC_E_BADARG;
  cudaStreamSynchronize(c->stream);
  for (int i = 0; i < 6; ++i) if (c->phase_ev[i]) cudaEventDestroy(c->phase_ev[i]);
  for (cudaEvent_t e : c->prof_ev) cudaEventDestroy(e);
  for (auto& g : c->step_graph) if (g.exec) cudaGraphExecDestroy(g.exec);
  if (c->cap_stream) cudaStreamDestroy(c->cap_stream);
  if (c->n_ev) cudaEventDestroy(c->n_ev);
  if (c->h_n_pinned) cudaFreeHost(c->h_n_pinned);
  delete c;
  return SPEC_OK;
}

const char* spec_last_error(const spec_ctx* c) { return c ? c->err.c_str() : g_create_error.c_str(); }

int64_t spec_query(const spec_ctx* c, int32_t what) {
  if (!c) return -1;
  const spec_config& f = c->cfg;
  switch (what) {
    case SPEC_Q_KMAX: return c->kmax;
    case SPEC_Q_KERNEL_LAUNCHES: return c->launches;
    case SPEC_Q_N_NODES: return c->T;
    case SPEC_Q_BATCH: return c->B;
    case SPEC_Q_GRAPH_CAPTURES: return c->graph_captures;
    case SPEC_Q_WIDE_GEMM: return c->tc && c->wide_gemm ? 1 : 0;
    case SPEC_Q_CLUSTER_GATE_UP: return c->tc && cluster_gemm_ok(c, GC_SWIGLU, c->B * c->T, f.d_model) ? 1 : 0;
    case SPEC_Q_ALGO_BYTES_PER_STEP: {
      double d = f.d_model, F = f.d_ffn, V = f.vocab, HD = (double)f.n_heads * f.head_dim, KD = (double)f.n_kv_heads * f.head_dim;
      double layer = d * HD + 2 * d * KD + HD * d + 3 * d * F;
      double bytes = (f.n_layers * layer + 2 * V * d + c->K * (d * d + d)) * (double)c->esz;
      return (int64_t)(bytes / 1024.0);
    }
    default: return -1;
  }
}

int spec_set_option(spec_ctx* c, int32_t what, int32_t value) {
  if (!c) return SPEC_E_BADARG;
  switch (what) {
    case SPEC_OPT_GEMM_CTAS: case SPEC_OPT_SMALL_GEMM_CTAS:
      if (value < 1 || value > SM_SLOTS) return c->fail(SPEC_E_BADARG, "gemm CTA count out of range");
      break;
    case SPEC_OPT_L2_PREFETCH:
      if (value < 0 || value > 64) return c->fail(SPEC_E_BADARG, "L2 prefetch depth out of range");
      break;
    case SPEC_OPT_GRAPH: case SPEC_OPT_PHASE_TIMING: case SPEC_OPT_PDL: case SPEC_OPT_TRACE: case SPEC_OPT_CLUSTER_EPILOGUE: case SPEC_OPT_WIDE_GEMM: case SPEC_OPT_ATTN_UMMA: break;
    case SPEC_OPT_LONG_ATTN_KEYS:
      if (value < 0) return c->fail(SPEC_E_BADARG, "context threshold must not be negative");
      break;
    default: return c->fail(SPEC_E_BADARG, "unknown option");
  }
  c->graph_epoch++;   // the option is valid: a recorded step no longer matches the options
  switch (what) {
    case SPEC_OPT_GRAPH:
      c->graph_on = value != 0; return SPEC_OK;
    case SPEC_OPT_PHASE_TIMING:
      c->phase_timing = value != 0; c->phase_valid = false; return SPEC_OK;
    case SPEC_OPT_PDL: c->pdl = value != 0; return SPEC_OK;
    case SPEC_OPT_GEMM_CTAS:
      if (value < 1 || value > SM_SLOTS) return c->fail(SPEC_E_BADARG, "gemm CTA count out of range");
      c->gemm_ctas = value; return SPEC_OK;
    case SPEC_OPT_L2_PREFETCH:
      if (value < 0 || value > 64) return c->fail(SPEC_E_BADARG, "L2 prefetch depth out of range");
      c->l2_prefetch = value; return SPEC_OK;
    case SPEC_OPT_SMALL_GEMM_CTAS:
      if (value < 1 || value > SM_SLOTS) return c->fail(SPEC_E_BADARG, "out of range");
      c->small_gemm_ctas = value; return SPEC_OK;
    case SPEC_OPT_CLUSTER_EPILOGUE: c->cluster_epilogue = value & 7; return SPEC_OK;
    case SPEC_OPT_WIDE_GEMM: c->wide_gemm = value != 0; return SPEC_OK;
    case SPEC_OPT_LONG_ATTN_KEYS: c->long_attn_keys = value; return SPEC_OK;
    case SPEC_OPT_ATTN_UMMA: c->attn_umma = value != 0; return SPEC_OK;
    case SPEC_OPT_TRACE:
      c->trace_on = value != 0;
      if (c->trace_on && c->trace_init.empty()) {
        c->trace_init.resize((size_t)TRACE_CAP * 4);
        for (int i = 0; i < TRACE_CAP; ++i) { c->trace_init[4 * i] = ~0ull; c->trace_init[4 * i + 1] = 0; c->trace_init[4 * i + 2] = ~0ull; c->trace_init[4 * i + 3] = 0; }
      }
      return SPEC_OK;
    default: return c->fail(SPEC_E_BADARG, "unknown option");
  }
}

int spec_trace_read(spec_ctx* c, int32_t max_records, char* names, uint64_t* stamps, int32_t* n_records) {
  if (!c || !n_records || max_records < 0 || (max_records > 0 && (!names || !stamps))) return SPEC_E_BADARG;
  if (!c->trace_on) return c->fail(SPEC_E_STATE, "tracing is off (SPEC_OPT_TRACE)");
  int n = c->trace_n < max_records ? c->trace_n : max_records;
  if (n > 0) {
    CUDA_OK(cudaMemcpyAsync(stamps, c->d_trace, (size_t)n * 32, cudaMemcpyDeviceToHost, c->stream));
    CUDA_OK(cudaStreamSynchronize(c->stream));
    for (int i = 0; i < n; ++i) {
      strncpy(names + (size_t)i * SPEC_TRACE_NAME_LEN, c->trace_names[i].c_str(), SPEC_TRACE_NAME_LEN - 1);
      names[(size_t)i * SPEC_TRACE_NAME_LEN + SPEC_TRACE_NAME_LEN - 1] = 0;
    }
  }
  *n_records = c->trace_n;
  return SPEC_OK;
}

int spec_last_step_phase_ms(spec_ctx* c, float* ms) {
  if (!c || !ms) return SPEC_E_BADARG;
  if (!c->phase_valid) return c->fail(SPEC_E_STATE, "no step has run with SPEC_OPT_PHASE_TIMING on");
  CUDA_OK(cudaStreamSynchronize(c->stream));
  for (int i = 0; i < 5; ++i) CUDA_OK(cudaEventElapsedTime(&ms[i], c->phase_ev[i], c->phase_ev[i + 1]));
  return SPEC_OK;
}

int spec_profile_kernel(spec_ctx* c, int32_t kind) {
  if (!c || kind < 0 || kind > SPEC_PROFILE_ATTENTION) return SPEC_E_BADARG;
  c->profile_kind = kind;
  c->prof_ms = 0.0;
  c->prof_launches = 0;
  return SPEC_OK;
}

int spec_profile_read(spec_ctx* c, double* total_ms, int64_t* launches) {
  if (!c || !total_ms || !launches) return SPEC_E_BADARG;
  *total_ms = c->prof_ms;
  *launches = c->prof_launches;
  return SPEC_OK;
}

int spec_debug_read(spec_ctx* c, int32_t what, void* host_buf, size_t bytes) {
  if (!c || !host_buf) return SPEC_E_BADARG;
  const spec_config& f = c->cfg;
  size_t rows = (size_t)c->B * c->T;
  const void* src = nullptr;
  size_t need = 0;
  switch (what) {
    case SPEC_DBG_TOK: src = c->d_tok; need = rows * 4; break;
    case SPEC_DBG_POS: src = c->d_pos; need = rows * 4; break;
    case SPEC_DBG_LOGITS: src = c->d_logits; need = rows * f.vocab * 4; break;
    case SPEC_DBG_HIDDEN: src = c->d_hid; need = rows * f.d_model * 4; break;
    case SPEC_DBG_ARGMAX: src = c->d_am; need = rows * 4; break;
    case SPEC_DBG_PATH: src = c->d_path; need = (size_t)c->B * (c->K + 1) * 4; break;
    case SPEC_DBG_CAND: src = c->d_cand; need = (size_t)c->B * (c->K + 1) * c->kmax * 4; break;
    case SPEC_DBG_SEQLEN: src = c->d_n; need = (size_t)c->B * 4; break;
    case SPEC_DBG_NEXT_ROOT: src = c->d_root; need = (size_t)c->B * 4; break;
    case SPEC_DBG_H_LAST: src = c->d_h_last; need = (size_t)c->B * f.d_model * 4; break;
    case SPEC_DBG_STATUS: src = c->d_status; need = 16; break;
    default: return c->fail(SPEC_E_BADARG, "unknown debug tap");
  }
  if (!src) return c->fail(SPEC_E_STATE, "tap not available (logits need SPEC_FLAG_KEEP_LOGITS)");
  if (bytes < need) return c->fail(SPEC_E_BADARG, "host buffer too small");
  CUDA_OK(cudaMemcpyAsync(host_buf, src, need, cudaMemcpyDeviceToHost, c->stream));
  CUDA_OK(cudaStreamSynchronize(c->stream));
  return SPEC_OK;
}

int spec_debug_wait_timeout(spec_ctx* c, int32_t limit_us) {
  if (!c) return SPEC_E_BADARG;
  if (limit_us < 1 || limit_us > 100000) return c->fail(SPEC_E_BADARG, "limit must be 1..100000 microseconds");
  CUDA_OK(cudaStreamSynchronize(c->stream));
  wait_probe<<<1, 32, 0, c->stream>>>(c->d_status, (unsigned long long)limit_us * 1000ull);
  LAUNCH_CHECK("wait_probe");
  int r = check_status(c);           // reads the status word: SPEC_E_TIMEOUT with the probe's place code
  // the probe is the only writer here: clear the word so that the context stays usable
  CUDA_OK(cudaMemsetAsync(c->d_status, 0, 4 * sizeof(int), c->stream));
  CUDA_OK(cudaStreamSynchronize(c->stream));
  return r;
}

int spec_debug_read_kv(spec_ctx* c, int32_t seq, int32_t layer, int32_t slot0, int32_t n_slots, float* host_k, float* host_v) {
  if (!c || !host_k || !host_v) return SPEC_E_BADARG;
  const spec_config& f = c->cfg;
  if (seq < 0 || seq >= f.max_batch || layer < 0 || layer >= f.n_layers || slot0 < 0 || n_slots < 0 || slot0 + n_slots > c->cap)
    return c->fail(SPEC_E_BADARG, "bad KV range");
  int D = f.head_dim, Hkv = f.n_kv_heads, ps = f.page_size;
  std::vector<uint8_t> blk(c->geom.block_elems() * c->esz);
  CUDA_OK(cudaStreamSynchronize(c->stream));
  for (int kv = 0; kv < 2; ++kv) {
    float* dst = kv ? host_v : host_k;
    for (int h = 0; h < Hkv; ++h) {
      int cur_page = -1;
      for (int sl = slot0; sl < slot0 + n_slots; ++sl) {
        int page = (sl / ps) * f.max_batch + seq;   // same mapping as the device page table
        if (page != cur_page) {
          const uint8_t* src = static_cast<const uint8_t*>(c->d_pool) + c->geom.block_offset(page, layer, kv, h) * c->esz;
          CUDA_OK(cudaMemcpy(blk.data(), src, blk.size(), cudaMemcpyDeviceToHost));
          cur_page = page;
        }
        int row = sl % ps;
        for (int e = 0; e < D; ++e) {
          float v;
          if (c->esz == 2) {
            uint16_t raw = reinterpret_cast<uint16_t*>(blk.data())[(size_t)row * D + kv_elem<bf16>(row, e, D, ps)];
            uint32_t u32 = (uint32_t)raw << 16;
            memcpy(&v, &u32, 4);
          } else {
            v = reinterpret_cast<float*>(blk.data())[(size_t)row * D + e];
          }
          dst[((size_t)(sl - slot0) * Hkv + h) * D + e] = v;
        }
      }
    }
  }
  return SPEC_OK;
}

namespace {
// Shared body of the two stand-alone linear entry points (bf16): scratch holds the partial
// sums followed by the four-int status word.
int op_linear_bf16(const void* x, const void* w, float* y, int M, int N, int K, int ctas, float* scratch,
                   size_t scratch_floats, cudaStream_t st) {
  GemmPlan g;
  int rws[1] = {N};
  if (!plan_gemm(M, K, 1, rws, ctas, &g)) return SPEC_E_BADARG;
  StreamTmaps tm{};
  if (!make_tmap(&tm.a[0], w, N, K, 128) || !make_tmap(&tm.b, x, M, K, g.MT)) return SPEC_E_CUDA;
  g.p.part = scratch;
  g.p.slot_stride = (size_t)M * g.p.n_tiles * 128;
  g.p.l2_prefetch = 0;
  g.p.status = reinterpret_cast<int*>(scratch + scratch_floats);
  // the status word must start at zero; the partial sums are fully overwritten before they are read
  if (cudaMemsetAsync(g.p.status, 0, 16, st) != cudaSuccess) return SPEC_E_CUDA;
  if (launch_gs(st, false, g, tm) != cudaSuccess) return SPEC_E_CUDA;
  size_t total = (size_t)M * ((N + 3) / 4);
  part_sum_rows<<<(unsigned)std::min<size_t>((total + 255) / 256, 4096), 256, 0, st>>>(plan_view(g), y, M, N);
  if (cudaGetLastError() != cudaSuccess) return SPEC_E_CUDA;
  int stw[4];
  if (cudaMemcpyAsync(stw, g.p.status, 16, cudaMemcpyDeviceToHost, st) != cudaSuccess || cudaStreamSynchronize(st) != cudaSuccess)
    return SPEC_E_CUDA;
  return stw[0] == 0 ? SPEC_OK : SPEC_E_TIMEOUT;
}
bool op_linear_args_ok(int32_t dtype, const void* x, const void* w, const float* y, int M, int N, int K, int ctas) {
  if (!x || !w || !y || M < 1 || N < 1 || K < 8 || K % 8 || M > 2048) return false;
  if (dtype == 0) return true;
  return dtype == 1 && K % 64 == 0 && M % 16 == 0 && N >= 128 && ctas >= 1 && ctas <= 1024;
}
}  // namespace

int spec_build_labels(const int32_t* tokens, int32_t n_seq, int32_t seq_len, int32_t num_heads, int32_t frag_token,
                      int32_t pad_token, int32_t ignore_token, int32_t* labels, void* cuda_stream) {
  if (n_seq == 0 || seq_len == 0) return SPEC_OK;
  if (!tokens || !labels || n_seq < 0 || seq_len < 0 || num_heads < 0 || num_heads > LABEL_MAX_HEADS || n_seq > 65535)
    return SPEC_E_BADARG;
  dim3 grid((seq_len + LABEL_THREADS - 1) / LABEL_THREADS, n_seq);
  build_labels_kernel<<<grid, LABEL_THREADS, 0, static_cast<cudaStream_t>(cuda_stream)>>>(tokens, seq_len, num_heads, frag_token,
                                                                                        pad_token, ignore_token, labels);
  return cudaGetLastError() == cudaSuccess ? SPEC_OK : SPEC_E_CUDA;
}

size_t spec_packed_weight_bytes(int32_t rows, int32_t cols) {
  if (rows < 1 || cols < 64 || cols % 64) return 0;
  return (size_t)((rows + 127) / 128) * (size_t)(cols / 64) * 16384;
}

int spec_pack_weight(const void* w, int32_t rows, int32_t cols, void* packed, void* cuda_stream) {
  const size_t bytes = spec_packed_weight_bytes(rows, cols);
  if (!w || !packed || bytes == 0 || (reinterpret_cast<uintptr_t>(packed) & 15) || (reinterpret_cast<uintptr_t>(w) & 15)) {
    g_create_error = "spec_pack_weight: null or unaligned pointer, or cols not a multiple of 64";
    return SPEC_E_BADARG;
  }
  const size_t units = bytes / 16384;
  if (units > 0x7fffffffu) { g_create_error = "spec_pack_weight: matrix too large"; return SPEC_E_BADARG; }
  pack_weight_tiles<<<(unsigned)units, 256, 0, static_cast<cudaStream_t>(cuda_stream)>>>(static_cast<const bf16*>(w), rows, cols,
                                                                                        static_cast<uint8_t*>(packed));
  cudaError_t e = cudaGetLastError();
  if (e != cudaSuccess) { g_create_error = std::string("pack_weight_tiles: ") + cudaGetErrorString(e); return SPEC_E_CUDA; }
  return SPEC_OK;
}

size_t spec_op_linear_scratch_floats(int32_t M, int32_t N, int32_t K, int32_t ctas) {
  GemmPlan g;
  int rws[1] = {N};
  if (M < 1 || N < 1 || ctas < 1 || !plan_gemm(M, K, 1, rws, ctas, &g)) return 0;
  return plan_part_floats(g);
}

int spec_op_linear(int32_t dtype, const void* x, const void* w, float* y, int32_t M, int32_t N, int32_t K,
                   int32_t ctas, float* scratch, void* cuda_stream) {
  if (!op_linear_args_ok(dtype, x, w, y, M, N, K, ctas)) return SPEC_E_BADARG;
  cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
  if (dtype == 0) {
    constexpr int MC = 8;
    dim3 grid((N + 7) / 8, (M + MC - 1) / MC);
    linear_rows<float, MC><<<grid, 256, 0, st>>>(static_cast<const float*>(x), K, static_cast<const float*>(w), y, N, M, N, K);
    return cudaGetLastError() == cudaSuccess ? SPEC_OK : SPEC_E_CUDA;
  }
  if (!scratch) return SPEC_E_BADARG;
  return op_linear_bf16(x, w, y, M, N, K, ctas, scratch, spec_op_linear_scratch_floats(M, N, K, ctas), st);
}

}  // extern "C"

// ---- the linear operation for callers that cannot allocate device memory ----
// The partial sums and the status word of spec_op_linear_static live here instead of in a
// caller-provided buffer. Every context that loads the library holds these bytes until exit.
static __device__ __align__(256) float g_static_linear_scratch[SPEC_STATIC_SCRATCH_FLOATS + 4];

namespace {
constexpr int kMaxDevices = 64;
float* g_static_scratch_addr[kMaxDevices] = {};   // device address of the array, per device ordinal
}  // namespace

extern "C" int spec_op_linear_static(int32_t dtype, const void* x, const void* w, float* y, int32_t M, int32_t N, int32_t K,
                                     int32_t ctas, void* cuda_stream) {
  if (!op_linear_args_ok(dtype, x, w, y, M, N, K, ctas)) { g_create_error = "spec_op_linear_static: bad argument"; return SPEC_E_BADARG; }
  cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
  if (dtype == 0) {
    constexpr int MC = 8;
    dim3 grid((N + 7) / 8, (M + MC - 1) / MC);
    linear_rows<float, MC><<<grid, 256, 0, st>>>(static_cast<const float*>(x), K, static_cast<const float*>(w), y, N, M, N, K);
    return cudaGetLastError() == cudaSuccess ? SPEC_OK : SPEC_E_CUDA;
  }
  const size_t need = spec_op_linear_scratch_floats(M, N, K, ctas);
  if (need == 0) { g_create_error = "spec_op_linear_static: bad argument"; return SPEC_E_BADARG; }
  if (need > (size_t)SPEC_STATIC_SCRATCH_FLOATS) {
    char buf[200];
    snprintf(buf, sizeof(buf), "spec_op_linear_static: %zu floats of partial sums exceeds the built-in scratch of %u floats",
             need, (unsigned)SPEC_STATIC_SCRATCH_FLOATS);
    g_create_error = buf;
    return SPEC_E_NOMEM;
  }
  // Set-up, once per device: the array's name is only a host-side handle here, so ask the
  // runtime for its address on the current device and keep it.
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) { g_create_error = "spec_op_linear_static: cudaGetDevice failed"; return SPEC_E_CUDA; }
  float* scratch = g_static_scratch_addr[dev];
  if (!scratch) {
    void* ptr = nullptr;
    cudaError_t e = cudaGetSymbolAddress(&ptr, g_static_linear_scratch);
    if (e != cudaSuccess || !ptr) { g_create_error = std::string("spec_op_linear_static: cudaGetSymbolAddress: ") + cudaGetErrorString(e); return SPEC_E_CUDA; }
    scratch = static_cast<float*>(ptr);
    g_static_scratch_addr[dev] = scratch;
  }
  // the status word sits at the fixed end of the array
  int r = op_linear_bf16(x, w, y, M, N, K, ctas, scratch, (size_t)SPEC_STATIC_SCRATCH_FLOATS, st);
  if (r) g_create_error = "spec_op_linear_static: launch or device status failed";
  return r;
}
