/*
 * spec_decode.h -- C ABI of the draft-and-verify decode loop (Sec. III-B of
 * "Speculative Decoding for Verilog: Speed and Quality, All in One").
 *
 * One decode step, as the paper states it: with the model at position t the base model
 * predicts the token at t+1 and extra head i predicts the token at t+i+1; the heads'
 * top-k predictions form several candidates; the base model scores every candidate
 * position; a token is accepted only if the acceptance rule holds for it and for every
 * token before it; the step emits the longest accepted prefix among all candidates.
 *
 * Conventions
 *  - All functions return 0 on success or a negative SPEC_E_* code. Nothing aborts,
 *    throws or traps; spec_last_error() gives a one-line description of the last failure.
 *  - "DEVICE" pointers are CUDA global memory of the device that was current at
 *    spec_create. "HOST" pointers are ordinary (preferably pinned) host memory.
 *  - The library never calls the device allocator: every buffer it uses lies in the
 *    caller's workspace. (With SPEC_OPT_GRAPH the CUDA runtime keeps an instantiated graph
 *    of the step and the library one extra stream to record it on.) The caller owns
 *    weights, workspace and the stream; they must outlive the context.
 *  - Linear weights are row-major [out_features, in_features]; dtype 0 = float32,
 *    dtype 1 = bfloat16 (operands bf16, accumulation and residual stream float32).
 */
#ifndef SPEC_DECODE_H_
#define SPEC_DECODE_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define SPEC_MAX_NODES 128   /* tree nodes per sequence, root included          */
#define SPEC_MAX_HEADS 16    /* extra decoding heads                            */
#define SPEC_MAX_TOPK 16     /* candidates kept per head                        */

enum {
  SPEC_OK = 0,
  SPEC_E_BADARG = -1,   /* null pointer, non-positive size, unsupported shape            */
  SPEC_E_BADTREE = -2,  /* tree violates the rules listed at spec_tree                    */
  SPEC_E_NOMEM = -3,    /* workspace too small                                            */
  SPEC_E_SEQLEN = -4,   /* a sequence would exceed max_seq                                */
  SPEC_E_CUDA = -5,     /* a CUDA runtime or driver call failed                           */
  SPEC_E_TIMEOUT = -6,  /* a bounded device-side wait expired (device status word)        */
  SPEC_E_STATE = -7     /* call out of order (step before prefill, batch mismatch)        */
};

typedef struct spec_ctx spec_ctx; /* opaque */

typedef struct {
  int32_t n_layers, d_model, n_heads, n_kv_heads, head_dim, d_ffn, vocab;
  float rms_eps, rope_base;
  int32_t dtype;        /* 0 = float32, 1 = bfloat16                                      */
  int32_t n_medusa;     /* K extra heads (Sec. III-B)                                      */
  int32_t max_batch;    /* sequences decoded together                                     */
  int32_t max_seq;      /* committed tokens per sequence (prompt + generated)             */
  int32_t page_size;    /* tokens per KV page (16)                                        */
  int32_t accept_mode;  /* 0 = greedy argmax match; 1 = typical acceptance (Eq. 1)        */
  float typ_eps, typ_delta, temperature; /* Eq. 1 hyper-parameters; softmax temperature   */
  int32_t frag_token;   /* fragment marker id for the fragment-integrity rule; -1 = off   */
  int32_t flags;        /* SPEC_FLAG_* bits                                               */
  int32_t sampling;     /* 0 = the token that follows the accepted span is the base model's
                           argmax there; 1 = sampled decoding (Sec. IV-B): it is drawn from
                           softmax(logits / temperature) (needs accept_mode 1, temperature > 0) */
  uint32_t seed_lo, seed_hi; /* 64-bit seed of the sampler's counter-based generator        */
} spec_config;

#define SPEC_FLAG_KEEP_LOGITS 1 /* materialise verify logits [rows, vocab] for spec_debug_read  */
#define SPEC_FLAG_SIMPLE_KERNELS 2 /* bf16: run the plain CUDA-core kernels (debug aid, slow)  */
#define SPEC_FLAG_PACKED_WEIGHTS 4 /* bf16 tensor-core path: every linear weight pointer of spec_weights
                                      (wq, wk, wv, wo, w_gate, w_up, w_down, lm_head, medusa_w) is the
                                      pre-tiled image made by spec_pack_weight, not the row-major matrix
                                      (embed, norms and biases stay as they are)                    */

/* Candidate tree, HOST arrays of n_nodes entries, copied at spec_create. Rules: node 0 is
 * the root (parent -1, depth 0, rank 0) and carries the base model's own next token;
 * parent[v] < v; depth[v] = depth[parent[v]] + 1 <= n_medusa; node v carries candidate
 * rank[v] (< SPEC_MAX_TOPK) of head depth[v]; siblings have distinct ranks;
 * 1 <= n_nodes <= SPEC_MAX_NODES. */
typedef struct {
  int32_t n_nodes;
  const int32_t *parent, *depth, *rank;
} spec_tree;

/* DEVICE pointers to the weights (HOST arrays of DEVICE pointers where indexed by layer or
 * head). Element type follows spec_config.dtype except the RMSNorm gains, which are
 * always float32. */
typedef struct {
  const void *embed;            /* [vocab, d_model]                                      */
  const void *lm_head;          /* [vocab, d_model], untied                              */
  const float *final_norm;      /* [d_model]                                             */
  const float *const *attn_norm; /* [n_layers] -> [d_model]                              */
  const void *const *wq;        /* [n_layers] -> [n_heads*head_dim, d_model]             */
  const void *const *wk;        /* [n_layers] -> [n_kv_heads*head_dim, d_model]          */
  const void *const *wv;        /* [n_layers] -> [n_kv_heads*head_dim, d_model]          */
  const void *const *wo;        /* [n_layers] -> [d_model, n_heads*head_dim]             */
  const float *const *ffn_norm; /* [n_layers] -> [d_model]                               */
  const void *const *w_gate;    /* [n_layers] -> [d_ffn, d_model]                        */
  const void *const *w_up;      /* [n_layers] -> [d_ffn, d_model]                        */
  const void *const *w_down;    /* [n_layers] -> [d_model, d_ffn]                        */
  const void *const *medusa_w;  /* [n_medusa] -> [d_model, d_model]                      */
  const void *const *medusa_b;  /* [n_medusa] -> [d_model]                               */
} spec_weights;

/* Bytes of DEVICE workspace spec_create needs for this shape and tree (KV page pool, page
 * tables, activations, split-K and split-KV scratch, status word). 0 on invalid input. */
size_t spec_workspace_bytes(const spec_config *cfg, const spec_tree *tree);

/* Builds a context. `workspace` is a DEVICE buffer of at least spec_workspace_bytes(),
 * 1024-byte aligned, zero-filled or not (the library initialises what it needs).
 * `cuda_stream` is a cudaStream_t (NULL = default stream); all work is enqueued on it.
 * The q, k and v projections of a layer run as one launch (bf16) whether or not the three
 * matrices are one allocation.
 * Config and tree are copied; weights, workspace and stream are borrowed. */
int spec_create(const spec_config *cfg, const spec_weights *weights, const spec_tree *tree,
                void *workspace, size_t workspace_bytes, void *cuda_stream, spec_ctx **out);

/* Prompt processing: causal forward over `batch` prompts (HOST token ids, concatenated;
 * offsets[batch+1] HOST). Fills the KV cache for positions 0..len-1 of every sequence,
 * keeps each sequence's last hidden state for the first step's heads and sets the first
 * root token to the base model's argmax at the last prompt position. Resets any earlier
 * decode state. Synchronous. */
int spec_prefill(spec_ctx *ctx, int32_t batch, const int32_t *tokens, const int32_t *offsets);

/* One draft-and-verify step for every sequence of the batch (Sec. III-B):
 *  heads + shared lm_head + per-head top-k -> candidate tree -> one tree-masked
 *  verification forward of the base model -> longest accepted prefix (greedy: a node is
 *  accepted iff its token is the base model's argmax at its parent and its parent is
 *  accepted; ties between equally long paths go to the lowest node index) -> the accepted
 *  path's K/V rows are moved to the next cache positions.
 * out_tokens [batch][n_medusa+1] and out_counts [batch] are HOST buffers: sequence b emitted
 * out_counts[b] in [1, n_medusa+1] tokens, the accepted path root first. The call returns
 * after they are valid. If both are NULL the step is only enqueued on the stream (no host
 * synchronisation); emitted tokens are then read later with spec_read_generated.
 * cand_override: optional HOST table [batch][n_medusa][kmax] (kmax = spec_query(SPEC_Q_KMAX));
 * an entry >= 0 replaces that head candidate after the heads have run, -1 keeps it.
 * Sampled decoding (spec_config.sampling): the token after the accepted span -- the next step's
 * root -- is the first token j whose cumulative weight sum_{i<=j} exp((z_i - max z) / temperature)
 * exceeds u times the total, z the last accepted node's logits (double precision sums in token
 * order), u = (w >> 8) * 2^-24 with w the first output word of Philox-4x32-10 at counter
 * (draw index, sequence, 0, 0) and key (seed_lo, seed_hi); draw 0 is the token after the prompt
 * (spec_prefill), every step takes the next one. */
int spec_step(spec_ctx *ctx, int32_t *out_tokens, int32_t *out_counts, const int32_t *cand_override);

/* Copies up to `max_tokens` tokens generated so far by sequence `seq` (all steps since
 * prefill, in order) to HOST `out` and the total count to *n_generated. Synchronises. */
int spec_read_generated(spec_ctx *ctx, int32_t seq, int32_t *out, int32_t max_tokens, int32_t *n_generated);

int spec_destroy(spec_ctx *ctx);

/* Description of the last error of this context (or of the last failed spec_create when
 * ctx is NULL). Never NULL. */
const char *spec_last_error(const spec_ctx *ctx);

/* Integer properties of a context. */
enum { SPEC_Q_KMAX = 0, SPEC_Q_KERNEL_LAUNCHES = 1, SPEC_Q_N_NODES = 2, SPEC_Q_BATCH = 3,
       SPEC_Q_ALGO_BYTES_PER_STEP = 4 /* weights + lm_head (twice) + heads, in KiB */,
       SPEC_Q_GRAPH_CAPTURES = 5 /* times a step was recorded into a CUDA graph */,
       SPEC_Q_CLUSTER_GATE_UP = 6 /* 1 if a step's gate+up projection runs as the cluster kernel with the SwiGLU inside */,
       SPEC_Q_WIDE_GEMM = 7 /* 1 if passes of more than 128 rows use the 128 x 256-tile kernel */ };
int64_t spec_query(const spec_ctx *ctx, int32_t what);

/* Tuning knobs of a context (defaults in brackets). SPEC_OPT_PDL [1]: launch the kernels of
 * a step with programmatic dependent launch, so that each kernel's set-up and weight prefetch
 * overlap the tail of the one before. SPEC_OPT_GEMM_CTAS [288]: upper bound of the persistent
 * CTAs the weight-streaming GEMM deals its work to (1..296; the library takes the largest count
 * within 15% of it whose runs end on tile boundaries, e.g. 258 = 3 CTAs per 2 tiles for the 172
 * gate+up tiles); SPEC_OPT_SMALL_GEMM_CTAS [288]: the same for GEMMs of at most 48 weight tiles
 * (the output and down projections). SPEC_OPT_L2_PREFETCH [0]: 16 KiB weight
 * chunks each GEMM CTA requests into L2, beyond its shared-memory ring, before it waits for the
 * previous kernel (0..64). Results do not depend on SPEC_OPT_PDL or SPEC_OPT_L2_PREFETCH;
 * SPEC_OPT_GEMM_CTAS and SPEC_OPT_SMALL_GEMM_CTAS change the order in which partial sums are added. SPEC_OPT_TRACE [0]:
 * record a device timeline of every step (see spec_trace_read). SPEC_OPT_GRAPH [1]: record the
 * kernel sequence of a step into a CUDA graph once and replay it on the following steps (a new
 * recording when a sequence grows past the 768 positions the single-split attention launch covers,
 * after a prefill and after an option change; steps that are traced or profiled are enqueued
 * directly). Results do not depend on it. SPEC_OPT_PHASE_TIMING [0]: record an event at the five
 * phase boundaries of every step for spec_last_step_phase_ms (costs the programmatic overlap at
 * those boundaries: about 0.03 ms of a 7B step). SPEC_OPT_CLUSTER_EPILOGUE [7]: bit mask of the projections
 * that, in passes of at most 128 rows, run as thread-block clusters which add their split-K sums through
 * distributed shared memory and apply the step that follows themselves: 1 = output and down projections
 * (residual add in place), 2 = gate+up (SwiGLU, passes of at most 64 rows), 4 = q/k/v (RoPE and cache
 * store). A projection whose bit is clear leaves partial sums for a separate kernel (other summation
 * order, same rounding points). All three are on by default: on the 7B shape they shorten a step by 2.2%,
 * 2% and 4.4%. SPEC_OPT_WIDE_GEMM [1]: passes of more than
 * 128 rows (batched verification, batched prompt processing) run their projections as whole
 * [128 weight rows] x [256 activation rows] tiles that keep a weight tile for 256 rows at a time;
 * 0 = the weight-streaming kernel, which re-reads the weights for every 128 rows.
 * SPEC_OPT_LONG_ATTN_KEYS [2048]: passes whose context may exceed this many positions run a long-context
 * attention kernel, in which a CTA reads a head's K/V once for 64 query rows and the keys are split across
 * the CTAs of a cluster (0 = never; batched passes that need more than one wave of CTAs switch at 512
 * positions already). SPEC_OPT_ATTN_UMMA [1]: that kernel computes scores and P V on tcgen05 with
 * accumulators in tensor memory (head_dim 128, 16-row pages); 0 = the mma.sync kernel that shares K/V tiles
 * between the row blocks of a CTA (passes of more than 32 rows). Results differ from the other attention
 * kernels only in summation order. */
enum { SPEC_OPT_PDL = 0, SPEC_OPT_GEMM_CTAS = 1, SPEC_OPT_L2_PREFETCH = 2, SPEC_OPT_TRACE = 3,
       SPEC_OPT_SMALL_GEMM_CTAS = 4, SPEC_OPT_GRAPH = 5, SPEC_OPT_PHASE_TIMING = 6, SPEC_OPT_CLUSTER_EPILOGUE = 7,
       SPEC_OPT_WIDE_GEMM = 8, SPEC_OPT_LONG_ATTN_KEYS = 9,
       SPEC_OPT_ATTN_UMMA = 10 };
int spec_set_option(spec_ctx *ctx, int32_t what, int32_t value);

/* Device timeline of the LAST step, recorded while SPEC_OPT_TRACE is on: one record per kernel
 * launch of the step, in launch order. names: HOST [max_records][SPEC_TRACE_NAME_LEN] chars;
 * stamps: HOST [max_records][4] nanoseconds of the GPU's global timer: earliest block start,
 * latest block end, and for the weight-streaming GEMM the moment its first operands had landed
 * in shared memory and the moment its last MMA was issued (all-ones / 0 when a kernel has no
 * such mark). *n_records receives the number of launches of the step. Synchronises. */
#define SPEC_TRACE_NAME_LEN 32
int spec_trace_read(spec_ctx *ctx, int32_t max_records, char *names, uint64_t *stamps, int32_t *n_records);

/* Device time of the five parts of the LAST step, in milliseconds, from events recorded on
 * the stream at the part boundaries: ms[0] heads + lm_head + top-k, ms[1] tree expansion and
 * embedding gather, ms[2] verification forward incl. lm_head, ms[3] acceptance, ms[4] KV
 * compaction (the five parts of the step in Sec. III-B). Needs SPEC_OPT_PHASE_TIMING on during that
 * step (SPEC_E_STATE otherwise). Synchronises. */
int spec_last_step_phase_ms(spec_ctx *ctx, float *ms /* HOST [5] */);

/* Per-launch timing of one kernel kind of the verification forward: while `kind` != 0 every
 * launch of that kernel is bracketed by events, each step ends with a stream synchronise and
 * the elapsed times accumulate. spec_profile_kernel resets the totals. */
enum { SPEC_PROFILE_OFF = 0, SPEC_PROFILE_GATE_UP = 1, SPEC_PROFILE_QKV = 2, SPEC_PROFILE_WO = 3,
       SPEC_PROFILE_DOWN = 4, SPEC_PROFILE_ATTENTION = 5 };
int spec_profile_kernel(spec_ctx *ctx, int32_t kind);
int spec_profile_read(spec_ctx *ctx, double *total_ms, int64_t *launches); /* HOST outputs */

/* Debug taps (tests): copy an intermediate of the LAST step to HOST memory. Synchronises.
 * Rows are ordered [sequence][tree node]. */
enum {
  SPEC_DBG_TOK = 0,      /* int32 [rows]            tree tokens                               */
  SPEC_DBG_POS = 1,      /* int32 [rows]            RoPE positions                            */
  SPEC_DBG_LOGITS = 2,   /* float [rows][vocab]     verify logits (needs SPEC_FLAG_KEEP_LOGITS) */
  SPEC_DBG_HIDDEN = 3,   /* float [rows][d_model]   hidden state after the final norm        */
  SPEC_DBG_ARGMAX = 4,   /* int32 [rows]            per-node argmax of the base logits       */
  SPEC_DBG_PATH = 5,     /* int32 [batch][n_medusa+1] accepted node ids, -1 padded            */
  SPEC_DBG_CAND = 6,     /* int32 [batch][n_medusa+1][kmax] candidate table                   */
  SPEC_DBG_SEQLEN = 7,   /* int32 [batch]           committed tokens per sequence             */
  SPEC_DBG_NEXT_ROOT = 8,/* int32 [batch]           next step's root token                    */
  SPEC_DBG_H_LAST = 9,   /* float [batch][d_model]  hidden state feeding the next heads       */
  SPEC_DBG_STATUS = 10   /* int32 [4]               device status word (0 = clean)            */
};
int spec_debug_read(spec_ctx *ctx, int32_t what, void *host_buf, size_t bytes);

/* Copies cached K and V rows of sequence `seq`, layer `layer`, slots [slot0, slot0+n_slots)
 * to HOST float32 arrays [n_slots][n_kv_heads][head_dim] in logical (unpaged) order. */
int spec_debug_read_kv(spec_ctx *ctx, int32_t seq, int32_t layer, int32_t slot0, int32_t n_slots,
                       float *host_k, float *host_v);

/* Self test of the bounded device-side waits (SPEC_E_TIMEOUT). Every wait of the library's kernels on an
 * mbarrier gives up after a time limit, records ST_TIMEOUT and the place in the device status word and lets
 * the kernel return; the host then reports SPEC_E_TIMEOUT. This entry runs one warp that waits, with a limit
 * of limit_us microseconds (1..100000), on a barrier nothing completes: it returns SPEC_E_TIMEOUT (and
 * spec_last_error names place 99), clears the status word, and the context remains usable. Synchronises. */
int spec_debug_wait_timeout(spec_ctx *ctx, int32_t limit_us);

/* ---- single operations of the verify forward, for unit parity tests and profiling ---- */

/* Pre-tiled weights. The paper has no counterpart: it is a storage layout for this library's GEMM.
 * The weight stream of a step reads every matrix once, tile by tile; out of a row-major matrix
 * a tile is 128 separate 128-byte pieces, which the memory system serves at about 6.4 TB/s. In the
 * pre-tiled image each (128-row tile, 64-column K chunk) unit is 16 KiB contiguous, already in the
 * shared-memory layout the tensor cores read, and a CTA's run of units is one contiguous stretch:
 * about 7.3 TB/s. spec_packed_weight_bytes: size of the image of a [rows, cols] bf16 matrix
 * (cols % 64 == 0; rows are padded to a multiple of 128 with zeros), 0 if the shape is not
 * supported. spec_pack_weight: w DEVICE bf16 row-major [rows, cols] -> packed DEVICE (16-byte
 * aligned, spec_packed_weight_bytes bytes, must not overlap w), enqueued on `cuda_stream`. The
 * caller owns both buffers and may free w afterwards. A context created with
 * SPEC_FLAG_PACKED_WEIGHTS takes images instead of matrices. */
size_t spec_packed_weight_bytes(int32_t rows, int32_t cols);
int spec_pack_weight(const void *w, int32_t rows, int32_t cols, void *packed, void *cuda_stream);

/* y[M,N] (float32, DEVICE) = x[M,K] * W[N,K]^T for DEVICE x and W of type `dtype`
 * (Sec. III-B verification forward: every projection of the base model). bf16 runs the
 * tensor-core weight-streaming kernel: the (128-row weight tile, 64-wide K chunk) units are
 * dealt in equal contiguous runs to `ctas` persistent CTAs, runs that end inside a tile leave
 * float32 partial sums in `scratch` (DEVICE, spec_op_linear_scratch_floats() + 4 floats; the
 * last four hold the call's status word) and a second kernel adds a tile's partial sums in CTA
 * order into y. float32 runs the CUDA-core row kernel (ctas and scratch ignored).
 * M <= 2048; for bf16 K % 64 == 0, M % 16 == 0, N >= 128, 1 <= ctas <= 1024.
 * Synchronises in bf16 mode. */
size_t spec_op_linear_scratch_floats(int32_t M, int32_t N, int32_t K, int32_t ctas);
int spec_op_linear(int32_t dtype, const void *x, const void *w, float *y, int32_t M, int32_t N,
                   int32_t K, int32_t ctas, float *scratch, void *cuda_stream);

/* Syntax-enriched training labels (Sec. III-C). tokens: DEVICE int32 [n_seq][seq_len], each row
 * the token ids of one sample with the fragment marker inserted (L_0). labels: DEVICE int32
 * [n_seq][num_heads + 1][seq_len]; row i of a sample is L_0 shifted left by i and filled up with
 * pad_token, and in every column the labels beyond the column's last frag_token along the head
 * axis are ignore_token (a column without a marker keeps only row 0; the paper leaves that
 * case open). 0 <= num_heads <= 64, n_seq <= 65535; empty input is a no-op. Asynchronous on
 * `cuda_stream`; returns SPEC_E_BADARG / SPEC_E_CUDA on bad arguments / a failed launch. */
int spec_build_labels(const int32_t *tokens, int32_t n_seq, int32_t seq_len, int32_t num_heads,
                      int32_t frag_token, int32_t pad_token, int32_t ignore_token, int32_t *labels,
                      void *cuda_stream);

/* The same operation as spec_op_linear for callers that cannot allocate device memory and so
 * have no scratch buffer to pass: code running where cudaMalloc is forbidden (inside a
 * real-time or safety-certified loop, under a framework whose memory pool is frozen or
 * exhausted, in a plug-in that was handed only its input and output buffers). The paper has no
 * counterpart; this entry exists for those callers only.
 * The partial sums and the status word live in an array built into the library
 * (SPEC_STATIC_SCRATCH_FLOATS float32 values, 8 MiB, held by every GPU that loads the library
 * until the process exits). A call that needs more than that (spec_op_linear_scratch_floats()
 * says how much a shape needs) returns SPEC_E_NOMEM and spec_last_error(NULL) says by how much. A call that
 * succeeds allocates nothing, on host or device (a failing one builds its error text on the host).
 * The first call on each device looks the array's device address up (with that device
 * current) and keeps it; make that first call outside any stream capture. All calls share the
 * one array: it still holds the previous call's partial sums (the library clears the status
 * word itself), and two calls whose kernels overlap on the GPU - different streams, or
 * different host threads - race on it. Serialise them.
 * Arguments, limits, results and synchronisation are those of spec_op_linear. */
#define SPEC_STATIC_SCRATCH_FLOATS (2u << 20)
int spec_op_linear_static(int32_t dtype, const void *x, const void *w, float *y, int32_t M, int32_t N,
                          int32_t K, int32_t ctas, void *cuda_stream);

#ifdef __cplusplus
}
#endif
#endif /* SPEC_DECODE_H_ */
