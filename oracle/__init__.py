"""CPU oracle of the draft-and-verify decode loop (Sec. III-B of the paper).

TEST INFRASTRUCTURE ONLY. Plain, slow NumPy in float64; it shares no code with the
CUDA path and must never be imported by the product package. Only tests, the smoke
check and the benchmark's CPU-baseline leg may call it.

What it computes, and what each part is pinned to (tests marked "not gpu"):

* decoder forward (RMSNorm, rotate-half RoPE, masked attention, SwiGLU, untied lm_head):
  pinned to the transformers library's Llama implementation on a small shape with random
  gains, to closed forms (constant-vector RMSNorm, equal-key attention = mean of values,
  RoPE relative-position property) and to cache-vs-recompute equivalence;
* extra decoding heads and top-k: top-k pinned to a full stable sort; head block pinned to
  closed forms (zero matrix -> identity + SiLU(bias));
* candidate tree and ancestor mask: pinned to brute-force parent chasing and to the node
  counts per depth of the enumeration;
* greedy acceptance / longest accepted prefix: pinned to brute force over every
  root-to-node path;
* typical acceptance (Eq. 1): pinned to the one-hot and uniform closed forms;
* whole loop: pinned to plain no-cache greedy decoding (lossless property), for chain
  trees and for arbitrary trees and drafts.
* per-step accepted counts with the real random heads: parity unpinned (the paper prints
  no worked example); they are fixed only by the invariants above.
"""
