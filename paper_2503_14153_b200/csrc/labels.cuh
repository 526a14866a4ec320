// Syntax-enriched training labels (Sec. III-C): Labels[i][s] = L0[s + i] (padded with [PAD]
// past the end); per column the last [FRAG] along the head axis is found and every label
// beyond it becomes [IGNORE] (a column without a marker keeps only row 0). HBM-bound: the
// sequence is read once through a shared-memory window of blockDim.x + num_heads tokens and
// the (num_heads + 1) x seq_len matrix is written once, each row coalesced.
#pragma once
#include <stdint.h>

namespace spec {

constexpr int LABEL_THREADS = 256;
constexpr int LABEL_MAX_HEADS = 64;

__global__ void __launch_bounds__(LABEL_THREADS)
build_labels_kernel(const int32_t* __restrict__ tokens, int seq_len, int num_heads, int32_t frag, int32_t pad,
                    int32_t ignore, int32_t* __restrict__ labels) {
  __shared__ int32_t win[LABEL_THREADS + LABEL_MAX_HEADS];
  const int seq = blockIdx.y;
  const int s0 = blockIdx.x * LABEL_THREADS;
  const int32_t* l0 = tokens + (size_t)seq * seq_len;
  for (int c = threadIdx.x; c < LABEL_THREADS + num_heads; c += LABEL_THREADS) {
    const int s = s0 + c;
    win[c] = s < seq_len ? l0[s] : pad;
  }
  __syncthreads();
  const int s = s0 + threadIdx.x;
  if (s >= seq_len) return;
  int last = 0;
  for (int i = 0; i <= num_heads; ++i)
    if (win[threadIdx.x + i] == frag) last = i;
  int32_t* out = labels + (size_t)seq * (num_heads + 1) * seq_len + s;
  for (int i = 0; i <= num_heads; ++i) out[(size_t)i * seq_len] = i <= last ? win[threadIdx.x + i] : ignore;
}

}  // namespace spec
