// Kernels of sampling-based decoding and verification (Section 1; see sample.cu).
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

namespace asd {

// kinds of draw at one position of the sequence: a draft model's draw, the acceptance test of that draft, and the
// full model's own draw (first token, plain sampled decoding, the redrawn token after a rejection, the extra token)
enum DrawKind : int { kDrawDraft = 0, kDrawAccept = 1, kDrawTarget = 2 };

// probs[r][0..V) = softmax(logits[r][0..V) / T) for r < rows (device pointers; double precision)
cudaError_t launch_softmax_rows(const float* logits, int rows, int V, double T, double* probs, cudaStream_t s);
// one token drawn from probs[0..V) with the uniform number of (seed, position, kind); written to token_out and, when
// given, to token_out2
cudaError_t launch_draw(const double* probs, int V, unsigned long long seed, int position, int kind, int* token_out, int* token_out2,
                        cudaStream_t s);
// acceptance of the k drafts row_tokens[1..k] (p: k + 1 rows, q: k rows); accept_out[0] = a, then a + 1 tokens
cudaError_t launch_accept(const double* p, const double* q, const int* row_tokens, int k, int V, unsigned long long seed, int pos0,
                          int* accept_out, cudaStream_t s);

}  // namespace asd
