// Prompt processing as dense products on the tensor cores (the first step of inference in Section 3.2: the
// whole prompt goes through M once, which fills the KV cache and yields every row's per-sublayer cosine
// similarity, the summands of C_l).
//
// With hundreds of rows the sublayer products are dense contractions, so they run as tcgen05 GEMMs: operand
// tiles staged in shared memory by TMA (128-byte swizzle), accumulators in tensor memory, one elected thread
// issuing tcgen05.mma, four epilogue warps reading the accumulators back with tcgen05.ld. Causal attention
// over the prompt is a flash-style kernel on mma.sync. Row-wise work (embedding, RMSNorm, residual add with
// the cosine sums) runs one CTA per row.
#pragma once
#include <cuda.h>
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

namespace asd {

constexpr int kGemmBM = 128;  // rows of the activation tile of one CTA (the M of tcgen05.mma)
constexpr int kGemmBK = 64;   // reduction elements per pipeline stage: 128 bytes, one swizzle span

enum GemmEpilogue : int {
    kGemmF32 = 0,     // C[r, n] fp32
    kGemmQkv = 1,     // rotary embedding, bf16, queries to q, keys and values appended to the KV cache
    kGemmSwiglu = 2,  // columns alternate gate_i, up_i: t[r, i] = bf16(silu(gate_i) * up_i)
};

// What the epilogue of one GEMM does with the accumulators. Row r of the product is prompt row r of this chunk.
struct GemmEpi {
    int mode;
    int* err;  // device error words shared with the pass kernel (word 0 = code)
    // kGemmF32
    float* c;
    int ldc;
    int k_split;            // 1, or 2: the reduction dimension is cut in two halves, each a work item of its own
    size_t c_split_stride;  // floats between the partial results of the halves (the caller adds them: half 0 + half 1)
    // kGemmQkv: columns are [q | k | v]; inside every q and k head the rotary partners (j, j + head_dim/2) are
    // neighbours (2j, 2j+1); v columns are in natural order. Row r sits at position pos0 + r.
    __nv_bfloat16 *q, *k_cache, *v_cache;
    const float *rope_cos, *rope_sin;
    int pos0, d_model, kv_dim, head_dim;
    // kGemmSwiglu
    __nv_bfloat16* t;
    int ldt;
};

cudaError_t configure_prefill(int max_smem);

// C[M, N] = A[M, K] * W[N, K]^T, bf16 operands described by 2-D tensor maps (boxes of 64 x 128 for A, 64 x bn for W,
// 128-byte swizzle), fp32 accumulation. bn is 128 or 256.
cudaError_t launch_gemm_tn(const CUtensorMap& tm_a, const CUtensorMap& tm_w, int M, int N, int K, int bn, const GemmEpi& ep,
                           cudaStream_t s);

// x[r, :] = embedding row of tokens[r] (fp32); xn[r, :] = bf16(RMSNorm(x[r]) * gain)
cudaError_t launch_embed_norm(const int* tokens, int n_rows, int d, int vocab, const __nv_bfloat16* embed, const __nv_bfloat16* gain,
                              float eps, float* x, __nv_bfloat16* xn, cudaStream_t s);

// y = x + c (in place in x), cos_out[r] = <x, y> / (|x| |y|) (Section 3.2), and, when gain is given,
// xn[r, :] = bf16(RMSNorm(y) * gain) for the next sublayer
cudaError_t launch_resid_norm(int n_rows, int d, float* x, const float* c, const float* c2, const __nv_bfloat16* gain, float eps, __nv_bfloat16* xn,
                              float* cos_out, cudaStream_t s);

// sumcos[b] += sum over rows of cos_rows[b * stride + r], rows in a fixed order, double precision
cudaError_t launch_sumcos(const float* cos_rows, int stride, int n_rows, int n_sub, double* sumcos, cudaStream_t s);

// causal attention of prompt rows [0, n_rows) at positions pos0 + r over keys 0 .. pos0 + r of the cache
cudaError_t launch_flash_prefill(const __nv_bfloat16* q, const __nv_bfloat16* k_cache, const __nv_bfloat16* v_cache, __nv_bfloat16* out,
                                 int n_rows, int pos0, int d_model, int kv_dim, int head_dim, int n_heads, int n_kv_heads, int max_seq,
                                 float scale, cudaStream_t s);

}  // namespace asd
