// Sampling-based decoding and verification (Section 1: when sampling is used, drafted tokens are accepted so that
// the output keeps the full model's distribution; the T > 0 columns of Tables 3 and 4).
//
// The pass kernel leaves the logits of its rows in device memory. Two small kernels follow it on the stream:
//   softmax_rows_kernel   a cluster of eight CTAs per row: p_i = exp(l_i / T - max) / sum, in double precision
//   draw_kernel           one CTA: a token drawn from one row by inverse-CDF sampling (first token, plain sampled
//                         decoding, a draft step's draw from the draft model's distribution q)
//   accept_kernel         one CTA: a drafted token x is accepted when its uniform number r satisfies r q(x) < p(x);
//                         the first rejected one is redrawn from max(0, p - q); a fully accepted round draws one
//                         more token from the last row
// Every decision (a comparison of r q with p, the search of a cumulative sum) is taken in double precision.
// Random numbers: Philox4x32-10 (Salmon, Moraes, Dror, Shaw, SC'11) with key = seed and counter = (position of the
// token being chosen, kind of draw, 0, 0); the first output word x gives the uniform number (x + 1/2) / 2^32.
#include "sample.h"

#include <cooperative_groups.h>
#include <limits.h>
#include <math.h>

namespace cg = cooperative_groups;

namespace asd {

constexpr int kSampleThreads = 1024;

// ten rounds of (c0,c1,c2,c3) <- (hi(B*c2) ^ c1 ^ k0, lo(B*c2), hi(A*c0) ^ c3 ^ k1, lo(A*c0)), key += Weyl constants
__device__ __forceinline__ uint32_t philox_first_word(uint32_t c0, uint32_t c1, uint32_t c2, uint32_t c3, uint32_t k0, uint32_t k1) {
    constexpr uint32_t kMulA = 0xD2511F53u, kMulB = 0xCD9E8D57u, kWeylA = 0x9E3779B9u, kWeylB = 0xBB67AE85u;
#pragma unroll
    for (int r = 0; r < 10; ++r) {
        const uint32_t hi_a = __umulhi(kMulA, c0), lo_a = kMulA * c0;
        const uint32_t hi_b = __umulhi(kMulB, c2), lo_b = kMulB * c2;
        const uint32_t n0 = hi_b ^ c1 ^ k0, n2 = hi_a ^ c3 ^ k1;
        c0 = n0, c1 = lo_b, c2 = n2, c3 = lo_a;
        k0 += kWeylA, k1 += kWeylB;
    }
    return c0;
}

__device__ __forceinline__ double uniform_number(unsigned long long seed, uint32_t position, uint32_t kind) {
    const uint32_t w = philox_first_word(position, kind, 0u, 0u, (uint32_t)seed, (uint32_t)(seed >> 32));
    return ((double)w + 0.5) * (1.0 / 4294967296.0);
}

// block-wide reductions over kSampleThreads threads (fixed order: lanes by butterfly, warps in index order)
__device__ double block_sum(double v, double* red) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    __syncthreads();
    if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = v;
    __syncthreads();
    double s = 0;
    for (int w = 0; w < kSampleThreads / 32; ++w) s += red[w];
    return s;
}
__device__ double block_max(double v, double* red) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v = fmax(v, __shfl_xor_sync(0xffffffffu, v, o));
    __syncthreads();
    if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = v;
    __syncthreads();
    double s = -INFINITY;
    for (int w = 0; w < kSampleThreads / 32; ++w) s = fmax(s, red[w]);
    return s;
}

// probs[row][i] = softmax(logits[row] / T)_i. A cluster of eight CTAs per row, each with an eighth of the vocabulary:
// the CTAs exchange their maximum and their sum through distributed shared memory (the eight sums are added in rank
// order), so the double-precision exponentials of a row run on eight SMs.
constexpr int kSoftmaxCluster = 8;
__global__ void __cluster_dims__(kSoftmaxCluster, 1, 1) __launch_bounds__(kSampleThreads)
    softmax_rows_kernel(const float* logits, int V, double T, double* probs) {
    cg::cluster_group cluster = cg::this_cluster();
    __shared__ double red[kSampleThreads / 32];
    __shared__ double mine[2];  // this CTA's largest logit and its sum of exponentials, read by the other CTAs of the cluster
    const int row = blockIdx.x / kSoftmaxCluster, rank = (int)cluster.block_rank();
    const int per = (V + kSoftmaxCluster - 1) / kSoftmaxCluster;
    const int i0 = min(V, rank * per), i1 = min(V, i0 + per);
    const float* l = logits + (size_t)row * V;
    double* p = probs + (size_t)row * V;
    // the largest logit in single precision (exact: it is one of the inputs), then its quotient: the same value as the
    // maximum of the quotients, without a double-precision division per element
    float mxf = -INFINITY;
    for (int i = i0 + threadIdx.x; i < i1; i += kSampleThreads) mxf = fmaxf(mxf, l[i]);
    const double mx_local = block_max((double)mxf, red);
    if (threadIdx.x == 0) mine[0] = mx_local;
    cluster.sync();
    double mx = -INFINITY;
    for (int r = 0; r < kSoftmaxCluster; ++r) mx = fmax(mx, *cluster.map_shared_rank(&mine[0], r));
    mx /= T;
    double sum = 0;
    for (int i = i0 + threadIdx.x; i < i1; i += kSampleThreads) {
        const double e = exp((double)l[i] / T - mx);
        p[i] = e;
        sum += e;
    }
    sum = block_sum(sum, red);
    if (threadIdx.x == 0) mine[1] = sum;
    cluster.sync();
    double total = 0;
    for (int r = 0; r < kSoftmaxCluster; ++r) total += *cluster.map_shared_rank(&mine[1], r);
    for (int i = i0 + threadIdx.x; i < i1; i += kSampleThreads) p[i] /= total;
    cluster.sync();  // no CTA leaves while another may still read its shared memory
}

// Inverse-CDF sampling by the whole block from non-negative weights w_i = max(0, a_i - b_i) (b may be null: w = a):
// the smallest i with w_0 + ... + w_i > u * total; if rounding leaves none, the last index with w_i > 0. Warp w owns
// the contiguous indices [w * span, (w + 1) * span), span a multiple of 32, and walks them in rows of 32 consecutive
// elements (coalesced loads); the cumulative sum at an index is the sum of the earlier warps' totals, of the warp's
// earlier rows and of the row's inclusive scan (a warp's total is added column-wise, so the two can differ in the last
// bits: a warp that finds no index although its total reaches past the target leaves the pick to the next warp). Returns the token in every thread; *total_out = total.
__device__ int block_sample(const double* a, const double* b, int V, double u, double* red, int* pick, double* total_out) {
    constexpr int kWarps = kSampleThreads / 32;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int span = ((V + kWarps - 1) / kWarps + 31) / 32 * 32;
    const int i0 = min(V, warp * span), i1 = min(V, i0 + span);
    auto weight = [&](int i) { return b ? fmax(0.0, a[i] - b[i]) : a[i]; };
    // warp total: every lane adds its column of the rows in order (loads of eight rows in flight), then a butterfly
    double wtot = 0;
    int last_pos = -1;
    for (int r = i0; r < i1; r += 8 * 32) {
        double w[8];
#pragma unroll
        for (int j = 0; j < 8; ++j) {
            const int i = r + j * 32 + lane;
            w[j] = i < i1 ? weight(i) : 0.0;
        }
#pragma unroll
        for (int j = 0; j < 8; ++j) {
            wtot += w[j];
            if (w[j] > 0) last_pos = r + j * 32 + lane;
        }
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
        wtot += __shfl_xor_sync(0xffffffffu, wtot, o);
        last_pos = max(last_pos, __shfl_xor_sync(0xffffffffu, last_pos, o));
    }
    __syncthreads();
    if (lane == 0) red[warp] = wtot;
    if (threadIdx.x == 0) pick[0] = INT_MAX, pick[1] = -1;
    __syncthreads();
    double before = 0, total = 0;
    for (int w = 0; w < kWarps; ++w) {
        if (w < warp) before += red[w];
        total += red[w];
    }
    const double target = u * total;
    // Every warp whose range reaches past the target looks for the first index with a positive weight whose cumulative
    // sum exceeds the target; the smallest reported index wins (for warps behind the crossing that is their first
    // positive weight).
    if (before + wtot > target) {
        double run = before;
        for (int r = i0; r < i1; r += 32) {
            const int i = r + lane;
            const double w = i < i1 ? weight(i) : 0.0;
            double s = w;  // inclusive scan of the row
#pragma unroll
            for (int o = 1; o < 32; o <<= 1) {
                const double n = __shfl_up_sync(0xffffffffu, s, o);
                if (lane >= o) s += n;
            }
            const unsigned hit = __ballot_sync(0xffffffffu, w > 0 && run + s > target);
            if (hit) {
                if (lane == 0) atomicMin(&pick[0], r + __ffs(hit) - 1);
                break;
            }
            run += __shfl_sync(0xffffffffu, s, 31);
        }
    }
    if (lane == 0 && last_pos >= 0) atomicMax(&pick[1], last_pos);
    __syncthreads();
    if (total_out) *total_out = total;
    const int tok = pick[0] != INT_MAX ? pick[0] : max(pick[1], 0);
    __syncthreads();
    return tok;
}

// one token drawn from probs (one row) with the uniform number of (seed, position, kind)
__global__ void __launch_bounds__(kSampleThreads) draw_kernel(const double* probs, int V, unsigned long long seed, int position, int kind,
                                                               int* token_out, int* token_out2) {
    __shared__ double red[kSampleThreads / 32];
    __shared__ int pick[2];
    const int tok = block_sample(probs, nullptr, V, uniform_number(seed, (uint32_t)position, (uint32_t)kind), red, pick, nullptr);
    if (threadIdx.x == 0) {
        *token_out = tok;
        if (token_out2) *token_out2 = tok;
    }
}

// Verification of k drafts: p has k + 1 rows, q has k rows, row_tokens[j + 1] is the draft at position pos0 + 1 + j.
// accept_out[0] = a, accept_out[1 .. a + 1] = the accepted drafts followed by the redrawn / extra token.
__global__ void __launch_bounds__(kSampleThreads) accept_kernel(const double* p, const double* q, const int* row_tokens, int k, int V,
                                                                 unsigned long long seed, int pos0, int* accept_out) {
    __shared__ double red[kSampleThreads / 32];
    __shared__ int pick[2];
    int a = 0;
    for (; a < k; ++a) {
        const int x = min(max(row_tokens[a + 1], 0), V - 1);
        const double pj = p[(size_t)a * V + x], qj = q[(size_t)a * V + x];
        const double r = uniform_number(seed, (uint32_t)(pos0 + 1 + a), kDrawAccept);
        if (r * qj < pj) {  // r < min(1, p/q), written without the division
            if (threadIdx.x == 0) accept_out[1 + a] = x;
            continue;
        }
        const double u = uniform_number(seed, (uint32_t)(pos0 + 1 + a), kDrawTarget);
        double mass;
        int tok = block_sample(p + (size_t)a * V, q + (size_t)a * V, V, u, red, pick, &mass);
        if (!(mass > 0)) tok = block_sample(p + (size_t)a * V, nullptr, V, u, red, pick, nullptr);  // p == q to rounding
        if (threadIdx.x == 0) {
            accept_out[1 + a] = tok;
            accept_out[0] = a;
        }
        return;
    }
    const int tok = block_sample(p + (size_t)k * V, nullptr, V, uniform_number(seed, (uint32_t)(pos0 + 1 + k), kDrawTarget), red, pick, nullptr);
    if (threadIdx.x == 0) {
        accept_out[1 + k] = tok;
        accept_out[0] = k;
    }
}

cudaError_t launch_softmax_rows(const float* logits, int rows, int V, double T, double* probs, cudaStream_t s) {
    if (rows <= 0 || V <= 0 || !(T > 0)) return cudaErrorInvalidValue;
    softmax_rows_kernel<<<rows * kSoftmaxCluster, kSampleThreads, 0, s>>>(logits, V, T, probs);
    return cudaGetLastError();
}
cudaError_t launch_draw(const double* probs, int V, unsigned long long seed, int position, int kind, int* token_out, int* token_out2,
                        cudaStream_t s) {
    draw_kernel<<<1, kSampleThreads, 0, s>>>(probs, V, seed, position, kind, token_out, token_out2);
    return cudaGetLastError();
}
cudaError_t launch_accept(const double* p, const double* q, const int* row_tokens, int k, int V, unsigned long long seed, int pos0,
                          int* accept_out, cudaStream_t s) {
    accept_kernel<<<1, kSampleThreads, 0, s>>>(p, q, row_tokens, k, V, seed, pos0, accept_out);
    return cudaGetLastError();
}

}  // namespace asd
