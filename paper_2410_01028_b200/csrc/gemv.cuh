// Fused RMSNorm -> GEMV -> epilogue for M <= 9 activation rows (decode, draft, verify, chunked prefill).
//
// One CTA per SM streams a contiguous slab of weight rows exactly once with 16-byte read-only loads.
// A warp work item is one PAIR of weight rows times one 1024-element segment of the reduction dimension:
// 4 KB of weights in flight per warp, with the next item's loads issued before the current item's math.
// The pair is the unit every epilogue needs together: the two rotary partners of a q/k head, gate_i and
// up_i of SwiGLU, or simply two neighbouring rows.
//
// Reduction order is fixed and does not depend on M: a lane sums its eight products of a 16-byte chunk in
// element order, its four chunks of a segment in order, lanes are combined by an xor butterfly, segments in
// ascending order. Row m of an M-row pass is therefore bit-identical to the same row of a 1-row pass, which
// is what makes the speculative output equal the autoregressive output bit for bit (Section 1).
//
// Epilogues
//   plain    : out[m][r] = a                                   (fp32)
//   swiglu   : t[m][i] = bf16(silu(gate_i) * up_i)
//   residual : y = x + a in place; per-row <x,y>, |x|^2, |y|^2 by warp shuffles, one block-level finish per
//              CTA, and the last CTA to arrive turns the per-CTA partials into the cosine similarity of the
//              hidden state before and after the sublayer (summand of C_l, Section 3.2)
#pragma once
#include <limits.h>

#include "common.cuh"

namespace asd {

struct WeightItem {
    uint4 a[4], b[4];
};

// the unit of work is a pair of neighbouring weight rows (gate_i and up_i for the SwiGLU epilogue)
__device__ __forceinline__ void pair_rows(int pair, int& ra, int& rb) {
    ra = 2 * pair;
    rb = 2 * pair + 1;
}

template <int EPI>
__device__ __forceinline__ void load_item(const GemvParams& p, int pair0, int n_seg, int it, int lane, WeightItem& w) {
    const int pl = it / n_seg, seg = it - pl * n_seg;
    int ra, rb;
    pair_rows(pair0 + pl, ra, rb);
    rb = min(rb, p.n_rows - 1);  // an odd row count: the missing partner re-reads the last row and is discarded
    const __nv_bfloat16* Wa = p.W + (size_t)ra * p.n_in;
    const __nv_bfloat16* Wb = p.W + (size_t)rb * p.n_in;
    const int k0 = seg * kSeg + lane * 8;
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        const int k = k0 + i * 256;
        if (k < p.n_in) {
            w.a[i] = ldg_stream(Wa + k);
            w.b[i] = ldg_stream(Wb + k);
        } else {
            w.a[i] = make_uint4(0, 0, 0, 0);
            w.b[i] = make_uint4(0, 0, 0, 0);
        }
    }
}

__device__ __forceinline__ float dot8(const uint4& w, const float (&x)[8], float acc) {
    acc = fmaf(bf_lo(w.x), x[0], acc);
    acc = fmaf(bf_hi(w.x), x[1], acc);
    acc = fmaf(bf_lo(w.y), x[2], acc);
    acc = fmaf(bf_hi(w.y), x[3], acc);
    acc = fmaf(bf_lo(w.z), x[4], acc);
    acc = fmaf(bf_hi(w.z), x[5], acc);
    acc = fmaf(bf_lo(w.w), x[6], acc);
    acc = fmaf(bf_hi(w.w), x[7], acc);
    return acc;
}

template <int M>
__device__ __forceinline__ void compute_item(const WeightItem& w, const __nv_bfloat16* xs, int n_in, int k0,
                                             float (&acc_a)[M], float (&acc_b)[M]) {
#pragma unroll
    for (int m = 0; m < M; ++m) acc_a[m] = acc_b[m] = 0.f;
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        const int k = k0 + i * 256;
        if (k < n_in) {
#pragma unroll
            for (int m = 0; m < M; ++m) {
                const uint4 xv = *reinterpret_cast<const uint4*>(xs + (size_t)m * n_in + k);
                const float x[8] = {bf_lo(xv.x), bf_hi(xv.x), bf_lo(xv.y), bf_hi(xv.y),
                                    bf_lo(xv.z), bf_hi(xv.z), bf_lo(xv.w), bf_hi(xv.w)};
                acc_a[m] = dot8(w.a[i], x, acc_a[m]);
                acc_b[m] = dot8(w.b[i], x, acc_b[m]);
            }
        }
    }
}

// Signal arrival of this CTA; returns true in every thread of the last CTA to arrive.
__device__ __forceinline__ bool last_cta_arrives(unsigned* counter, int* flag_smem) {
    __threadfence();
    __syncthreads();
    if (threadIdx.x == 0) {
        const unsigned t = atomicAdd(counter, 1u);
        *flag_smem = (t == gridDim.x - 1) ? 1 : 0;
    }
    __syncthreads();
    const bool last = *flag_smem != 0;
    if (last) __threadfence();
    return last;
}

template <int M, int EPI, bool NORM>
__global__ void __launch_bounds__(kGemvThreads, 1) gemv_kernel(const GemvParams p) {
    extern __shared__ __align__(16) unsigned char smem_raw[];
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int n_in = p.n_in;
    const int n_pairs = (p.n_rows + 1) >> 1;
    const int pair0 = (int)((long long)blockIdx.x * n_pairs / gridDim.x);
    const int pair1 = (int)((long long)(blockIdx.x + 1) * n_pairs / gridDim.x);
    const int np = pair1 - pair0;
    const int n_seg = (n_in + kSeg - 1) / kSeg;
    const int n_items = np * n_seg;
    const int max_np = (n_pairs + gridDim.x - 1) / gridDim.x;

    float* red = reinterpret_cast<float*>(smem_raw);           // [kGemvWarps][kMaxRows * 4]
    int* flag = reinterpret_cast<int*>(red + kGemvWarps * kMaxRows * 4);
    float* psum = reinterpret_cast<float*>(flag + 4);          // [n_items][2][M]
    size_t psum_floats = ((size_t)max_np * n_seg * 2 * M + 3) & ~(size_t)3;
    __nv_bfloat16* xs_smem = reinterpret_cast<__nv_bfloat16*>(psum + psum_floats);  // [M][n_in]

    // ---- the first item's weights do not depend on the activations: get them moving before the prologue
    WeightItem cur;
    int it = warp;
    if (it < n_items) load_item<EPI>(p, pair0, n_seg, it, lane, cur);

    // ---- prologue: activations -> bf16 rows in shared memory (RMSNorm fused here)
    const __nv_bfloat16* xs;
    if (NORM) {
        const float* xf = reinterpret_cast<const float*>(p.x);
        float ss[M];
#pragma unroll
        for (int m = 0; m < M; ++m) {
            float s = 0.f;
            for (int i = tid * 4; i < n_in; i += kGemvThreads * 4) {
                const float4 v = *reinterpret_cast<const float4*>(xf + (size_t)m * n_in + i);
                s = fmaf(v.x, v.x, s);
                s = fmaf(v.y, v.y, s);
                s = fmaf(v.z, v.z, s);
                s = fmaf(v.w, v.w, s);
            }
            s = warp_sum(s);
            if (lane == 0) red[warp * (kMaxRows * 4) + m] = s;
        }
        __syncthreads();
#pragma unroll
        for (int m = 0; m < M; ++m) {
            float s = 0.f;
#pragma unroll
            for (int w = 0; w < kGemvWarps; ++w) s += red[w * (kMaxRows * 4) + m];
            ss[m] = 1.0f / sqrtf(s / (float)n_in + p.eps);
        }
        for (int i = tid * 4; i < n_in; i += kGemvThreads * 4) {
            const uint2 gv = *reinterpret_cast<const uint2*>(p.gain + i);
            const float g0 = bf_lo(gv.x), g1 = bf_hi(gv.x), g2 = bf_lo(gv.y), g3 = bf_hi(gv.y);
#pragma unroll
            for (int m = 0; m < M; ++m) {
                const float4 v = *reinterpret_cast<const float4*>(xf + (size_t)m * n_in + i);
                __nv_bfloat162 lo = __floats2bfloat162_rn(v.x * ss[m] * g0, v.y * ss[m] * g1);
                __nv_bfloat162 hi = __floats2bfloat162_rn(v.z * ss[m] * g2, v.w * ss[m] * g3);
                uint2 o;
                o.x = *reinterpret_cast<uint32_t*>(&lo);
                o.y = *reinterpret_cast<uint32_t*>(&hi);
                *reinterpret_cast<uint2*>(xs_smem + (size_t)m * n_in + i) = o;
            }
        }
        xs = xs_smem;
        __syncthreads();
    } else {
        const __nv_bfloat16* xb = reinterpret_cast<const __nv_bfloat16*>(p.x);
        if (p.x_in_smem) {
            const int n16 = M * n_in / 8;
            for (int i = tid; i < n16; i += kGemvThreads)
                reinterpret_cast<uint4*>(xs_smem)[i] = reinterpret_cast<const uint4*>(xb)[i];
            xs = xs_smem;
            __syncthreads();
        } else {
            xs = xb;
        }
    }

    // ---- main loop: stream the slab, two items in registers per warp
    while (it < n_items) {
        const int nxt = it + kGemvWarps;
        WeightItem next;
        if (nxt < n_items) load_item<EPI>(p, pair0, n_seg, nxt, lane, next);
        const int pl = it / n_seg, seg = it - pl * n_seg;
        float acc_a[M], acc_b[M];
        compute_item<M>(cur, xs, n_in, seg * kSeg + lane * 8, acc_a, acc_b);
#pragma unroll
        for (int m = 0; m < M; ++m) {
            acc_a[m] = warp_sum(acc_a[m]);
            acc_b[m] = warp_sum(acc_b[m]);
        }
        if (lane == 0) {
#pragma unroll
            for (int m = 0; m < M; ++m) {
                psum[((size_t)it * 2 + 0) * M + m] = acc_a[m];
                psum[((size_t)it * 2 + 1) * M + m] = acc_b[m];
            }
        }
        if (nxt < n_items) cur = next;
        it = nxt;
    }
    __syncthreads();

    // ---- epilogue: thread t owns pairs t, t+512, ... of this CTA and all M rows of them
    float s_loc[M][3];
#pragma unroll
    for (int m = 0; m < M; ++m) s_loc[m][0] = s_loc[m][1] = s_loc[m][2] = 0.f;
    for (int pl = tid; pl < np; pl += kGemvThreads) {
        int ra, rb;
        pair_rows(pair0 + pl, ra, rb);
        const bool has_b = rb < p.n_rows;
#pragma unroll
        for (int m = 0; m < M; ++m) {
            float va = 0.f, vb = 0.f;
            for (int sgi = 0; sgi < n_seg; ++sgi) {
                va += psum[((size_t)(pl * n_seg + sgi) * 2 + 0) * M + m];
                vb += psum[((size_t)(pl * n_seg + sgi) * 2 + 1) * M + m];
            }
            if (EPI == kEpiPlain) {
                float* out = reinterpret_cast<float*>(p.out);
                out[(size_t)m * p.n_rows + ra] = va;
                if (has_b) out[(size_t)m * p.n_rows + rb] = vb;
            } else if (EPI == kEpiSwiglu) {
                const float t = va / (1.0f + expf(-va)) * vb;
                reinterpret_cast<__nv_bfloat16*>(p.out)[(size_t)m * (p.n_rows >> 1) + (pair0 + pl)] = __float2bfloat16_rn(t);
            } else if (EPI == kEpiResidual) {
                float* out = reinterpret_cast<float*>(p.out);
                {
                    const float x0 = out[(size_t)m * p.n_rows + ra];
                    const float y0 = x0 + va;
                    out[(size_t)m * p.n_rows + ra] = y0;
                    s_loc[m][0] = fmaf(x0, y0, s_loc[m][0]);
                    s_loc[m][1] = fmaf(x0, x0, s_loc[m][1]);
                    s_loc[m][2] = fmaf(y0, y0, s_loc[m][2]);
                }
                if (has_b) {
                    const float x1 = out[(size_t)m * p.n_rows + rb];
                    const float y1 = x1 + vb;
                    out[(size_t)m * p.n_rows + rb] = y1;
                    s_loc[m][0] = fmaf(x1, y1, s_loc[m][0]);
                    s_loc[m][1] = fmaf(x1, x1, s_loc[m][1]);
                    s_loc[m][2] = fmaf(y1, y1, s_loc[m][2]);
                }
            }
        }
    }

    if (EPI == kEpiResidual) {
        // warp-shuffle partial dot and norm products, then one block-level finish
#pragma unroll
        for (int m = 0; m < M; ++m)
#pragma unroll
            for (int j = 0; j < 3; ++j) {
                const float v = warp_sum(s_loc[m][j]);
                if (lane == 0) red[warp * (kMaxRows * 4) + m * 4 + j] = v;
            }
        __syncthreads();
        if (tid < M * 3) {
            const int m = tid / 3, j = tid - m * 3;
            float tot = 0.f;
#pragma unroll
            for (int w = 0; w < kGemvWarps; ++w) tot += red[w * (kMaxRows * 4) + m * 4 + j];
            p.partials[((size_t)blockIdx.x * kMaxRows + m) * 4 + j] = tot;
        }
        if (last_cta_arrives(p.counter, flag)) {
            // one warp per activation row: lanes add the per-CTA partials b = lane, lane+32, ... in order, then an
            // xor butterfly in double precision (fixed order, independent of the row count)
            if (warp < M) {
                double sxy = 0, sxx = 0, syy = 0;
                for (unsigned b = lane; b < gridDim.x; b += 32) {
                    sxy += (double)__ldcg(p.partials + ((size_t)b * kMaxRows + warp) * 4 + 0);
                    sxx += (double)__ldcg(p.partials + ((size_t)b * kMaxRows + warp) * 4 + 1);
                    syy += (double)__ldcg(p.partials + ((size_t)b * kMaxRows + warp) * 4 + 2);
                }
#pragma unroll
                for (int o = 16; o > 0; o >>= 1) {
                    sxy += __shfl_xor_sync(0xffffffffu, sxy, o);
                    sxx += __shfl_xor_sync(0xffffffffu, sxx, o);
                    syy += __shfl_xor_sync(0xffffffffu, syy, o);
                }
                if (lane == 0) {
                    const double c = sxy / fmax(sqrt(sxx) * sqrt(syy), 1e-30);
                    p.cos_out[warp] = (float)c;
                    red[warp] = (float)c;
                }
            }
            __syncthreads();
            if (tid == 0) {
                if (p.sumcos) {
                    double acc = *p.sumcos;
                    for (int m = 0; m < M; ++m) acc += (double)red[m];
                    *p.sumcos = acc;
                }
                *p.counter = 0u;
            }
        }
    }
}

}  // namespace asd
