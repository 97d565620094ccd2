// Contiguous-KV attention for M <= 9 query rows (decode: 1 row; verify and chunked prefill: several causal
// rows), split over the sequence.
//
// Work item = (kv head, chunk of 128 keys). Chunks are aligned to absolute positions, so the partition of the
// keys of a row, the order of the sums inside a chunk and the order in which chunks are merged do not depend
// on how many rows share the pass: row m of a (k+1)-row verify pass is bit-identical to a 1-row decode pass
// at the same position. Each K/V tile is staged once in shared memory and used by all M rows (and all query
// heads of the group). The CTA that finishes last for a kv head merges that head's chunk partials in chunk
// order and writes the bf16 attention output; no separate merge launch, no atomics on data.
#pragma once
#include "common.cuh"

namespace asd {

template <int M>
__global__ void __launch_bounds__(kAttnThreads) attn_kernel(const AttnParams p) {
    extern __shared__ __align__(16) unsigned char smem_raw[];
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int hd = p.head_dim;
    const int kstride = hd + 8;  // bf16 elements; 16 bytes of padding keep 16-byte row reads conflict free
    const int chunk = blockIdx.x, kvh = blockIdx.y;
    const int group = p.n_heads / p.n_kv_heads;
    const int key0 = chunk * kAttnChunk;
    const int last_pos = p.pos0 + M - 1;
    const int n_valid = min(kAttnChunk, last_pos + 1 - key0);  // keys of this chunk that exist (>= 1)

    __nv_bfloat16* Ks = reinterpret_cast<__nv_bfloat16*>(smem_raw);           // [128][hd+8]
    __nv_bfloat16* Vs = Ks + (size_t)kAttnChunk * kstride;                    // [128][hd]
    float* qs = reinterpret_cast<float*>(Vs + (size_t)kAttnChunk * hd);      // [M][hd]
    float* Ps = qs + M * hd;                                                  // [M][128]
    float* red = Ps + M * kAttnChunk;                                         // [4][kMaxRows]
    int* flag = reinterpret_cast<int*>(red + 4 * kMaxRows);

    // ---- stage the K and V tiles (16-byte coalesced loads; rows past n_valid are zero)
    const int vec_per_row = hd / 8;
    for (int i = tid; i < kAttnChunk * vec_per_row; i += kAttnThreads) {
        const int r = i / vec_per_row, c = i - r * vec_per_row;
        uint4 kv = make_uint4(0, 0, 0, 0), vv = make_uint4(0, 0, 0, 0);
        if (r < n_valid) {
            const size_t off = (size_t)(key0 + r) * p.kv_dim + (size_t)kvh * hd + c * 8;
            kv = ldg_stream(p.k_cache + off);
            vv = ldg_stream(p.v_cache + off);
        }
        *reinterpret_cast<uint4*>(Ks + (size_t)r * kstride + c * 8) = kv;
        *reinterpret_cast<uint4*>(Vs + (size_t)r * hd + c * 8) = vv;
    }

    for (int g = 0; g < group; ++g) {
        const int head = kvh * group + g;
        __syncthreads();  // tiles staged / previous head's Ps and qs consumed
        for (int i = tid; i < M * hd; i += kAttnThreads) {
            const int m = i / hd, e = i - m * hd;
            qs[i] = __bfloat162float(p.q[(size_t)m * p.d_model + (size_t)head * hd + e]);
        }
        __syncthreads();

        // ---- scores: thread t owns key key0 + t
        float sc[M];
#pragma unroll
        for (int m = 0; m < M; ++m) sc[m] = 0.f;
        for (int c = 0; c < vec_per_row; ++c) {
            const uint4 kv = *reinterpret_cast<const uint4*>(Ks + (size_t)tid * kstride + c * 8);
            const float kf[8] = {bf_lo(kv.x), bf_hi(kv.x), bf_lo(kv.y), bf_hi(kv.y),
                                 bf_lo(kv.z), bf_hi(kv.z), bf_lo(kv.w), bf_hi(kv.w)};
#pragma unroll
            for (int m = 0; m < M; ++m) {
                const float4 q0 = *reinterpret_cast<const float4*>(qs + m * hd + c * 8);
                const float4 q1 = *reinterpret_cast<const float4*>(qs + m * hd + c * 8 + 4);
                float a = sc[m];
                a = fmaf(q0.x, kf[0], a);
                a = fmaf(q0.y, kf[1], a);
                a = fmaf(q0.z, kf[2], a);
                a = fmaf(q0.w, kf[3], a);
                a = fmaf(q1.x, kf[4], a);
                a = fmaf(q1.y, kf[5], a);
                a = fmaf(q1.z, kf[6], a);
                a = fmaf(q1.w, kf[7], a);
                sc[m] = a;
            }
        }
        // ---- chunk-local softmax statistics; the row at position pos0+m sees keys <= pos0+m
        const int key = key0 + tid;
        float cmax[M];
#pragma unroll
        for (int m = 0; m < M; ++m) {
            const bool ok = key <= p.pos0 + m;
            sc[m] = ok ? sc[m] * p.scale : -INFINITY;
            const float v = warp_max(sc[m]);
            if (lane == 0) red[warp * kMaxRows + m] = v;
        }
        __syncthreads();
#pragma unroll
        for (int m = 0; m < M; ++m)
            cmax[m] = fmaxf(fmaxf(red[0 * kMaxRows + m], red[1 * kMaxRows + m]),
                            fmaxf(red[2 * kMaxRows + m], red[3 * kMaxRows + m]));
        __syncthreads();
        float pe[M];
#pragma unroll
        for (int m = 0; m < M; ++m) {
            pe[m] = (sc[m] == -INFINITY) ? 0.f : expf(sc[m] - cmax[m]);
            Ps[m * kAttnChunk + tid] = pe[m];
            const float v = warp_sum(pe[m]);
            if (lane == 0) red[warp * kMaxRows + m] = v;
        }
        __syncthreads();
        if (tid < M) {
            const float l = ((red[0 * kMaxRows + tid] + red[1 * kMaxRows + tid]) + red[2 * kMaxRows + tid]) +
                            red[3 * kMaxRows + tid];
            p.part_ml[(((size_t)head * p.chunk_stride + chunk) * kMaxRows + tid) * 2 + 1] = l;
        }
        if (tid == 0) {
#pragma unroll
            for (int m = 0; m < M; ++m)
                p.part_ml[(((size_t)head * p.chunk_stride + chunk) * kMaxRows + m) * 2 + 0] = cmax[m];
        }

        // ---- P V: thread e owns output dimension e
        for (int e = tid; e < hd; e += kAttnThreads) {
            float acc[M];
#pragma unroll
            for (int m = 0; m < M; ++m) acc[m] = 0.f;
            for (int j = 0; j < n_valid; ++j) {
                const float v = __bfloat162float(Vs[(size_t)j * hd + e]);
#pragma unroll
                for (int m = 0; m < M; ++m) acc[m] = fmaf(Ps[m * kAttnChunk + j], v, acc[m]);
            }
#pragma unroll
            for (int m = 0; m < M; ++m)
                p.part_acc[(((size_t)head * p.chunk_stride + chunk) * kMaxRows + m) * hd + e] = acc[m];
        }
    }

    // ---- the last CTA of this kv head merges the chunk partials in chunk order
    __threadfence();
    __syncthreads();
    if (tid == 0) {
        const unsigned t = atomicAdd(p.counters + kvh, 1u);
        *flag = (t == (unsigned)p.n_chunks - 1) ? 1 : 0;
    }
    __syncthreads();
    if (*flag == 0) return;
    __threadfence();
    if (tid == 0) p.counters[kvh] = 0u;
    for (int g = 0; g < group; ++g) {
        const int head = kvh * group + g;
        for (int e = tid; e < hd; e += kAttnThreads) {
#pragma unroll
            for (int m = 0; m < M; ++m) {
                const int nc = (p.pos0 + m) / kAttnChunk + 1;  // chunks that hold keys visible to this row
                float mx = -INFINITY, l = 0.f, acc = 0.f;
                for (int c = 0; c < nc; ++c) {
                    const size_t base = ((size_t)head * p.chunk_stride + c) * kMaxRows + m;
                    const float cm = __ldcg(p.part_ml + base * 2 + 0);
                    const float cl = __ldcg(p.part_ml + base * 2 + 1);
                    const float pa = __ldcg(p.part_acc + base * hd + e);
                    const float mn = fmaxf(mx, cm);
                    const float s_old = expf(mx - mn), s_new = expf(cm - mn);
                    acc = acc * s_old + pa * s_new;
                    l = l * s_old + cl * s_new;
                    mx = mn;
                }
                p.a_out[(size_t)m * p.d_model + (size_t)head * hd + e] = __float2bfloat16_rn(acc / l);
            }
        }
    }
}

}  // namespace asd
