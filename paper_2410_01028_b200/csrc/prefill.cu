// Kernels of the dense prompt path (see prefill.h).
#include "prefill.h"

#include "common.cuh"
#include "ring.cuh"

namespace asd {

constexpr int kErrGemmWait = 4;  // a pipeline barrier of the GEMM never completed

// ============================================================================================ tcgen05 helpers
__device__ __forceinline__ void tmem_alloc(uint32_t* smem_slot, uint32_t n_cols) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(smem_slot)), "r"(n_cols) : "memory");
}
__device__ __forceinline__ void tmem_relinquish() { asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory"); }
__device__ __forceinline__ void tmem_dealloc(uint32_t taddr, uint32_t n_cols) {
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(taddr), "r"(n_cols) : "memory");
}
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
// all tcgen05.mma issued so far by this thread arrive on the barrier when they have finished
__device__ __forceinline__ void tc_commit(uint64_t* bar) {
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(smem_u32(bar)) : "memory");
}
// D (tensor memory, 128 lanes x N columns fp32) (+)= A (smem, 128 x 16 bf16, K-major) * B (smem, N x 16 bf16, K-major)^T
__device__ __forceinline__ void tc_mma_bf16(uint32_t tmem_d, uint64_t a_desc, uint64_t b_desc, uint32_t idesc, uint32_t accumulate) {
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.u32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
        ::"r"(tmem_d), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate)
        : "memory");
}
// 32 consecutive fp32 columns of this thread's lane of tensor memory
__device__ __forceinline__ void tmem_ld32(uint32_t taddr, float (&v)[32]) {
    uint32_t r[32];
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
        "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
        "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
        : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]), "=r"(r[9]),
          "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]), "=r"(r[16]), "=r"(r[17]), "=r"(r[18]),
          "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]), "=r"(r[24]), "=r"(r[25]), "=r"(r[26]), "=r"(r[27]),
          "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
        : "r"(taddr)
        : "memory");
    asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
#pragma unroll
    for (int i = 0; i < 32; ++i) v[i] = __uint_as_float(r[i]);
}

// Shared-memory matrix descriptor of a K-major bf16 tile whose rows are 128 bytes (64 elements) stored with the
// 128-byte swizzle, tile base 1024-byte aligned: groups of 8 rows are 1024 bytes apart (stride byte offset);
// the leading byte offset is not used by swizzled K-major layouts. Fields: start address >> 4 in bits 0-13,
// leading offset >> 4 in bits 16-29, stride offset >> 4 in bits 32-45, descriptor version 1 in bits 46-47,
// swizzle mode (2 = 128 bytes) in bits 61-63.
__device__ __forceinline__ uint64_t umma_desc_k128(uint32_t smem_addr) {
    uint64_t d = 0;
    d |= (uint64_t)((smem_addr & 0x3FFFFu) >> 4);
    d |= (uint64_t)1 << 16;
    d |= (uint64_t)(1024 >> 4) << 32;
    d |= (uint64_t)1 << 46;
    d |= (uint64_t)2 << 61;
    return d;
}
// Instruction descriptor of kind::f16: fp32 accumulator (bits 4-5 = 1), bf16 A and B (bits 7-9, 10-12 = 1), both
// K-major (bits 15, 16 = 0), N >> 3 in bits 17-22, M >> 4 in bits 24-28.
__host__ __device__ constexpr uint32_t umma_idesc_bf16(int m, int n) {
    return (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(n >> 3) << 17) | ((uint32_t)(m >> 4) << 24);
}

// ============================================================================================ GEMM epilogues
// One call per (row, 32 consecutive columns starting at col0) with the fp32 accumulators in v.
__device__ __forceinline__ void epi_f32(const GemmEpi& ep, int row, int col0, int N, const float (&v)[32], int half) {
    float* dst = ep.c + (size_t)half * ep.c_split_stride + (size_t)row * ep.ldc + col0;
    if (col0 + 32 <= N && (ep.ldc & 3) == 0) {
#pragma unroll
        for (int i = 0; i < 8; ++i) reinterpret_cast<float4*>(dst)[i] = make_float4(v[4 * i], v[4 * i + 1], v[4 * i + 2], v[4 * i + 3]);
    } else {
#pragma unroll
        for (int i = 0; i < 32; ++i)
            if (col0 + i < N) dst[i] = v[i];
    }
}

__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi) {
    const __nv_bfloat162 h = __floats2bfloat162_rn(lo, hi);
    return *reinterpret_cast<const uint32_t*>(&h);
}

__device__ __forceinline__ void epi_swiglu(const GemmEpi& ep, int row, int col0, int N, const float (&v)[32]) {
    __nv_bfloat16* dst = ep.t + (size_t)row * ep.ldt + (col0 >> 1);
    float t[16];
#pragma unroll
    for (int i = 0; i < 16; ++i) {
        const float g = v[2 * i], u = v[2 * i + 1];
        t[i] = g / (1.0f + expf(-g)) * u;
    }
    if (col0 + 32 <= N && (ep.ldt & 7) == 0) {
        uint4 o0, o1;
        o0.x = pack_bf16(t[0], t[1]), o0.y = pack_bf16(t[2], t[3]), o0.z = pack_bf16(t[4], t[5]), o0.w = pack_bf16(t[6], t[7]);
        o1.x = pack_bf16(t[8], t[9]), o1.y = pack_bf16(t[10], t[11]), o1.z = pack_bf16(t[12], t[13]), o1.w = pack_bf16(t[14], t[15]);
        reinterpret_cast<uint4*>(dst)[0] = o0;
        reinterpret_cast<uint4*>(dst)[1] = o1;
    } else {
#pragma unroll
        for (int i = 0; i < 16; ++i)
            if (col0 + 2 * i + 1 < N) dst[i] = __float2bfloat16_rn(t[i]);
    }
}

// head_dim is a multiple of 32 and the q, k and v column ranges start at multiples of head_dim, so the 32 columns
// belong to one head of one of q, k, v.
__device__ __forceinline__ void epi_qkv(const GemmEpi& ep, int row, int col0, int N, const float (&v)[32]) {
    if (col0 >= N) return;
    const int pos = ep.pos0 + row;
    const int hd = ep.head_dim, half = hd >> 1;
    if (col0 >= ep.d_model + ep.kv_dim) {  // values: natural order, no rotation
        __nv_bfloat16* dst = ep.v_cache + (size_t)pos * ep.kv_dim + (col0 - ep.d_model - ep.kv_dim);
        uint4 o[4];
        uint32_t* w = reinterpret_cast<uint32_t*>(o);
#pragma unroll
        for (int i = 0; i < 16; ++i) w[i] = pack_bf16(v[2 * i], v[2 * i + 1]);
#pragma unroll
        for (int i = 0; i < 4; ++i) reinterpret_cast<uint4*>(dst)[i] = o[i];
        return;
    }
    const bool is_q = col0 < ep.d_model;
    const int c = is_q ? col0 : col0 - ep.d_model;
    const int head = c / hd, j0 = (c - head * hd) >> 1;  // pairs j0 .. j0+15 of this head
    const float4* cs = reinterpret_cast<const float4*>(ep.rope_cos + (size_t)pos * half + j0);
    const float4* sn = reinterpret_cast<const float4*>(ep.rope_sin + (size_t)pos * half + j0);
    float lo[16], hi[16];
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        const float4 c4 = cs[i], s4 = sn[i];
        const float cc[4] = {c4.x, c4.y, c4.z, c4.w}, ss[4] = {s4.x, s4.y, s4.z, s4.w};
#pragma unroll
        for (int u = 0; u < 4; ++u) {
            const float va = v[2 * (4 * i + u)], vb = v[2 * (4 * i + u) + 1];
            lo[4 * i + u] = va * cc[u] - vb * ss[u];
            hi[4 * i + u] = vb * cc[u] + va * ss[u];
        }
    }
    __nv_bfloat16* base = is_q ? ep.q + (size_t)row * ep.d_model : ep.k_cache + (size_t)pos * ep.kv_dim;
    __nv_bfloat16* dlo = base + (size_t)head * hd + j0;
    __nv_bfloat16* dhi = dlo + half;
    uint4 o[2];
    uint32_t* w = reinterpret_cast<uint32_t*>(o);
#pragma unroll
    for (int i = 0; i < 8; ++i) w[i] = pack_bf16(lo[2 * i], lo[2 * i + 1]);
    reinterpret_cast<uint4*>(dlo)[0] = o[0];
    reinterpret_cast<uint4*>(dlo)[1] = o[1];
#pragma unroll
    for (int i = 0; i < 8; ++i) w[i] = pack_bf16(hi[2 * i], hi[2 * i + 1]);
    reinterpret_cast<uint4*>(dhi)[0] = o[0];
    reinterpret_cast<uint4*>(dhi)[1] = o[1];
}

// ============================================================================================ the GEMM
// Persistent CTAs (one per SM) walk the 128 x BN tiles of the product, row tiles fastest. Warp 0 (one lane) is the TMA
// producer, warp 1 (one lane) issues the MMAs and owns the tensor-memory allocation, warps 2-5 are the epilogue (warp
// w reads lanes 32 * (w % 4) .. + 31 of tensor memory, the quarter its position in the warp group gives it access
// to). The accumulator is double-buffered in tensor memory (2 x BN columns), so the epilogue of a tile runs while the
// MMAs of the next tile are already filling the other buffer. Barriers: full[s] (TMA bytes landed in stage s),
// empty[s] (the MMAs reading stage s have finished: tcgen05.commit), acc_full[b] (all MMAs of the tile in buffer b
// have finished), acc_empty[b] (the 128 epilogue threads have read buffer b). Ragged edges: TMA fills out-of-range
// rows and reduction elements with zeros; the epilogue skips rows >= M and columns >= N. Every wait is bounded; after
// a failed wait the roles fall through to the common exit, where the producer lets its copies in flight land and
// the tensor memory is freed.
constexpr int kGemmThreads = 192;
static int g_gemm_ctas = 148;  // persistent CTAs per launch: the SM count of the device (set by configure_prefill)

template <int BN>
struct GemmCfg {
    static constexpr int kStages = (BN == 256) ? 4 : 6;
    static constexpr uint32_t kABytes = kGemmBM * kGemmBK * 2;
    static constexpr uint32_t kBBytes = BN * kGemmBK * 2;
    static constexpr uint32_t kStageBytes = kABytes + kBBytes;
    static constexpr size_t kSmem = (size_t)kStages * kStageBytes + 1024 /* alignment */ + 256 /* barriers */;
};

template <int BN>
__global__ void __launch_bounds__(kGemmThreads, 1)
gemm_tn_kernel(const __grid_constant__ CUtensorMap tm_a, const __grid_constant__ CUtensorMap tm_w, int M, int N, int K, int m_tiles,
               int n_tiles_total, const GemmEpi ep) {
    using Cfg = GemmCfg<BN>;
    constexpr int kStages = Cfg::kStages;
    extern __shared__ unsigned char gemm_smem_raw[];
    unsigned char* base = gemm_smem_raw + ((1024u - (smem_u32(gemm_smem_raw) & 1023u)) & 1023u);
    uint64_t* full = reinterpret_cast<uint64_t*>(base + (size_t)kStages * Cfg::kStageBytes);
    uint64_t* empty = full + kStages;
    uint64_t* acc_full = empty + kStages;   // [2]
    uint64_t* acc_empty = acc_full + 2;     // [2]
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(acc_empty + 2);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int num_kb = (K + kGemmBK - 1) / kGemmBK;
    // Work item = (tile, half of the reduction dimension); without a split there is one half. Items of half 0 come
    // first, so CTAs that run together still share their weight tile.
    const int k_split = (ep.mode == kGemmF32 && ep.k_split == 2) ? 2 : 1;
    const int kb_per = (num_kb + k_split - 1) / k_split;
    const int n_items = n_tiles_total * k_split;
    volatile int* err = ep.err;

    if (threadIdx.x == 0) {
        for (int s = 0; s < kStages; ++s) {
            mbar_init(&full[s], 1);
            mbar_init(&empty[s], 1);
        }
        for (int b = 0; b < 2; ++b) {
            mbar_init(&acc_full[b], 1);
            mbar_init(&acc_empty[b], 128);
        }
        mbar_fence_init();
    }
    if (warp == 1) {
        tmem_alloc(tmem_slot, 2 * BN);
        tmem_relinquish();
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = *tmem_slot;

    if (warp == 0) {
        if (lane == 0) {
            int issued = 0;  // k-blocks requested so far, over all tiles of this CTA
            bool ok = true;
            for (int item = blockIdx.x; item < n_items && ok; item += gridDim.x) {
                // row tiles vary fastest: CTAs that run together share their weight tile (read once from HBM, then from L2)
                const int tile = item % n_tiles_total, half = item / n_tiles_total;
                const int m0 = (tile % m_tiles) * kGemmBM, n0 = (tile / m_tiles) * BN;
                for (int kb = half * kb_per; kb < min(num_kb, (half + 1) * kb_per); ++kb) {
                    const int s = issued % kStages;
                    if (issued >= kStages) ok = mbar_wait(&empty[s], (uint32_t)((issued / kStages - 1) & 1), err, kErrGemmWait, 0, issued, s, 1);
                    if (!ok) break;
                    unsigned char* a_dst = base + (size_t)s * Cfg::kStageBytes;
                    mbar_expect_tx(&full[s], Cfg::kStageBytes);
                    tma_load_2d(a_dst, &tm_a, kb * kGemmBK, m0, &full[s]);
                    tma_load_2d(a_dst + Cfg::kABytes, &tm_w, kb * kGemmBK, n0, &full[s]);
                    ++issued;
                }
            }
            if (!ok || *err != kErrNone) {
                // abandoned: let the copies still in flight land before the CTA gives its shared memory back
                for (int i = max(0, issued - kStages); i < issued; ++i) {
                    const long long t0 = clock64();
                    while (!mbar_try_wait(&full[i % kStages], (uint32_t)((i / kStages) & 1)) && clock64() - t0 < 20000000LL) {
                    }
                }
            }
        }
    } else if (warp == 1) {
        if (lane == 0) {
            constexpr uint32_t idesc = umma_idesc_bf16(kGemmBM, BN);
            int done = 0, local = 0;  // k-blocks consumed so far; tiles of this CTA started so far
            bool ok = true;
            for (int item = blockIdx.x; item < n_items && ok; item += gridDim.x, ++local) {
                const int buf = local & 1;
                const int kb0 = (item / n_tiles_total) * kb_per, kb1 = min(num_kb, kb0 + kb_per);
                // the epilogue must have read this buffer's previous tile (tile local - 2) before it is overwritten
                if (local >= 2) ok = mbar_wait(&acc_empty[buf], (uint32_t)((local / 2 - 1) & 1), err, kErrGemmWait, 3, local, buf, 4);
                if (!ok) break;
                tc_fence_after();
                const uint32_t tmem_d = tmem + (uint32_t)(buf * BN);
                for (int kb = kb0; kb < kb1; ++kb) {
                    const int s = done % kStages;
                    ok = mbar_wait(&full[s], (uint32_t)((done / kStages) & 1), err, kErrGemmWait, 1, done, s, 2);
                    if (!ok) break;
                    tc_fence_after();
                    const uint32_t a_addr = smem_u32(base + (size_t)s * Cfg::kStageBytes);
                    const uint64_t a_desc = umma_desc_k128(a_addr), b_desc = umma_desc_k128(a_addr + Cfg::kABytes);
#pragma unroll
                    for (int k = 0; k < kGemmBK / 16; ++k)  // 16 elements = 32 bytes further along the swizzled row: +2 in the address field
                        tc_mma_bf16(tmem_d, a_desc + (uint64_t)(2 * k), b_desc + (uint64_t)(2 * k), idesc, ((kb - kb0) | k) != 0 ? 1u : 0u);
                    tc_commit(&empty[s]);  // the stage may be refilled once these MMAs have read it
                    ++done;
                }
                tc_commit(&acc_full[buf]);  // arrives when every MMA issued above has finished
            }
        }
    } else {
        const int quarter = warp & 3;
        bool ok = true;
        int local = 0;
        for (int item = blockIdx.x; item < n_items && ok; item += gridDim.x, ++local) {
            const int buf = local & 1;
            const int tile = item % n_tiles_total, half = item / n_tiles_total;
            const int m0 = (tile % m_tiles) * kGemmBM, n0 = (tile / m_tiles) * BN;
            const int row = m0 + quarter * 32 + lane;
            ok = mbar_wait(&acc_full[buf], (uint32_t)((local / 2) & 1), err, kErrGemmWait, 2, local, buf, 3) && *err == kErrNone;
            tc_fence_after();
            if (!ok) break;
            for (int cb = 0; cb < BN / 32; ++cb) {
                const int col0 = n0 + cb * 32;
                if (col0 >= N) break;  // uniform across the warp
                float v[32];
                tmem_ld32(tmem + ((uint32_t)(quarter * 32) << 16) + (uint32_t)(buf * BN + cb * 32), v);
                if (row < M) {
                    if (ep.mode == kGemmF32) epi_f32(ep, row, col0, N, v, half);
                    else if (ep.mode == kGemmSwiglu) epi_swiglu(ep, row, col0, N, v);
                    else epi_qkv(ep, row, col0, N, v);
                }
            }
            tc_fence_before();
            mbar_arrive(&acc_empty[buf]);  // this thread has read its lanes of the buffer
        }
    }
    tc_fence_before();
    __syncthreads();
    if (warp == 1) {
        tc_fence_after();
        tmem_dealloc(tmem, 2 * BN);
    }
}

template <int BN>
static cudaError_t launch_gemm_bn(const CUtensorMap& tm_a, const CUtensorMap& tm_w, int M, int N, int K, const GemmEpi& ep, cudaStream_t s) {
    const int m_tiles = (M + kGemmBM - 1) / kGemmBM, n_tiles = (N + BN - 1) / BN;
    const int total = m_tiles * n_tiles;
    const int items = total * ((ep.mode == kGemmF32 && ep.k_split == 2) ? 2 : 1);
    gemm_tn_kernel<BN><<<items < g_gemm_ctas ? items : g_gemm_ctas, kGemmThreads, GemmCfg<BN>::kSmem, s>>>(tm_a, tm_w, M, N, K, m_tiles, total, ep);
    return cudaGetLastError();
}

cudaError_t launch_gemm_tn(const CUtensorMap& tm_a, const CUtensorMap& tm_w, int M, int N, int K, int bn, const GemmEpi& ep,
                           cudaStream_t s) {
    if (M <= 0 || N <= 0 || K <= 0) return cudaErrorInvalidValue;
    if (bn == 256) return launch_gemm_bn<256>(tm_a, tm_w, M, N, K, ep, s);
    if (bn == 128) return launch_gemm_bn<128>(tm_a, tm_w, M, N, K, ep, s);
    return cudaErrorInvalidValue;
}

// ============================================================================================ row kernels
constexpr int kRowThreads = 256;

// block-wide sums of up to three values; result valid in every thread
template <int NV>
__device__ __forceinline__ void block_sum(float (&v)[NV], float* red /* [NV][8] */) {
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
#pragma unroll
    for (int j = 0; j < NV; ++j) {
        v[j] = warp_sum(v[j]);
        if (lane == 0) red[j * 8 + warp] = v[j];
    }
    __syncthreads();
#pragma unroll
    for (int j = 0; j < NV; ++j) {
        float t = 0.f;
#pragma unroll
        for (int w = 0; w < kRowThreads / 32; ++w) t += red[j * 8 + w];
        v[j] = t;
    }
    __syncthreads();
}

__global__ void __launch_bounds__(kRowThreads) embed_norm_kernel(const int* tokens, int d, int vocab, const __nv_bfloat16* embed,
                                                                const __nv_bfloat16* gain, float eps, float* x, __nv_bfloat16* xn) {
    __shared__ float red[8];
    const int r = blockIdx.x;
    int t = tokens[r];
    t = min(max(t, 0), vocab - 1);
    const __nv_bfloat16* e = embed + (size_t)t * d;
    float s[1] = {0.f};
    for (int i = threadIdx.x; i < d; i += kRowThreads) {
        const float v = __bfloat162float(e[i]);
        x[(size_t)r * d + i] = v;
        s[0] = fmaf(v, v, s[0]);
    }
    block_sum<1>(s, red);
    const float inv = 1.0f / sqrtf(s[0] / (float)d + eps);
    for (int i = threadIdx.x; i < d; i += kRowThreads)
        xn[(size_t)r * d + i] = __float2bfloat16_rn(__bfloat162float(e[i]) * inv * __bfloat162float(gain[i]));
}

// The residual add with the cosine similarity of the hidden state before and after the sublayer (Section 3.2), and
// the RMSNorm that feeds the next sublayer (its statistic is the |y|^2 just computed).
__global__ void __launch_bounds__(kRowThreads) resid_norm_kernel(int d, float* x, const float* c, const float* c2, const __nv_bfloat16* gain, float eps,
                                                                __nv_bfloat16* xn, float* cos_out) {
    __shared__ float red[24];
    const int r = blockIdx.x;
    float* xr = x + (size_t)r * d;
    const float* cr = c + (size_t)r * d;
    const float* cr2 = c2 ? c2 + (size_t)r * d : nullptr;  // second half of a product whose reduction dimension was cut in two
    float s[3] = {0.f, 0.f, 0.f};
    for (int i = threadIdx.x; i < d; i += kRowThreads) {
        const float xv = xr[i];
        const float y = xv + (cr2 ? cr[i] + cr2[i] : cr[i]);
        xr[i] = y;
        s[0] = fmaf(xv, y, s[0]);
        s[1] = fmaf(xv, xv, s[1]);
        s[2] = fmaf(y, y, s[2]);
    }
    block_sum<3>(s, red);
    if (threadIdx.x == 0) {
        const double den = fmax(sqrt((double)s[1]) * sqrt((double)s[2]), 1e-30);
        cos_out[r] = (float)((double)s[0] / den);
    }
    if (gain) {
        const float inv = 1.0f / sqrtf(s[2] / (float)d + eps);
        for (int i = threadIdx.x; i < d; i += kRowThreads)
            xn[(size_t)r * d + i] = __float2bfloat16_rn(xr[i] * inv * __bfloat162float(gain[i]));
    }
}

// The same with the row held in registers (rows of at most kRowThreads * 4 * NV elements, a multiple of 4): x and the
// sublayer output are read once, 16 bytes per load, and the sums, the new hidden state and the normalised row all
// come from those registers.
template <int NV>
__global__ void __launch_bounds__(kRowThreads) resid_norm_vec_kernel(int d, float* x, const float* c, const float* c2, const __nv_bfloat16* gain, float eps,
                                                                    __nv_bfloat16* xn, float* cos_out) {
    __shared__ float red[24];
    const int r = blockIdx.x, nvec = d >> 2;
    float4* xr = reinterpret_cast<float4*>(x + (size_t)r * d);
    const float4* cr = reinterpret_cast<const float4*>(c + (size_t)r * d);
    float4 y[NV], cv[NV];
#pragma unroll
    for (int v = 0; v < NV; ++v) {
        const int i = threadIdx.x + v * kRowThreads;
        y[v] = cv[v] = make_float4(0.f, 0.f, 0.f, 0.f);
        if (i < nvec) y[v] = xr[i], cv[v] = cr[i];
    }
    if (c2) {  // the product came in two halves of its reduction dimension: half 0 + half 1
        const float4* cr2 = reinterpret_cast<const float4*>(c2 + (size_t)r * d);
#pragma unroll
        for (int v = 0; v < NV; ++v) {
            const int i = threadIdx.x + v * kRowThreads;
            if (i < nvec) {
                const float4 o = cr2[i];
                cv[v].x += o.x, cv[v].y += o.y, cv[v].z += o.z, cv[v].w += o.w;
            }
        }
    }
    float s[3] = {0.f, 0.f, 0.f};
#pragma unroll
    for (int v = 0; v < NV; ++v) {
        const int i = threadIdx.x + v * kRowThreads;
        if (i < nvec) {
            const float4 xv = y[v];
            float4 o;
            o.x = xv.x + cv[v].x, o.y = xv.y + cv[v].y, o.z = xv.z + cv[v].z, o.w = xv.w + cv[v].w;
            s[0] = fmaf(xv.x, o.x, s[0]), s[1] = fmaf(xv.x, xv.x, s[1]), s[2] = fmaf(o.x, o.x, s[2]);
            s[0] = fmaf(xv.y, o.y, s[0]), s[1] = fmaf(xv.y, xv.y, s[1]), s[2] = fmaf(o.y, o.y, s[2]);
            s[0] = fmaf(xv.z, o.z, s[0]), s[1] = fmaf(xv.z, xv.z, s[1]), s[2] = fmaf(o.z, o.z, s[2]);
            s[0] = fmaf(xv.w, o.w, s[0]), s[1] = fmaf(xv.w, xv.w, s[1]), s[2] = fmaf(o.w, o.w, s[2]);
            xr[i] = o;
            y[v] = o;
        }
    }
    block_sum<3>(s, red);
    if (threadIdx.x == 0) {
        const double den = fmax(sqrt((double)s[1]) * sqrt((double)s[2]), 1e-30);
        cos_out[r] = (float)((double)s[0] / den);
    }
    if (gain) {
        const float inv = 1.0f / sqrtf(s[2] / (float)d + eps);
#pragma unroll
        for (int v = 0; v < NV; ++v) {
            const int i = threadIdx.x + v * kRowThreads;
            if (i < nvec) {
                const uint2 g = *reinterpret_cast<const uint2*>(gain + (size_t)i * 4);
                const __nv_bfloat162 lo = __floats2bfloat162_rn(y[v].x * inv * bf_lo(g.x), y[v].y * inv * bf_hi(g.x));
                const __nv_bfloat162 hi = __floats2bfloat162_rn(y[v].z * inv * bf_lo(g.y), y[v].w * inv * bf_hi(g.y));
                uint2 o;
                o.x = *reinterpret_cast<const uint32_t*>(&lo);
                o.y = *reinterpret_cast<const uint32_t*>(&hi);
                *reinterpret_cast<uint2*>(xn + (size_t)r * d + (size_t)i * 4) = o;
            }
        }
    }
}

__global__ void __launch_bounds__(32) sumcos_kernel(const float* cos_rows, int stride, int n_rows, double* sumcos) {
    const float* c = cos_rows + (size_t)blockIdx.x * stride;
    double acc = 0.0;
    for (int r = threadIdx.x; r < n_rows; r += 32) acc += (double)c[r];
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, o);
    if (threadIdx.x == 0) sumcos[blockIdx.x] += acc;
}

cudaError_t launch_embed_norm(const int* tokens, int n_rows, int d, int vocab, const __nv_bfloat16* embed, const __nv_bfloat16* gain,
                              float eps, float* x, __nv_bfloat16* xn, cudaStream_t s) {
    embed_norm_kernel<<<n_rows, kRowThreads, 0, s>>>(tokens, d, vocab, embed, gain, eps, x, xn);
    return cudaGetLastError();
}
cudaError_t launch_resid_norm(int n_rows, int d, float* x, const float* c, const float* c2, const __nv_bfloat16* gain, float eps, __nv_bfloat16* xn,
                              float* cos_out, cudaStream_t s) {
    const int nv = (d + kRowThreads * 4 - 1) / (kRowThreads * 4);
    if (d % 4 != 0 || nv > 8) resid_norm_kernel<<<n_rows, kRowThreads, 0, s>>>(d, x, c, c2, gain, eps, xn, cos_out);
    else if (nv <= 1) resid_norm_vec_kernel<1><<<n_rows, kRowThreads, 0, s>>>(d, x, c, c2, gain, eps, xn, cos_out);
    else if (nv <= 2) resid_norm_vec_kernel<2><<<n_rows, kRowThreads, 0, s>>>(d, x, c, c2, gain, eps, xn, cos_out);
    else if (nv <= 4) resid_norm_vec_kernel<4><<<n_rows, kRowThreads, 0, s>>>(d, x, c, c2, gain, eps, xn, cos_out);
    else if (nv <= 5) resid_norm_vec_kernel<5><<<n_rows, kRowThreads, 0, s>>>(d, x, c, c2, gain, eps, xn, cos_out);
    else resid_norm_vec_kernel<8><<<n_rows, kRowThreads, 0, s>>>(d, x, c, c2, gain, eps, xn, cos_out);
    return cudaGetLastError();
}
cudaError_t launch_sumcos(const float* cos_rows, int stride, int n_rows, int n_sub, double* sumcos, cudaStream_t s) {
    sumcos_kernel<<<n_sub, 32, 0, s>>>(cos_rows, stride, n_rows, sumcos);
    return cudaGetLastError();
}

// ============================================================================================ causal attention over the prompt
// One CTA = 64 query rows of one head (4 warps x 16 rows); keys and values stream through shared memory in tiles of
// 64 keys (double-buffered cp.async). Scores are bf16 x bf16 products accumulated in fp32 (mma.sync m16n8k16), the
// softmax is kept on line in fp32 (running maximum and sum per row), and the probabilities enter the P V product as
// the sum of three bf16 numbers (p = hi + mid + lo, three MMAs), which represents every fp32 probability exactly:
// with fewer terms the 2^-17 error of P flips bf16 roundings of the attention output in about every second row.
constexpr int kFaRows = 64, kFaKeys = 64, kFaThreads = 128;

__device__ __forceinline__ void cp_async16(void* smem_dst, const void* gsrc) {
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(smem_u32(smem_dst)), "l"(gsrc) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int N>
__device__ __forceinline__ void cp_async_wait() {
    asm volatile("cp.async.wait_group %0;" ::"n"(N) : "memory");
}
__device__ __forceinline__ void ldsm_x4(uint32_t (&r)[4], const void* smem_src) {
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3])
                 : "r"(smem_u32(smem_src)));
}
__device__ __forceinline__ void ldsm_x4_trans(uint32_t (&r)[4], const void* smem_src) {
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0,%1,%2,%3}, [%4];"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3])
                 : "r"(smem_u32(smem_src)));
}
__device__ __forceinline__ void mma16816(float (&c)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1) {
    asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
                 : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
                 : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}

template <int HD>
__global__ void __launch_bounds__(kFaThreads, 3)
flash_prefill_kernel(const __nv_bfloat16* __restrict__ q, const __nv_bfloat16* __restrict__ kc, const __nv_bfloat16* __restrict__ vc,
                     __nv_bfloat16* __restrict__ out, int n_rows, int pos0, int d_model, int kv_dim, int group, int max_seq, float scale) {
    constexpr int LD = HD + 8;  // padded row: rows stay 16-byte aligned and ldmatrix reads are free of bank conflicts
    constexpr int VPR = HD / 8;  // 16-byte vectors per row
    extern __shared__ __align__(16) unsigned char fa_smem[];
    __nv_bfloat16* Ks = reinterpret_cast<__nv_bfloat16*>(fa_smem);  // [2][64][LD]
    __nv_bfloat16* Vs = Ks + 2 * kFaKeys * LD;                      // [2][64][LD]
    __nv_bfloat16* Qs = Vs + kFaKeys * LD;  // [64][LD]: the queries are staged in the second V buffer, which is first filled after they are in registers

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31, g = lane >> 2, q4 = lane & 3;
    const int qt = gridDim.x - 1 - blockIdx.x;  // the tiles with the most keys start first
    const int head = blockIdx.y, kvh = head / group;
    const int r0 = qt * kFaRows;
    const int last_row = min(r0 + kFaRows - 1, n_rows - 1);
    const int n_kt = (pos0 + last_row) / kFaKeys + 1;

    auto load_tile = [&](int kt, int buf) {
        for (int idx = tid; idx < kFaKeys * VPR; idx += kFaThreads) {
            const int row = idx / VPR, c = idx - row * VPR;
            const int key = kt * kFaKeys + row;
            __nv_bfloat16* kd = Ks + (size_t)(buf * kFaKeys + row) * LD + c * 8;
            __nv_bfloat16* vd = Vs + (size_t)(buf * kFaKeys + row) * LD + c * 8;
            if (key < max_seq) {
                const size_t off = (size_t)key * kv_dim + (size_t)kvh * HD + c * 8;
                cp_async16(kd, kc + off);
                cp_async16(vd, vc + off);
            } else {
                *reinterpret_cast<uint4*>(kd) = make_uint4(0u, 0u, 0u, 0u);
                *reinterpret_cast<uint4*>(vd) = make_uint4(0u, 0u, 0u, 0u);
            }
        }
        cp_async_commit();
    };
    load_tile(0, 0);
    for (int idx = tid; idx < kFaRows * VPR; idx += kFaThreads) {
        const int row = idx / VPR, c = idx - row * VPR;
        const int r = min(r0 + row, n_rows - 1);  // rows past the prompt repeat the last row and are not stored
        *reinterpret_cast<uint4*>(Qs + (size_t)row * LD + c * 8) =
            *reinterpret_cast<const uint4*>(q + (size_t)r * d_model + (size_t)head * HD + c * 8);
    }
    __syncthreads();
    uint32_t qf[HD / 16][4];
#pragma unroll
    for (int kk = 0; kk < HD / 16; ++kk) ldsm_x4(qf[kk], Qs + (size_t)(warp * 16 + (lane & 15)) * LD + kk * 16 + (lane >> 4) * 8);
    __syncthreads();  // every warp has its queries: the buffer may now receive values

    const int pos_a = pos0 + min(r0 + warp * 16 + g, n_rows - 1);
    const int pos_b = pos0 + min(r0 + warp * 16 + g + 8, n_rows - 1);
    float o[HD / 8][4];
#pragma unroll
    for (int i = 0; i < HD / 8; ++i) o[i][0] = o[i][1] = o[i][2] = o[i][3] = 0.f;
    float m_run[2] = {-INFINITY, -INFINITY}, l_run[2] = {0.f, 0.f};

    for (int kt = 0; kt < n_kt; ++kt) {
        const int buf = kt & 1;
        if (kt + 1 < n_kt) {
            load_tile(kt + 1, buf ^ 1);
            cp_async_wait<1>();
        } else {
            cp_async_wait<0>();
        }
        __syncthreads();
        const __nv_bfloat16* Kb = Ks + (size_t)buf * kFaKeys * LD;
        const __nv_bfloat16* Vb = Vs + (size_t)buf * kFaKeys * LD;

        // ---- scores of 16 rows x 64 keys
        float sc[8][4];
#pragma unroll
        for (int nt = 0; nt < 8; ++nt) sc[nt][0] = sc[nt][1] = sc[nt][2] = sc[nt][3] = 0.f;
#pragma unroll
        for (int k2 = 0; k2 < HD / 32; ++k2) {  // 32 dimensions at a time over all 8 key blocks: consecutive MMAs are independent
            uint32_t b[8][4];
#pragma unroll
            for (int nt = 0; nt < 8; ++nt) ldsm_x4(b[nt], Kb + (size_t)(nt * 8 + (lane & 7)) * LD + k2 * 32 + (lane >> 3) * 8);
#pragma unroll
            for (int nt = 0; nt < 8; ++nt) mma16816(sc[nt], qf[2 * k2], b[nt][0], b[nt][1]);
#pragma unroll
            for (int nt = 0; nt < 8; ++nt) mma16816(sc[nt], qf[2 * k2 + 1], b[nt][2], b[nt][3]);
        }
        // ---- scale, causal mask (the row at position p sees keys <= p), running maximum
        const int key0 = kt * kFaKeys + 2 * q4;
        float mx[2] = {-INFINITY, -INFINITY};
#pragma unroll
        for (int nt = 0; nt < 8; ++nt)
#pragma unroll
            for (int e = 0; e < 4; ++e) {
                const int key = key0 + nt * 8 + (e & 1);
                const int pos = (e < 2) ? pos_a : pos_b;
                const float s = (key <= pos) ? sc[nt][e] * scale : -INFINITY;
                sc[nt][e] = s;
                mx[e >> 1] = fmaxf(mx[e >> 1], s);
            }
        float alpha[2];
#pragma unroll
        for (int h = 0; h < 2; ++h) {
            mx[h] = fmaxf(mx[h], __shfl_xor_sync(0xffffffffu, mx[h], 1));
            mx[h] = fmaxf(mx[h], __shfl_xor_sync(0xffffffffu, mx[h], 2));
            const float m_new = fmaxf(m_run[h], mx[h]);  // finite from the first tile on: key 0 is visible to every row
            alpha[h] = expf(m_run[h] - m_new);
            m_run[h] = m_new;
            l_run[h] *= alpha[h];
        }
#pragma unroll
        for (int nt = 0; nt < 8; ++nt)
#pragma unroll
            for (int e = 0; e < 4; ++e) {
                const float p = expf(sc[nt][e] - m_run[e >> 1]);
                sc[nt][e] = p;
                l_run[e >> 1] += p;  // this lane's share of the row sum; the four lanes of a row are added at the end
            }
#pragma unroll
        for (int i = 0; i < HD / 8; ++i) {
            o[i][0] *= alpha[0], o[i][1] *= alpha[0];
            o[i][2] *= alpha[1], o[i][3] *= alpha[1];
        }
        // ---- O += P V, P = hi + mid + lo in bf16
#pragma unroll
        for (int kk = 0; kk < kFaKeys / 16; ++kk) {
            uint32_t a_hi[4], a_mid[4], a_lo[4];
#pragma unroll
            for (int u = 0; u < 4; ++u) {
                const int nt = 2 * kk + (u >> 1), e = (u & 1) * 2;
                const float p0 = sc[nt][e], p1 = sc[nt][e + 1];
                const __nv_bfloat162 hi = __floats2bfloat162_rn(p0, p1);
                const float r0 = p0 - __low2float(hi), r1 = p1 - __high2float(hi);  // exact
                const __nv_bfloat162 mid = __floats2bfloat162_rn(r0, r1);
                const __nv_bfloat162 lo = __floats2bfloat162_rn(r0 - __low2float(mid), r1 - __high2float(mid));
                a_hi[u] = *reinterpret_cast<const uint32_t*>(&hi);
                a_mid[u] = *reinterpret_cast<const uint32_t*>(&mid);
                a_lo[u] = *reinterpret_cast<const uint32_t*>(&lo);
            }
            // all value fragments of the 16 keys first, then one term of the probabilities after the other (smallest first)
            // over all output blocks: consecutive MMAs never depend on each other
            uint32_t b[HD / 16][4];
#pragma unroll
            for (int n2 = 0; n2 < HD / 16; ++n2)
                ldsm_x4_trans(b[n2], Vb + (size_t)(kk * 16 + (lane & 7) + ((lane >> 3) & 1) * 8) * LD + n2 * 16 + (lane >> 4) * 8);
#pragma unroll
            for (int n2 = 0; n2 < HD / 16; ++n2) {
                mma16816(o[2 * n2], a_lo, b[n2][0], b[n2][1]);
                mma16816(o[2 * n2 + 1], a_lo, b[n2][2], b[n2][3]);
            }
#pragma unroll
            for (int n2 = 0; n2 < HD / 16; ++n2) {
                mma16816(o[2 * n2], a_mid, b[n2][0], b[n2][1]);
                mma16816(o[2 * n2 + 1], a_mid, b[n2][2], b[n2][3]);
            }
#pragma unroll
            for (int n2 = 0; n2 < HD / 16; ++n2) {
                mma16816(o[2 * n2], a_hi, b[n2][0], b[n2][1]);
                mma16816(o[2 * n2 + 1], a_hi, b[n2][2], b[n2][3]);
            }
        }
        __syncthreads();  // this buffer is refilled two iterations from now
    }

#pragma unroll
    for (int h = 0; h < 2; ++h) {
        l_run[h] += __shfl_xor_sync(0xffffffffu, l_run[h], 1);
        l_run[h] += __shfl_xor_sync(0xffffffffu, l_run[h], 2);
    }
    const int ra = r0 + warp * 16 + g, rb = ra + 8;
    const float inv_a = 1.0f / l_run[0], inv_b = 1.0f / l_run[1];
#pragma unroll
    for (int i = 0; i < HD / 8; ++i) {
        const size_t col = (size_t)head * HD + i * 8 + 2 * q4;
        if (ra < n_rows) *reinterpret_cast<uint32_t*>(out + (size_t)ra * d_model + col) = pack_bf16(o[i][0] * inv_a, o[i][1] * inv_a);
        if (rb < n_rows) *reinterpret_cast<uint32_t*>(out + (size_t)rb * d_model + col) = pack_bf16(o[i][2] * inv_b, o[i][3] * inv_b);
    }
}

template <int HD>
static constexpr size_t fa_smem_bytes() { return (size_t)4 * kFaKeys * (HD + 8) * 2; }

cudaError_t launch_flash_prefill(const __nv_bfloat16* q, const __nv_bfloat16* k_cache, const __nv_bfloat16* v_cache, __nv_bfloat16* out,
                                 int n_rows, int pos0, int d_model, int kv_dim, int head_dim, int n_heads, int n_kv_heads, int max_seq,
                                 float scale, cudaStream_t s) {
    if (n_rows <= 0) return cudaErrorInvalidValue;
    const dim3 grid((n_rows + kFaRows - 1) / kFaRows, n_heads);
    const int group = n_heads / n_kv_heads;
    if (head_dim == 128)
        flash_prefill_kernel<128><<<grid, kFaThreads, fa_smem_bytes<128>(), s>>>(q, k_cache, v_cache, out, n_rows, pos0, d_model, kv_dim, group, max_seq, scale);
    else if (head_dim == 64)
        flash_prefill_kernel<64><<<grid, kFaThreads, fa_smem_bytes<64>(), s>>>(q, k_cache, v_cache, out, n_rows, pos0, d_model, kv_dim, group, max_seq, scale);
    else
        return cudaErrorInvalidValue;
    return cudaGetLastError();
}

cudaError_t configure_prefill(int max_smem) {
    cudaError_t e;
    (void)max_smem;
    int dev = 0, sms = 0;
    if ((e = cudaGetDevice(&dev)) != cudaSuccess) return e;
    if ((e = cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev)) != cudaSuccess) return e;
    if (sms > 0) g_gemm_ctas = sms;
    if ((e = cudaFuncSetAttribute(gemm_tn_kernel<256>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)GemmCfg<256>::kSmem)) != cudaSuccess) return e;
    if ((e = cudaFuncSetAttribute(gemm_tn_kernel<128>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)GemmCfg<128>::kSmem)) != cudaSuccess) return e;
    if ((e = cudaFuncSetAttribute(flash_prefill_kernel<128>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)fa_smem_bytes<128>())) != cudaSuccess) return e;
    if ((e = cudaFuncSetAttribute(flash_prefill_kernel<64>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)fa_smem_bytes<64>())) != cudaSuccess) return e;
    return cudaSuccess;
}

}  // namespace asd
