// Shared declarations of the CUDA library: kernel parameter blocks and small device helpers.
#pragma once
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

namespace asd {

constexpr int kMaxRows = 9;        // rows of the stand-alone fused GEMV: max draft length 8, plus the last accepted token
constexpr int kPassMaxRows = 16;   // rows of one pass of the persistent kernel (prefill feeds the prompt 16 rows at a time)
constexpr int kGemvThreads = 512;  // 16 warps per CTA, one CTA per SM
constexpr int kGemvWarps = kGemvThreads / 32;
constexpr int kSeg = 1024;         // elements of the reduction dimension per warp work item
constexpr int kAttnChunk = 128;    // keys per attention work item; chunks are aligned to absolute positions

enum Epilogue : int { kEpiPlain = 0, kEpiSwiglu = 1, kEpiResidual = 2 };

// Parameter block of the fused RMSNorm -> GEMV -> epilogue kernel.
struct GemvParams {
    const __nv_bfloat16* W;  // [n_rows, n_in]
    int n_rows, n_in;
    const void* x;              // gain ? float [M, n_in] : bf16 [M, n_in]
    const __nv_bfloat16* gain;  // [n_in] or null
    float eps;
    int x_in_smem;  // stage the activations in shared memory (else read them through L1)
    // plain / swiglu / residual
    void* out;
    float* cos_out;   // residual: [M]
    double* sumcos;   // residual: running sum over prompt rows, or null
    float* partials;  // [gridDim.x][kMaxRows][4] cross-CTA partial results
    unsigned* counter;  // zero before launch; reset by the last CTA
};

struct PassParams;

// launchers, one translation unit per row count (inst.cu compiled with -DASD_M=1..9)
#define ASD_DECLARE_LAUNCHERS(M)                                                                                 \
    cudaError_t launch_gemv_m##M(int epi, bool norm, const GemvParams& p, int grid, size_t smem, cudaStream_t s); \
    cudaError_t launch_pass_m##M(const PassParams& p, int grid, size_t smem, cudaStream_t s);                    \
    cudaError_t configure_m##M(int max_smem);
ASD_DECLARE_LAUNCHERS(1)
ASD_DECLARE_LAUNCHERS(2)
ASD_DECLARE_LAUNCHERS(3)
ASD_DECLARE_LAUNCHERS(4)
ASD_DECLARE_LAUNCHERS(5)
ASD_DECLARE_LAUNCHERS(6)
ASD_DECLARE_LAUNCHERS(7)
ASD_DECLARE_LAUNCHERS(8)
ASD_DECLARE_LAUNCHERS(9)
cudaError_t launch_pass_m16(const PassParams& p, int grid, size_t smem, cudaStream_t s);
cudaError_t configure_m16(int max_smem);

size_t gemv_smem_bytes(int M, int n_rows, int n_in, int grid, bool x_in_smem);

// ---------------------------------------------------------------- device helpers
__device__ __forceinline__ float bf_lo(uint32_t u) { return __uint_as_float(u << 16); }
__device__ __forceinline__ float bf_hi(uint32_t u) { return __uint_as_float(u & 0xFFFF0000u); }

// streaming 16-byte load of weights: read-only path, do not keep in L1
__device__ __forceinline__ uint4 ldg_stream(const void* p) {
    uint4 v;
    asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];"
                 : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w)
                 : "l"(p));
    return v;
}

__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    return v;
}
__device__ __forceinline__ float warp_max(float v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, o));
    return v;
}

}  // namespace asd
