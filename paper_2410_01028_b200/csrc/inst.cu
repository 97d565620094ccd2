// Instantiations of the row-count-templated kernels; compiled once per ASD_M in 1..9 (both kernels) and 16 (pass
// kernel only: the row count of a prefill pass).
#include "gemv.cuh"
#include "pass.cuh"

#ifndef ASD_M
#error "compile with -DASD_M=<rows>"
#endif

namespace asd {

#define ASD_CAT2(a, b) a##b
#define ASD_CAT(a, b) ASD_CAT2(a, b)

#if ASD_M <= 9
template <int EPI, bool NORM>
static cudaError_t launch_one(const GemvParams& p, int grid, size_t smem, cudaStream_t s) {
    gemv_kernel<ASD_M, EPI, NORM><<<grid, kGemvThreads, smem, s>>>(p);
    return cudaGetLastError();
}

cudaError_t ASD_CAT(launch_gemv_m, ASD_M)(int epi, bool norm, const GemvParams& p, int grid, size_t smem, cudaStream_t s) {
    switch (epi) {
        case kEpiPlain: return norm ? launch_one<kEpiPlain, true>(p, grid, smem, s) : launch_one<kEpiPlain, false>(p, grid, smem, s);
        case kEpiSwiglu: return norm ? launch_one<kEpiSwiglu, true>(p, grid, smem, s) : launch_one<kEpiSwiglu, false>(p, grid, smem, s);
        case kEpiResidual: return norm ? launch_one<kEpiResidual, true>(p, grid, smem, s) : launch_one<kEpiResidual, false>(p, grid, smem, s);
    }
    return cudaErrorInvalidValue;
}
#endif

// the one-row pass exists in two variants: activations handed over through tagged words (p.use_ll) or through
// plain buffers behind the grid barrier
cudaError_t ASD_CAT(launch_pass_m, ASD_M)(const PassParams& p, int grid, size_t smem, cudaStream_t s) {
    void* args[] = {const_cast<PassParams*>(&p)};
    const void* fn = reinterpret_cast<const void*>(&pass_kernel<ASD_M, false>);
#if ASD_M == 1
    if (p.use_ll) fn = reinterpret_cast<const void*>(&pass_kernel<ASD_M, true>);
#else
    if (p.use_ll) return cudaErrorInvalidValue;
#endif
    return cudaLaunchCooperativeKernel(fn, dim3(grid), dim3(kPassThreads), args, smem, s);
}

// opt every instantiation in to large dynamic shared memory
cudaError_t ASD_CAT(configure_m, ASD_M)(int max_smem) {
    cudaError_t e;
#define ASD_SET(k)                                                                              \
    e = cudaFuncSetAttribute(k, cudaFuncAttributeMaxDynamicSharedMemorySize, max_smem);         \
    if (e != cudaSuccess) return e;
#if ASD_M <= 9
    ASD_SET((gemv_kernel<ASD_M, kEpiPlain, true>))
    ASD_SET((gemv_kernel<ASD_M, kEpiPlain, false>))
    ASD_SET((gemv_kernel<ASD_M, kEpiSwiglu, true>))
    ASD_SET((gemv_kernel<ASD_M, kEpiSwiglu, false>))
    ASD_SET((gemv_kernel<ASD_M, kEpiResidual, true>))
    ASD_SET((gemv_kernel<ASD_M, kEpiResidual, false>))
#endif
    ASD_SET((pass_kernel<ASD_M, false>))
#if ASD_M == 1
    ASD_SET((pass_kernel<ASD_M, true>))
#endif
#undef ASD_SET
    return cudaSuccess;
}

}  // namespace asd
