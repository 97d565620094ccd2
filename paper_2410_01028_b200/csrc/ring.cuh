// Shared-memory ring fed by the TMA engine, its mbarriers, and bounded waits.
//
// Every wait in this file gives up after a cycle budget, records why in a global error word and returns, and
// every later wait returns at once when that word is set: a lost signal turns into an error code on the
// host (ASD_ERR_DEVICE_TIMEOUT) instead of a hung GPU.
#pragma once
#include <cuda.h>
#include <cuda_runtime.h>
#include <stdint.h>

namespace asd {

constexpr int kSlotBytes = 8192;             // one ring slot: 8 weight rows x 512 bf16 inputs, or one 64-key K/V box
constexpr long long kWaitCycles = 4000000000LL;  // default budget of one wait: ~2 s at 2 GHz

enum DeviceError : int {
    kErrNone = 0,
    kErrFullWait = 1,    // consumer: data never arrived in a slot
    kErrEmptyWait = 2,   // producer: slot never released
    kErrGridWait = 3,    // grid barrier never completed
};

__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint64_t* bar, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(bar)), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_fence_init() { asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory"); }
__device__ __forceinline__ void mbar_expect_tx(uint64_t* bar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_u32(bar)), "r"(bytes) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint64_t* bar) {
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_u32(bar)) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint64_t* bar, uint32_t parity) {
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok)
        : "r"(smem_u32(bar)), "r"(parity)
        : "memory");
    return ok != 0;
}

// Wait for a phase of an mbarrier. Returns false when the wait was abandoned (error word set).
// The first wait to give up also records where it was: err[1..7] = stage, ring item, slot, CTA, thread, tag, parity.
__device__ __forceinline__ bool mbar_wait(uint64_t* bar, uint32_t parity, volatile int* err, int code, int stage = -1,
                                          unsigned item = 0, int slot = -1, int tag = 0, long long budget = kWaitCycles) {
    if (mbar_try_wait(bar, parity)) return true;
    const long long t0 = clock64();
    for (unsigned spin = 1;; ++spin) {
        if (mbar_try_wait(bar, parity)) return true;
        if ((spin & 255u) != 0) continue;  // the error word lives in global memory: look at it only now and then
        if (*err != kErrNone) return false;
        if (clock64() - t0 > budget) {
            if (atomicCAS(const_cast<int*>(err), kErrNone, code) == kErrNone) {
                err[1] = stage, err[2] = (int)item, err[3] = slot, err[4] = blockIdx.x, err[5] = threadIdx.x, err[6] = tag;
                err[7] = (int)parity;
            }
            return false;
        }
    }
}

// 1-D bulk copy global -> shared, completion counted on an mbarrier. Both addresses 16-byte aligned, size % 16 == 0.
__device__ __forceinline__ void tma_load_1d(void* smem_dst, const void* gsrc, uint32_t bytes, uint64_t* bar) {
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(
                     smem_u32(smem_dst)),
                 "l"(gsrc), "r"(bytes), "r"(smem_u32(bar))
                 : "memory");
}
// same, with an L2 eviction-priority policy (from make_policy_evict_first): data that is read exactly once
__device__ __forceinline__ void tma_load_1d_hint(void* smem_dst, const void* gsrc, uint32_t bytes, uint64_t* bar, uint64_t policy) {
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes.L2::cache_hint [%0], [%1], %2, [%3], %4;" ::"r"(
                     smem_u32(smem_dst)),
                 "l"(gsrc), "r"(bytes), "r"(smem_u32(bar)), "l"(policy)
                 : "memory");
}
__device__ __forceinline__ uint64_t make_policy_evict_first() {
    uint64_t pol;
    asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(pol));
    return pol;
}
// 2-D tiled copy global -> shared through a tensor map (x = innermost coordinate; x * element size % 16 == 0).
__device__ __forceinline__ void tma_load_2d(void* smem_dst, const CUtensorMap* map, int x, int y, uint64_t* bar) {
    asm volatile(
        "cp.async.bulk.tensor.2d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];" ::"r"(
            smem_u32(smem_dst)),
        "l"(map), "r"(x), "r"(y), "r"(smem_u32(bar))
        : "memory");
}
// make generic-proxy accesses to shared memory ordered before later async-proxy (TMA) accesses
__device__ __forceinline__ void fence_proxy_async_smem() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }

__device__ __forceinline__ void bar_sync(int id, int threads) {
    asm volatile("bar.sync %0, %1;" ::"r"(id), "r"(threads) : "memory");
}

__device__ __forceinline__ unsigned ld_acquire_gpu(const unsigned* p) {
    unsigned v;
    asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
    return v;
}

// packed fp32 pair arithmetic (two FMAs per instruction on sm_100)
__device__ __forceinline__ unsigned long long pack2(float lo, float hi) {
    unsigned long long r;
    asm("mov.b64 %0, {%1, %2};" : "=l"(r) : "f"(lo), "f"(hi));
    return r;
}
__device__ __forceinline__ void unpack2(unsigned long long v, float& lo, float& hi) {
    asm("mov.b64 {%0, %1}, %2;" : "=f"(lo), "=f"(hi) : "l"(v));
}
__device__ __forceinline__ unsigned long long ffma2(unsigned long long a, unsigned long long b, unsigned long long c) {
    unsigned long long d;
    asm("fma.rn.f32x2 %0, %1, %2, %3;" : "=l"(d) : "l"(a), "l"(b), "l"(c));
    return d;
}
// exact g / d for 0 <= g < 2^22 and 1 <= d <= 64, with magic = 2^32 / d + 1 (computed on the host)
__device__ __forceinline__ uint32_t fast_div(uint32_t g, uint32_t magic) { return __umulhi(g, magic); }

// a packed bf16 pair (element k in the low half, k+1 in the high half) widened to a packed fp32 pair
__device__ __forceinline__ unsigned long long bf2_to_f2(uint32_t u) {
    return pack2(__uint_as_float(u << 16), __uint_as_float(u & 0xFFFF0000u));
}

}  // namespace asd
