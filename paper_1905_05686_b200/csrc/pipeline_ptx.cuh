// Pieces shared by the kernels that run a TMA + mbarrier pipeline: bounded barrier waits, bulk tensor
// copies, and the host-side tensor-map encoder.
#pragma once
#include <cuda.h>

#include <mutex>

#include "lrbi_common.cuh"

namespace lrbi {

constexpr long long TC_WAIT_LIMIT_CYCLES = 4000000000ll;          // about 2 s of SM clock
constexpr uint32_t TC_SUSPEND_HINT_NS = 20000u;                   // a waiting thread may sleep this long per try

// ------------------------------------------------------------------------------ PTX wrappers
__device__ __forceinline__ uint32_t smem_u32(const void *p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint64_t *bar, uint32_t count)
{
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(bar)), "r"(count));
}
__device__ __forceinline__ void mbar_arrive(uint64_t *bar)
{
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_u32(bar)) : "memory");
}
__device__ __forceinline__ void mbar_arrive_expect_tx(uint64_t *bar, uint32_t bytes)
{
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_u32(bar)), "r"(bytes) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint64_t *bar, uint32_t parity)
{
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2, %3;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok) : "r"(smem_u32(bar)), "r"(parity), "r"(TC_SUSPEND_HINT_NS) : "memory");
    return ok != 0;
}
// Bounded wait.  Returns false if the block is aborting or the limit ran out (then it records
// `code` and raises the abort flag).  The limit is counted on the SM's own cycle counter, which is
// cheap to read; it is looked at once every 64 unsuccessful tries.
__device__ __forceinline__ bool mbar_wait(uint64_t *bar, uint32_t parity, volatile int *abort_flag,
                                          int *status, int code, long long limit = TC_WAIT_LIMIT_CYCLES)
{
    if (mbar_try_wait(bar, parity)) return true;
    long long t0 = 0;
    unsigned backoff = 32;
    for (unsigned spins = 1;; ++spins) {
        // back off between tries: a hot polling loop steals issue slots and shared-memory queue
        // bandwidth from the warps that are doing the work this warp is waiting for
        __nanosleep(backoff);
        if (backoff < 256) backoff <<= 1;
        if (mbar_try_wait(bar, parity)) return true;
        if (*abort_flag) return false;
        if ((spins & 63u) == 0) {
            const long long now = clock64();
            if (t0 == 0) t0 = now;
            else if (now - t0 > limit) {
                atomicCAS(status, 0, code);
                *abort_flag = 1;
                __threadfence_block();
                return false;
            }
        }
    }
}

__device__ __forceinline__ void tma_load_2d(void *dst, const CUtensorMap *map, uint64_t *bar, int x, int y)
{
    asm volatile(
        "cp.async.bulk.tensor.2d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4}], [%2];"
        ::"r"(smem_u32(dst)), "l"(map), "r"(smem_u32(bar)), "r"(x), "r"(y) : "memory");
}


// ------------------------------------------------------------------------------ host: tensor maps
typedef CUresult (*EncodeTiledFn)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *,
                                  const cuuint64_t *, const cuuint32_t *, const cuuint32_t *, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

inline EncodeTiledFn get_encode_fn()
{
    static EncodeTiledFn fn = nullptr;
    std::lock_guard<std::mutex> lock(lib_mutex());
    if (!fn) {
        void *p = nullptr;
        cudaDriverEntryPointQueryResult qres;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &qres) == cudaSuccess &&
            qres == cudaDriverEntryPointSuccess)
            fn = reinterpret_cast<EncodeTiledFn>(p);
    }
    return fn;
}


}  // namespace lrbi
