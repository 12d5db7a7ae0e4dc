// Bounded device-side waits on readiness entries, shared by the kernels whose warps hand work to
// one another through global memory (trv_pipe.cu).
#pragma once
#include "trv_dev.cuh"

namespace trv {

constexpr unsigned kSpinLimit = 1u << 21;     // polls of >= 200 ns each: gives up after roughly half a second
constexpr size_t kPipeHeaderBytes = 256;

struct PipeHeader {
    unsigned long long ticket;
    int error;                  // 0, or TRV_ERR_TIMEOUT
    int pad;
    long long where;            // the item that gave up
};

__device__ __forceinline__ int ld_acquire(const int* p) {
    int v;
    asm volatile("ld.acquire.gpu.global.s32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
    return v;
}
__device__ __forceinline__ void st_release(int* p, int v) {
    asm volatile("st.release.gpu.global.s32 [%0], %1;" ::"l"(p), "r"(v) : "memory");
}
// Waits until *entry >= need.  false: gave up (limit reached or another waiter already gave up).
__device__ __forceinline__ bool wait_entry(const int* entry, int need, PipeHeader* hdr, unsigned limit, long long item) {
    unsigned spins = 0;
    while (ld_acquire(entry) < need) {
        if (ld_acquire(&hdr->error) != 0) return false;
        if (++spins > limit) {
            if (atomicCAS(&hdr->error, 0, (int)TRV_ERR_TIMEOUT) == 0) hdr->where = item;
            return false;
        }
        __nanosleep(200);
    }
    return true;
}

}  // namespace trv
