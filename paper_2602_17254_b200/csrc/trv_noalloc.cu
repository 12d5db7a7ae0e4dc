// trv_allreduce_noalloc: the step-by-step latency-form AllReduce for callers that must not
// allocate device memory.  Its ping-pong scratch is a fixed array that is part of the library
// image, so the call needs no cudaMalloc, no cudaFree and no memory pool.
#include <algorithm>
#include <mutex>
#include <vector>

#include "trv_dev.cuh"

#define TRV_NOALLOC_SCRATCH_BYTES (16u << 20)

// Device-resident scratch, reserved on every GPU that loads the library, for as long as the
// process lives.  Host code must never use this name as an address: on the host it is only a
// handle for cudaGetSymbolAddress.
static __device__ __align__(256) unsigned char g_noalloc_scratch[TRV_NOALLOC_SCRATCH_BYTES];

namespace {
constexpr int kMaxDevices = 64;
std::mutex g_setup_mutex;
void* g_scratch_addr[kMaxDevices] = {nullptr};

// Device address of the scratch array on the CURRENT device; looked up once per device.
trv_status_t scratch_address(void** out) {
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return TRV_ERR_CUDA;
    std::lock_guard<std::mutex> lock(g_setup_mutex);
    if (!g_scratch_addr[dev]) {
        void* ptr = nullptr;
        if (cudaGetSymbolAddress(&ptr, g_noalloc_scratch) != cudaSuccess || !ptr) {
            (void)cudaGetLastError();
            return TRV_ERR_CUDA;
        }
        g_scratch_addr[dev] = ptr;
    }
    *out = g_scratch_addr[dev];
    return TRV_OK;
}
}  // namespace

extern "C" {

size_t trv_noalloc_max_scratch_bytes(void) { return TRV_NOALLOC_SCRATCH_BYTES; }

trv_status_t trv_allreduce_noalloc(trv_plan_t plan, void* const* rank_buffers, size_t count, trv_dtype_t dtype,
                                   trv_op_t op, void* cuda_stream) {
    using namespace trv;
    if (!plan || !rank_buffers) return TRV_ERR_INVALID_ARG;
    const Plan& p = plan->plan;
    if (p.algo != TRV_ALGO_TRIVANCE || p.variant != TRV_LATENCY_OPTIMAL) return TRV_ERR_UNSUPPORTED;
    if (dtype != TRV_INT32 && dtype != TRV_FLOAT32) return TRV_ERR_INVALID_ARG;
    if (op != TRV_SUM) return TRV_ERR_UNSUPPORTED;
    if (count >= ((size_t)1 << 40)) return TRV_ERR_TOO_LARGE;     // before any count * 4 below
    // 16-byte aligned, pairwise disjoint: sort the start addresses (host stack/heap only, no device memory)
    std::vector<uintptr_t> starts((size_t)p.n);
    for (int r = 0; r < p.n; ++r) {
        if (!rank_buffers[r] || ((uintptr_t)rank_buffers[r] & 15)) return TRV_ERR_INVALID_ARG;
        starts[r] = (uintptr_t)rank_buffers[r];
    }
    std::sort(starts.begin(), starts.end());
    for (int r = 1; r < p.n; ++r)
        if (starts[r] - starts[r - 1] < count * 4) return TRV_ERR_INVALID_ARG;
    const size_t need = step_scratch_bytes(p, count, /*in_place=*/true);
    if (need > TRV_NOALLOC_SCRATCH_BYTES) return TRV_ERR_TOO_LARGE;
    if (count == 0) return TRV_OK;
    void* scratch = nullptr;
    trv_status_t st = scratch_address(&scratch);
    if (st != TRV_OK) return st;
    // Every step writes each scratch element it later reads, so nothing has to be cleared.
    Call c{&p, (const void* const*)rank_buffers, rank_buffers, count, count, 0, (int)dtype, true,
           scratch, TRV_NOALLOC_SCRATCH_BYTES, (cudaStream_t)cuda_stream};
    return run_step_latency(c);
}

}  // extern "C"
