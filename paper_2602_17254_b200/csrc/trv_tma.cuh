// Tile fetch by TMA for the fused latency kernels whose tile is 32 element columns x n ranks in
// shared memory.  When the caller's rank buffers are equally spaced, one tensor map describes them as
// an [n][count] matrix of 4-byte words; one thread of a CTA issues n / rows_per_box bulk tensor copies
// (cp.async.bulk.tensor.2d, boxes of 32 columns x at most 243 ranks, each to this CTA alone) that complete on
// an mbarrier, so the whole tile is in flight at once.  Columns beyond `count` arrive as zeros.
// It pays where a thread would otherwise have few loads in flight (9x9x9: nine per thread, 10.1 -> 8.4 ms);
// the line-group kernel, whose threads issue 27 or 81 loads at once, got slower with it (27x27: 0.60 -> 0.39
// of the copy bandwidth) and keeps its direct loads.
// The wait on the mbarrier is bounded; a CTA that gives up adds one to a device-side counter
// (kernel argument from tma_giveup_counter(); trv_tma_giveups in the C interface) and leaves without storing anything.
#pragma once
#include <cuda.h>

#include "trv_dev.cuh"

namespace trv {

constexpr unsigned kTmaWaitLimit = 1u << 22;    // try_wait polls (each suspends for a while): far beyond any real copy

__device__ __forceinline__ unsigned smem_u32(const void* p) { return (unsigned)__cvta_generic_to_shared(p); }

// Called by every thread of the CTA.  slab: [rows][32] words, 128-byte aligned; bar: 8 bytes of shared
// memory; x0: first column (a multiple of 4); rows = boxes * box_rows.  True when the tile has arrived.
__device__ __forceinline__ bool tma_fetch_tile(const CUtensorMap* tmap, void* slab, unsigned long long* bar, int x0, int boxes,
                                               int box_rows, unsigned* giveups) {
    const unsigned bar_s = smem_u32(bar), slab_s = smem_u32(slab);
    if (threadIdx.x == 0) {
        asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar_s), "r"(1) : "memory");
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
        asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar_s), "r"(boxes * box_rows * 128) : "memory");
        for (int b = 0; b < boxes; ++b)
            asm volatile(
                "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];" ::"r"(
                    slab_s + b * box_rows * 128),
                "l"(tmap), "r"(x0), "r"(b * box_rows), "r"(bar_s)
                : "memory");
    }
    __syncthreads();                    // the barrier is initialised before anybody polls it
    unsigned done = 0;
    for (unsigned spins = 0; spins < kTmaWaitLimit; ++spins) {
        asm volatile(
            "{\n\t.reg .pred p;\n\tmbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\tselp.u32 %0, 1, 0, p;\n\t}"
            : "=r"(done)
            : "r"(bar_s), "r"(0)
            : "memory");
        if (done) break;
    }
    if (!__syncthreads_and((int)done)) {
        if (threadIdx.x == 0) atomicAdd(giveups, 1u);
        return false;
    }
    return true;
}

// Host: the tensor map of n equally spaced rank buffers of `count` words, boxes of 32 x box_rows.
// false: not expressible (spacing no multiple of 16 bytes, buffers overlapping, driver entry missing).
bool tma_encode_ranks(const StrideAddr& in, int n, size_t count, int box_rows, CUtensorMap* out);
// Tensor maps of the three slices of a 9 x 9 x 9 torus, one C-plane of box_cols columns per box (trv_fused_t999_tma.cu)
struct PlaneMaps {
    CUtensorMap in[3], out[3];      // one pair per slice: dimensions ordered by increasing rank stride
};
bool encode_planes(const StrideAddr& base, size_t count, const int strides[3], int box_cols, CUtensorMap* out);
bool tma_encode_raw(CUtensorMap* out, int rank, void* base, const cuuint64_t* gdim, const cuuint64_t* gstride, const cuuint32_t* box);
unsigned* tma_giveup_counter();     // device address of the counter on the current device (NULL on failure)
unsigned tma_giveups();             // its value (synchronous copy); ~0u on failure

}  // namespace trv
