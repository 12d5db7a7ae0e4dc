// Shared device-side helpers and the internal call descriptor.
#pragma once
#include <cuda_runtime.h>

#include <atomic>
#include <cstdint>
#include <type_traits>

#include "trv_plan.h"

namespace trv {

// Rank-pointer table passed BY VALUE in kernel parameter space (sm_100 allows 32 KB of
// parameters): no device-side table to upload, so a call is a pure launch sequence.
template <int CAP>
struct PtrTab {
    void* p[CAP];
};

struct Call {
    const Plan* plan;
    const void* const* in;      // host array of n device pointers
    void* const* out;           // host array of n device pointers (may equal in)
    size_t count;               // local elements per rank
    size_t gcount, goff;        // global vector length and offset of local element 0
    int dtype;
    bool in_place;
    void* scratch;
    size_t scratch_bytes;
    cudaStream_t st;
};

extern std::atomic<uint64_t> g_launches;
extern thread_local const char* g_last_kernel;

#define TRV_LAUNCH(kernel, grid, block, smem, stream, ...)                \
    do {                                                                  \
        kernel<<<(grid), (block), (smem), (stream)>>>(__VA_ARGS__);       \
        ::trv::g_launches.fetch_add(1, std::memory_order_relaxed);        \
    } while (0)

// Programmatic dependent launch: a kernel launched with TRV_LAUNCH_PDL may become resident while
// the previous kernel of the stream is still draining.  pdl_trigger() (first thing in a kernel)
// lets the NEXT kernel do that; pdl_wait() (before the first global-memory access) blocks until the
// PREVIOUS kernel has completed and its writes are visible, so stream order is fully preserved:
// only launch latency and the prologue overlap.  Both are no-ops without the launch attribute.
__device__ __forceinline__ void pdl_trigger() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }
__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }

template <typename... KArgs, typename... Args>
inline void launch_pdl(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t st, Args... args) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid; cfg.blockDim = block; cfg.dynamicSmemBytes = smem; cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr; cfg.numAttrs = 1;
    cudaLaunchKernelEx(&cfg, kernel, KArgs(args)...);
    g_launches.fetch_add(1, std::memory_order_relaxed);
}

// Kernels that need more than 48 KB of dynamic shared memory must opt in; the attribute belongs
// to the current device's copy of the function, so it is set (a cheap host-side call) at every
// launch rather than cached per process.
template <typename K>
inline bool allow_big_smem(K kernel, int bytes) {
    return cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, bytes) == cudaSuccess;
}

// (a + b) + c, one rounding per add, never contracted or reassociated.
__device__ __forceinline__ float add3(float a, float b, float c) { return __fadd_rn(__fadd_rn(a, b), c); }
__device__ __forceinline__ uint32_t add3(uint32_t a, uint32_t b, uint32_t c) { return (a + b) + c; }
__device__ __forceinline__ float add2(float a, float b) { return __fadd_rn(a, b); }
__device__ __forceinline__ uint32_t add2(uint32_t a, uint32_t b) { return a + b; }

// Two binary32 adds in one instruction (sm_100 packed FP32): each lane is an independent IEEE add,
// round to nearest even, no flush to zero -- bit-identical to two scalar adds, half the issue slots.
__device__ __forceinline__ float2 add2_f32x2(float2 a, float2 b) {
    unsigned long long ra = *reinterpret_cast<unsigned long long*>(&a);
    unsigned long long rb = *reinterpret_cast<unsigned long long*>(&b);
    unsigned long long rd;
    asm("add.rn.f32x2 %0, %1, %2;" : "=l"(rd) : "l"(ra), "l"(rb));
    return *reinterpret_cast<float2*>(&rd);
}

// V consecutive elements of one rank
template <typename T, int V>
struct alignas(sizeof(T) * V) Elem {
    T x[V];
};

template <typename T, int V>
__device__ __forceinline__ Elem<T, V> add2(const Elem<T, V>& a, const Elem<T, V>& b) {
    Elem<T, V> r;
    if constexpr (std::is_same<T, float>::value && V % 2 == 0) {      // even width: packed adds
#pragma unroll
        for (int k = 0; k < V; k += 2) {
            const float2 s = add2_f32x2(make_float2(a.x[k], a.x[k + 1]), make_float2(b.x[k], b.x[k + 1]));
            r.x[k] = s.x;
            r.x[k + 1] = s.y;
        }
    } else {
#pragma unroll
        for (int k = 0; k < V; ++k) r.x[k] = add2(a.x[k], b.x[k]);
    }
    return r;
}
template <typename T, int V>
__device__ __forceinline__ Elem<T, V> add3(const Elem<T, V>& a, const Elem<T, V>& b, const Elem<T, V>& c) {
    return add2(add2(a, b), c);
}

// Where rank r's buffer starts: either a table of n pointers in parameter space, or, when the
// caller's buffers are equally spaced (rows of one tensor), base + r * stride with no table at all.
template <int CAP>
struct TabAddr {
    PtrTab<CAP> t;
    __device__ __forceinline__ char* ptr(int rank) const { return (char*)t.p[rank]; }
};
struct StrideAddr {
    char* base;
    unsigned stride;    // bytes; 32-bit so that base + stride * rank is ONE 32x32->64 multiply-add
    __device__ __forceinline__ char* ptr(int rank) const { return base + (unsigned long long)stride * (unsigned)rank; }
};
// true (and base/stride filled) iff p[r] == p[0] + r * stride for all r with 0 <= stride < 2^32
inline bool uniform_stride(const void* const* p, int n, StrideAddr* out) {
    out->base = (char*)const_cast<void*>(p[0]);
    const long long st = n > 1 ? (long long)((const char*)p[1] - (const char*)p[0]) : 0;
    if (st < 0 || st > 0xffffffffLL) return false;
    out->stride = (unsigned)st;
    for (int r = 2; r < n; ++r)
        if ((const char*)p[r] - (const char*)p[r - 1] != st) return false;
    return true;
}

template <typename T> struct Vec4;
template <> struct Vec4<float> { using type = float4; };
template <> struct Vec4<uint32_t> { using type = uint4; };

template <typename V>
__device__ __forceinline__ V add3v(const V& a, const V& b, const V& c) {
    V r;
    r.x = add3(a.x, b.x, c.x); r.y = add3(a.y, b.y, c.y);
    r.z = add3(a.z, b.z, c.z); r.w = add3(a.w, b.w, c.w);
    return r;
}

// Torus geometry for kernels that do rank arithmetic on the device (sides of any size, at most four dimensions).
struct TorusGeo {
    int nd;
    int dims[4], stride[4];
    int shift[4];       // bit position of coordinate d in a packed coordinate vector (fields of ceil(log2 side) bits)
};
inline TorusGeo make_geo(const Plan& p) {
    TorusGeo g;
    g.nd = p.ndims;
    int pos = 0;
    for (int d = 0; d < 4; ++d) {
        g.dims[d] = d < p.ndims ? p.dims[d] : 1;
        g.stride[d] = d < p.ndims ? p.stride[d] : p.n;
        g.shift[d] = pos;
        int w = 0;
        while ((1 << w) < g.dims[d]) ++w;
        pos += w;
    }
    return g;
}
// coordinates of a rank (or of an offset), packed; and base + offset from two packed vectors
__device__ __forceinline__ unsigned geo_pack(const TorusGeo& g, int r) {
    unsigned v = 0;
#pragma unroll
    for (int d = 0; d < 4; ++d)
        if (d < g.nd) v |= (unsigned)((r / g.stride[d]) % g.dims[d]) << g.shift[d];
    return v;
}
__device__ __forceinline__ int geo_add_packed(const TorusGeo& g, unsigned base, unsigned off) {
    int out = 0;
#pragma unroll
    for (int d = 0; d < 4; ++d)
        if (d < g.nd) {
            const unsigned hi = d + 1 < g.nd ? (unsigned)g.shift[d + 1] : 32u;
            const unsigned m = hi - g.shift[d] >= 32u ? ~0u : ((1u << (hi - g.shift[d])) - 1u);
            int x = (int)((base >> g.shift[d]) & m) + (int)((off >> g.shift[d]) & m);
            if (x >= g.dims[d]) x -= g.dims[d];
            out += x * g.stride[d];
        }
    return out;
}
// node + offset and node - offset, coordinate by coordinate modulo the sides
__device__ __forceinline__ int geo_add(const TorusGeo& g, int r, int o) {
    int out = 0;
#pragma unroll
    for (int d = 0; d < 4; ++d)
        if (d < g.nd) {
            int x = (r / g.stride[d]) % g.dims[d] + (o / g.stride[d]) % g.dims[d];
            if (x >= g.dims[d]) x -= g.dims[d];
            out += x * g.stride[d];
        }
    return out;
}
__device__ __forceinline__ int geo_sub(const TorusGeo& g, int r, int o) {
    int out = 0;
#pragma unroll
    for (int d = 0; d < 4; ++d)
        if (d < g.nd) {
            int x = (r / g.stride[d]) % g.dims[d] - (o / g.stride[d]) % g.dims[d];
            if (x < 0) x += g.dims[d];
            out += x * g.stride[d];
        }
    return out;
}
// the node `delta` positions further along dimension d (|delta| < side)
__device__ __forceinline__ int geo_shift(const TorusGeo& g, int r, int d, int delta) {
    const int a = g.dims[d], st = g.stride[d];
    const int x = (r / st) % a;
    int y = x + delta;
    if (y < 0) y += a;
    if (y >= a) y -= a;
    return r + (y - x) * st;
}

// step-family launchers (trv_step.cu)
trv_status_t run_step_latency(const Call& c);
trv_status_t run_step_bandwidth(const Call& c);
trv_status_t run_step_general(const Call& c);
size_t step_scratch_bytes(const Plan& p, size_t count, bool in_place);

// fused-family launchers (trv_fused_lat.cu / trv_fused_bw.cu)
bool fused_latency_supported(const Plan& p);
bool fused_bandwidth_supported(const Plan& p);
trv_status_t run_fused_latency(const Call& c);
trv_status_t run_fused_bandwidth(const Call& c);
// rings of any other size (trv_fused_tree.cu)
bool fused_tree_supported(const Plan& p);
void tree_prepare(Plan& p);         // once per plan: the stack-machine programs
void latency_prepare(Plan& p);      // once per plan: which latency kernel, and the line-group program if that is the one
trv_status_t run_fused_tree(const Call& c);

// chunk-level readiness engine (trv_pipe.cu)
bool pipeline_supported(const Plan& p, bool in_place);
size_t pipeline_scratch_bytes(const Plan& p, size_t count);
trv_status_t run_pipeline_latency(const Call& c);
trv_status_t pipeline_status(const void* scratch, cudaStream_t st);
trv_status_t pipeline_selftest_timeout(void* scratch, size_t scratch_bytes, cudaStream_t st);
// the same engine for the bandwidth-optimal form (trv_pipe_bw.cu)
bool pipeline_bw_supported(const Plan& p);
size_t pipeline_bw_scratch_bytes(const Plan& p, size_t gcount);
trv_status_t run_pipeline_bandwidth(const Call& c);

// joint reduction on host-described segments (trv_joint.cu); the comparator schedules run through it (trv_comparator.cu)
trv_status_t joint_run(const void* const* left, const void* const* own, const void* const* right, void* const* out,
                       const size_t* counts, size_t nsegments, int dtype, cudaStream_t st);
size_t comparator_scratch_bytes(const Plan& p, size_t count);
trv_status_t run_comparator(const Call& c);

// link-load tally (trv_linkloads.cu)
trv_status_t run_link_loads(const Plan& p, size_t count, size_t elem_size, int32_t* msgs, int64_t* bytes,
                            int32_t* max_msgs, int64_t* max_bytes);

// local column range [lo,hi) of slice c inside the window the call holds
inline void local_slice(const Call& c, int slice, long long* lo, long long* hi) {
    const int D = c.plan->ndims;
    long long glo = slice_lo((int64_t)c.gcount, D, slice), ghi = slice_lo((int64_t)c.gcount, D, slice + 1);
    long long w0 = (long long)c.goff, w1 = (long long)(c.goff + c.count);
    glo = glo < w0 ? w0 : (glo > w1 ? w1 : glo);
    ghi = ghi < w0 ? w0 : (ghi > w1 ? w1 : ghi);
    *lo = glo - w0;
    *hi = ghi - w0;
}

}  // namespace trv
