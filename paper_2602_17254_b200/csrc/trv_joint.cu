// trv_joint_reduce: the joint reduction of Sec. 3.1 / 4.2 on caller-described segments,
//     out[s][e] = (left[s][e] + own[s][e]) + right[s][e],      e < counts[s],
// a side whose pointer is NULL being left out.  It is the one arithmetic primitive a schedule needs whose steps are
// driven from outside the library: the rank-sharded form, where every process holds the partials of its own ranks
// and the two received partials lie in receive buffers (rank_shard.py), runs its steps through it.
//
// Up to kJointBatch segments travel by value in kernel-parameter space per launch; a CTA row (blockIdx.y) owns a
// segment.  Accesses are 16 bytes wide where the four pointers of a segment share their alignment, else scalar.
#include "trv_dev.cuh"

namespace trv {

constexpr int kJointBatch = 512;
constexpr int kJointThreads = 256;

struct JointBatch {
    const void* l[kJointBatch];
    const void* m[kJointBatch];
    const void* r[kJointBatch];
    void* o[kJointBatch];
    long long cnt[kJointBatch];
};

template <typename T>
__global__ void __launch_bounds__(kJointThreads) k_joint_reduce(const __grid_constant__ JointBatch b) {
    using V = typename Vec4<T>::type;
    const int s = blockIdx.y;
    const T* __restrict__ L = (const T*)b.l[s];
    const T* __restrict__ M = (const T*)b.m[s];
    const T* __restrict__ R = (const T*)b.r[s];
    T* __restrict__ O = (T*)b.o[s];
    const long long cnt = b.cnt[s];
    const long long tid = (long long)blockIdx.x * blockDim.x + threadIdx.x, nth = (long long)gridDim.x * blockDim.x;
    auto one = [&](long long e) {
        T v = M[e];
        if (L) v = add2(L[e], v);
        if (R) v = add2(v, R[e]);
        O[e] = v;
    };
    // elements before the first 16-byte boundary of O; the body is vectorised if every pointer reaches a boundary there too
    const unsigned mis = (unsigned)((uintptr_t)O & 15);
    const bool same = (((uintptr_t)M & 15) == mis) && (!L || ((uintptr_t)L & 15) == mis) && (!R || ((uintptr_t)R & 15) == mis);
    if (!same) {
        for (long long e = tid; e < cnt; e += nth) one(e);
        return;
    }
    long long head = mis ? (16 - mis) / 4 : 0;
    if (head > cnt) head = cnt;
    const long long body = (cnt - head) / 4;
    if (tid < head) one(tid);
    for (long long e = head + 4 * body + tid; e < cnt; e += nth) one(e);
    for (long long v = tid; v < body; v += nth) {
        const long long e = head + 4 * v;
        V x = *(const V*)(M + e);
        if (L) {
            const V l = *(const V*)(L + e);
            x.x = add2(l.x, x.x); x.y = add2(l.y, x.y); x.z = add2(l.z, x.z); x.w = add2(l.w, x.w);
        }
        if (R) {
            const V r = *(const V*)(R + e);
            x.x = add2(x.x, r.x); x.y = add2(x.y, r.y); x.z = add2(x.z, r.z); x.w = add2(x.w, r.w);
        }
        *(V*)(O + e) = x;
    }
}

}  // namespace trv

namespace trv {
trv_status_t joint_run(const void* const* left, const void* const* own, const void* const* right, void* const* out,
                       const size_t* counts, size_t nsegments, int dtype, cudaStream_t st) {
    static thread_local JointBatch b;        // 20 KB: kept off the stack
    size_t s = 0;
    while (s < nsegments) {
        int k = 0;
        long long longest = 0;
        for (; s < nsegments && k < kJointBatch; ++s) {
            if (counts[s] == 0) continue;
            b.l[k] = left ? left[s] : nullptr; b.m[k] = own[s]; b.r[k] = right ? right[s] : nullptr; b.o[k] = out[s];
            b.cnt[k] = (long long)counts[s];
            if (b.cnt[k] > longest) longest = b.cnt[k];
            ++k;
        }
        if (k == 0) break;
        long long gx = (longest / 4 + kJointThreads - 1) / kJointThreads;
        if (gx < 1) gx = 1;
        if (gx > 2048) gx = 2048;
        if (dtype == TRV_FLOAT32) TRV_LAUNCH(k_joint_reduce<float>, dim3((unsigned)gx, k, 1), kJointThreads, 0, st, b);
        else TRV_LAUNCH(k_joint_reduce<uint32_t>, dim3((unsigned)gx, k, 1), kJointThreads, 0, st, b);
        if (cudaGetLastError() != cudaSuccess) return TRV_ERR_CUDA;
    }
    return TRV_OK;
}
}  // namespace trv

using namespace trv;

extern "C" trv_status_t trv_joint_reduce(const void* const* left, const void* const* own, const void* const* right, void* const* out,
                                         const size_t* counts, size_t nsegments, trv_dtype_t dtype, void* cuda_stream) {
    if (!own || !out || !counts) return TRV_ERR_INVALID_ARG;
    if (dtype != TRV_INT32 && dtype != TRV_FLOAT32) return TRV_ERR_INVALID_ARG;
    for (size_t s = 0; s < nsegments; ++s) {
        if (counts[s] == 0) continue;
        if (!own[s] || !out[s]) return TRV_ERR_INVALID_ARG;
        if (((uintptr_t)own[s] | (uintptr_t)out[s] | (uintptr_t)(left ? left[s] : nullptr) | (uintptr_t)(right ? right[s] : nullptr)) & 3)
            return TRV_ERR_INVALID_ARG;
        if (counts[s] >= ((size_t)1 << 40)) return TRV_ERR_UNSUPPORTED;
    }
    const trv_status_t st = joint_run(left, own, right, out, counts, nsegments, (int)dtype, (cudaStream_t)cuda_stream);
    g_last_kernel = "joint_reduce";
    return st;
}
