// STEP kernels for rings and tori with a side that is no power of three (Sec. 4.4, Sec. 5), bandwidth-optimal form.
//
// One launch per schedule step and collective, in place in the output buffers.  The tree a block follows is
// stored by offset from the block's owner (Plan::gstep / gsgn); per step the host lists
//   Reduce-Scatter: the offsets o at which a node receives, with which sides send to it;
//                   the node p at offset o from block b = p - o adds (left + own) + right,
//                   leaving out a side nothing comes from;
//   AllGather:      the offsets o at which a node receives the finished block, and from which side.
// A node writes its partial of a block only in steps before the one in which it sends it on, and
// the node it sends to reads it in exactly that step, so no step reads what the same step writes.
#include <algorithm>
#include <vector>

#include "trv_dev.cuh"

namespace trv {

constexpr int kGenThreads = 256;

// entry: offset (bits 0..9) | flag A (bit 10) | flag B (bit 11)
template <int CAP>
struct GenTab {
    int cnt;
    unsigned short e[CAP];
};
struct GenArgs {
    long long slo, shi, w0, w1;     // the collective's slice of the global vector; the buffers hold elements [w0, w1)
    int n, dim, dist;               // the step's dimension and distance
    TorusGeo geo;
};

__device__ __forceinline__ void gen_block_range(const GenArgs& a, int j, long long* lo, long long* hi) {
    const unsigned long long len = (unsigned long long)(a.shi - a.slo);
    long long b0 = a.slo + (long long)(((unsigned long long)j * len) / (unsigned)a.n);
    long long b1 = a.slo + (long long)(((unsigned long long)(j + 1) * len) / (unsigned)a.n);
    b0 = b0 < a.w0 ? a.w0 : (b0 > a.w1 ? a.w1 : b0);
    b1 = b1 < a.w0 ? a.w0 : (b1 > a.w1 ? a.w1 : b1);
    *lo = b0 - a.w0;
    *hi = b1 - a.w0;
}

// elements [lo, hi) spread over the x dimension of the grid; 16-byte accesses on the aligned body
template <typename F1, typename F4>
__device__ __forceinline__ void gen_for_range(long long lo, long long hi, F1 f1, F4 f4) {
    if (hi <= lo) return;
    long long alo = (lo + 3) & ~3LL;
    if (alo > hi) alo = hi;
    long long ahi = hi & ~3LL;
    if (ahi < alo) ahi = alo;
    const long long tid = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    const long long nth = (long long)gridDim.x * blockDim.x;
    const long long head = alo - lo, tail = hi - ahi;
    if (tid < head) f1(lo + tid);
    else if (tid < head + tail) f1(ahi + (tid - head));
    for (long long v = tid; v < (ahi - alo) / 4; v += nth) f4(alo + 4 * v);
}

template <typename V>
__device__ __forceinline__ V add2v(const V& a, const V& b) {
    V r;
    r.x = add2(a.x, b.x); r.y = add2(a.y, b.y);
    r.z = add2(a.z, b.z); r.w = add2(a.w, b.w);
    return r;
}

// Reduce-Scatter step: grid (x, receiving offsets, n)
template <typename T, int CAP>
__global__ void __launch_bounds__(kGenThreads) k_rs_gen(PtrTab<CAP> buf, GenTab<CAP> tab, GenArgs a) {
    using V = typename Vec4<T>::type;
    pdl_trigger();
    pdl_wait();
    const int p = blockIdx.z;
    const unsigned ent = tab.e[blockIdx.y];
    const int o = ent & 1023;
    const bool from_left = ent & 1024, from_right = ent & 2048;
    const int b = geo_sub(a.geo, p, o);
    const int ql = geo_shift(a.geo, p, a.dim, -a.dist), qr = geo_shift(a.geo, p, a.dim, a.dist);
    const T* __restrict__ L = (const T*)buf.p[ql];
    const T* __restrict__ R = (const T*)buf.p[qr];
    T* __restrict__ O = (T*)buf.p[p];
    long long lo, hi;
    gen_block_range(a, b, &lo, &hi);
    if (from_left && from_right) {
        gen_for_range(
            lo, hi, [&](long long e) { O[e] = add3(L[e], O[e], R[e]); },
            [&](long long e) { *(V*)(O + e) = add3v(*(const V*)(L + e), *(const V*)(O + e), *(const V*)(R + e)); });
    } else if (from_left) {
        gen_for_range(
            lo, hi, [&](long long e) { O[e] = add2(L[e], O[e]); },
            [&](long long e) { *(V*)(O + e) = add2v(*(const V*)(L + e), *(const V*)(O + e)); });
    } else {
        gen_for_range(
            lo, hi, [&](long long e) { O[e] = add2(O[e], R[e]); },
            [&](long long e) { *(V*)(O + e) = add2v(*(const V*)(O + e), *(const V*)(R + e)); });
    }
}

// AllGather step: grid (x, receiving offsets, n); flag A = the block comes from node + dist
template <int CAP>
__global__ void __launch_bounds__(kGenThreads) k_ag_gen(PtrTab<CAP> buf, GenTab<CAP> tab, GenArgs a) {
    pdl_trigger();
    pdl_wait();
    const int p = blockIdx.z;
    const unsigned ent = tab.e[blockIdx.y];
    const int o = ent & 1023;
    const int b = geo_sub(a.geo, p, o);
    const int q = geo_shift(a.geo, p, a.dim, (ent & 1024) ? a.dist : -a.dist);
    const uint32_t* __restrict__ S = (const uint32_t*)buf.p[q];
    uint32_t* __restrict__ O = (uint32_t*)buf.p[p];
    long long lo, hi;
    gen_block_range(a, b, &lo, &hi);
    gen_for_range(
        lo, hi, [&](long long e) { O[e] = S[e]; }, [&](long long e) { *(uint4*)(O + e) = *(const uint4*)(S + e); });
}

template <int CAP>
__global__ void __launch_bounds__(kGenThreads) k_copy_gen(PtrTab<CAP> src, PtrTab<CAP> dst, long long count) {
    pdl_trigger();
    pdl_wait();
    const uint32_t* __restrict__ S = (const uint32_t*)src.p[blockIdx.y];
    uint32_t* __restrict__ O = (uint32_t*)dst.p[blockIdx.y];
    gen_for_range(
        0, count, [&](long long e) { O[e] = S[e]; }, [&](long long e) { *(uint4*)(O + e) = *(const uint4*)(S + e); });
}

static unsigned gen_grid_x(long long len) {
    long long g = (len / 4 + kGenThreads - 1) / kGenThreads;
    if (g < 1) g = 1;
    if (g > 4096) g = 4096;
    return (unsigned)g;
}

template <int CAP>
static trv_status_t gen_impl(const Call& c) {
    const Plan& p = *c.plan;
    const int n = p.n, S = p.S;
    PtrTab<CAP> IN, OUT;
    for (int r = 0; r < n; ++r) { IN.p[r] = const_cast<void*>(c.in[r]); OUT.p[r] = c.out[r]; }
    if (!c.in_place) {
        dim3 grid(gen_grid_x((long long)c.count), n, 1);
        launch_pdl(k_copy_gen<CAP>, grid, dim3(kGenThreads), 0, c.st, IN, OUT, (long long)c.count);
    }
    GenArgs a;
    a.w0 = (long long)c.goff; a.w1 = (long long)(c.goff + c.count); a.n = n;
    a.geo = make_geo(p);
    for (int row = 0; row < 2 * S; ++row) {
        const int t = p.step_of_row(row);
        for (int sl = 0; sl < p.nslices; ++sl) {
            a.slo = slice_lo((int64_t)c.gcount, p.nslices, sl); a.shi = slice_lo((int64_t)c.gcount, p.nslices, sl + 1);
            if (std::min(a.shi, a.w1) <= std::max(a.slo, a.w0)) continue;      // nothing of this collective in the window
            const long long max_len = (a.shi - a.slo) / n + 1;
            const std::vector<int8_t>&gs = p.gstep[sl], &gg = p.gsgn[sl];
            a.dim = p.steps[sl][t].dim; a.dist = p.steps[sl][t].dist;
            GenTab<CAP> tab;
            tab.cnt = 0;
            if (row < S) {
                for (int o = 0; o < n; ++o) {
                    const int ol = p.shift(o, a.dim, -a.dist), orr = p.shift(o, a.dim, a.dist);
                    const bool fl = gs[ol] == t && gg[ol] > 0;
                    const bool fr = orr != ol && gs[orr] == t && gg[orr] < 0;
                    if (fl || fr) tab.e[tab.cnt++] = (unsigned short)(o | (fl ? 1024 : 0) | (fr ? 2048 : 0));
                }
            } else {
                for (int o = 1; o < n; ++o)
                    if (gs[o] == t) tab.e[tab.cnt++] = (unsigned short)(o | (gg[o] > 0 ? 1024 : 0));
            }
            if (tab.cnt == 0) continue;
            dim3 grid(gen_grid_x(max_len), tab.cnt, n);
            if (row >= S) launch_pdl(k_ag_gen<CAP>, grid, dim3(kGenThreads), 0, c.st, OUT, tab, a);
            else if (c.dtype == TRV_FLOAT32) launch_pdl(k_rs_gen<float, CAP>, grid, dim3(kGenThreads), 0, c.st, OUT, tab, a);
            else launch_pdl(k_rs_gen<uint32_t, CAP>, grid, dim3(kGenThreads), 0, c.st, OUT, tab, a);
        }
    }
    return cudaGetLastError() == cudaSuccess ? TRV_OK : TRV_ERR_CUDA;
}

trv_status_t run_step_general(const Call& c) {
    g_last_kernel = "step_general";
    if (!c.plan->general) return TRV_ERR_UNSUPPORTED;
    if (c.plan->n <= 32) return gen_impl<32>(c);
    if (c.plan->n <= 256) return gen_impl<256>(c);
    return gen_impl<TRV_MAX_RANKS>(c);
}

}  // namespace trv
