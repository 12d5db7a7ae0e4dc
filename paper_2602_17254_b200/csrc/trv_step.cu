// STEP kernel family: one launch per schedule step, exactly as the paper states the steps.
//   latency form   (Sec. 4.2): new[p] = (old[p - dist] + old[p]) + old[p + dist] for every rank p
//                              and every element; ping-pong between buffers.
//   bandwidth form (Sec. 4.1, 4.3): Reduce-Scatter step = the same three-input reduction on the
//                              blocks of the closed-form set Pi only; AllGather step = block copies
//                              from both peers, steps in reverse order.  Both run in place: in a
//                              step the blocks a rank writes agree with it modulo 3^(k+1), the
//                              blocks it reads from its peers agree with it too and therefore
//                              disagree with the peer (3^k is no multiple of 3^(k+1)), so nobody
//                              reads a block that somebody writes in the same step.
#include "trv_dev.cuh"

namespace trv {

constexpr int kThreads = 256;

struct SliceStep {
    long long lo, hi;   // local element range of the slice
    int stride, size, dist;
};
struct LatStepArgs {
    int nslices;
    SliceStep s[TRV_MAX_DIMS];
};

// Applies f1(e) to the unaligned edges and f4(e) (e a multiple of 4) to the aligned body of [lo,hi),
// spread over gridDim.x * blockDim.x threads.
template <typename F1, typename F4>
__device__ __forceinline__ void for_range(long long lo, long long hi, F1 f1, F4 f4) {
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

template <typename T, int CAP>
__global__ void __launch_bounds__(kThreads) k_lat_step(PtrTab<CAP> src, PtrTab<CAP> dst, LatStepArgs a) {
    using V = typename Vec4<T>::type;
    pdl_trigger();
    pdl_wait();
    const int p = blockIdx.y;
    for (int c = 0; c < a.nslices; ++c) {
        const SliceStep s = a.s[c];
        const int x = (p / s.stride) % s.size;
        int xl = x - s.dist; if (xl < 0) xl += s.size;
        int xr = x + s.dist; if (xr >= s.size) xr -= s.size;
        const T* __restrict__ L = (const T*)src.p[p + (xl - x) * s.stride];
        const T* __restrict__ M = (const T*)src.p[p];
        const T* __restrict__ R = (const T*)src.p[p + (xr - x) * s.stride];
        T* __restrict__ O = (T*)dst.p[p];
        for_range(
            s.lo, s.hi, [&](long long e) { O[e] = add3(L[e], M[e], R[e]); },
            [&](long long e) {
                V l = *(const V*)(L + e), m = *(const V*)(M + e), r = *(const V*)(R + e);
                *(V*)(O + e) = add3v(l, m, r);
            });
    }
}

template <int CAP>
__global__ void __launch_bounds__(kThreads) k_copy(PtrTab<CAP> src, PtrTab<CAP> dst, long long count) {
    pdl_trigger();
    pdl_wait();
    const uint32_t* __restrict__ S = (const uint32_t*)src.p[blockIdx.y];
    uint32_t* __restrict__ O = (uint32_t*)dst.p[blockIdx.y];
    for_range(
        0, count, [&](long long e) { O[e] = S[e]; }, [&](long long e) { *(uint4*)(O + e) = *(const uint4*)(S + e); });
}

struct BwSlice {
    long long glo, ghi;         // global element range of the slice
    int stride, size, dist;     // this step's dimension
    int mod[TRV_MAX_DIMS];      // congruence modulus per dimension after this step
};
struct BwStepArgs {
    int nslices, n, D, nact;    // nact = blocks in one message = n / prod(mod)
    long long w0, w1;           // global window the buffers hold: elements [w0, w1)
    int dims[TRV_MAX_DIMS], dstride[TRV_MAX_DIMS];
    BwSlice s[TRV_MAX_DIMS];
};

// q-th block (0 <= q < nact) of the set that agrees with rank `r` modulo mod[d] in every dimension
__device__ __forceinline__ int nth_block(const BwStepArgs& a, const BwSlice& s, int r, int q) {
    int j = 0;
    for (int d = 0; d < a.D; ++d) {
        const int m = s.mod[d], cnt = a.dims[d] / m;
        const int i = q % cnt; q /= cnt;
        const int x = (r / a.dstride[d]) % a.dims[d];
        j += ((x % m) + m * i) * a.dstride[d];
    }
    return j;
}
__device__ __forceinline__ void block_range(const BwStepArgs& a, const BwSlice& s, int j, long long* lo, long long* hi) {
    const unsigned long long L = (unsigned long long)(s.ghi - s.glo);
    long long b0 = s.glo + (long long)(((unsigned long long)j * L) / (unsigned)a.n);
    long long b1 = s.glo + (long long)(((unsigned long long)(j + 1) * L) / (unsigned)a.n);
    b0 = b0 < a.w0 ? a.w0 : (b0 > a.w1 ? a.w1 : b0);
    b1 = b1 < a.w0 ? a.w0 : (b1 > a.w1 ? a.w1 : b1);
    *lo = b0 - a.w0;
    *hi = b1 - a.w0;
}

// Reduce-Scatter step: grid (x, nact, n)
template <typename T, int CAP>
__global__ void __launch_bounds__(kThreads) k_rs_step(PtrTab<CAP> buf, BwStepArgs a) {
    using V = typename Vec4<T>::type;
    pdl_trigger();
    pdl_wait();
    const int p = blockIdx.z;
    for (int c = 0; c < a.nslices; ++c) {
        const BwSlice& s = a.s[c];
        const int x = (p / s.stride) % s.size;
        int xl = x - s.dist; if (xl < 0) xl += s.size;
        int xr = x + s.dist; if (xr >= s.size) xr -= s.size;
        const T* __restrict__ L = (const T*)buf.p[p + (xl - x) * s.stride];
        const T* __restrict__ R = (const T*)buf.p[p + (xr - x) * s.stride];
        T* __restrict__ O = (T*)buf.p[p];
        long long lo, hi;
        block_range(a, s, nth_block(a, s, p, blockIdx.y), &lo, &hi);
        for_range(
            lo, hi, [&](long long e) { O[e] = add3(L[e], O[e], R[e]); },
            [&](long long e) {
                V l = *(const V*)(L + e), m = *(const V*)(O + e), r = *(const V*)(R + e);
                *(V*)(O + e) = add3v(l, m, r);
            });
    }
}

// AllGather step: grid (x, 2 * nact, n): rank p copies the finished blocks of both peers
template <int CAP>
__global__ void __launch_bounds__(kThreads) k_ag_step(PtrTab<CAP> buf, BwStepArgs a) {
    pdl_trigger();
    pdl_wait();
    const int p = blockIdx.z;
    const int side = blockIdx.y / a.nact, q = blockIdx.y % a.nact;
    for (int c = 0; c < a.nslices; ++c) {
        const BwSlice& s = a.s[c];
        const int x = (p / s.stride) % s.size;
        int y = side ? x + s.dist : x - s.dist;
        if (y < 0) y += s.size;
        if (y >= s.size) y -= s.size;
        const int peer = p + (y - x) * s.stride;
        const uint32_t* __restrict__ S = (const uint32_t*)buf.p[peer];
        uint32_t* __restrict__ O = (uint32_t*)buf.p[p];
        long long lo, hi;
        block_range(a, s, nth_block(a, s, peer, q), &lo, &hi);
        for_range(
            lo, hi, [&](long long e) { O[e] = S[e]; }, [&](long long e) { *(uint4*)(O + e) = *(const uint4*)(S + e); });
    }
}

// ------------------------------------------------------------------ host side

static size_t padded(size_t count) { return (count + 63) & ~(size_t)63; }

static int scratch_buffers(const Plan& p, bool in_place) {
    if (p.variant != TRV_LATENCY_OPTIMAL) return 0;
    if (!in_place) return p.S >= 2 ? 1 : 0;
    return (p.S % 2 == 0) ? 1 : (p.S == 1 ? 1 : 2);
}

size_t step_scratch_bytes(const Plan& p, size_t count, bool in_place) {
    return (size_t)scratch_buffers(p, in_place) * (size_t)p.n * padded(count) * 4;
}

static unsigned grid_x(long long max_len) {
    long long g = (max_len / 4 + kThreads - 1) / kThreads;
    if (g < 1) g = 1;
    if (g > 4096) g = 4096;
    return (unsigned)g;
}

template <int CAP>
static trv_status_t lat_impl(const Call& c) {
    const Plan& p = *c.plan;
    const int n = p.n, S = p.S;
    PtrTab<CAP> IN, OUT, A, B;
    const size_t pc = padded(c.count);
    for (int r = 0; r < n; ++r) {
        IN.p[r] = const_cast<void*>(c.in[r]);
        OUT.p[r] = c.out[r];
        A.p[r] = (char*)c.scratch + (size_t)r * pc * 4;
        B.p[r] = (char*)c.scratch + ((size_t)n + r) * pc * 4;
    }
    // destination of every step: the last one is OUT, no step writes what it reads
    const PtrTab<CAP>* dst[64];
    if (!c.in_place) {
        for (int t = S - 1, k = 0; t >= 0; --t, ++k) dst[t] = (k % 2 == 0) ? &OUT : &A;
    } else if (S % 2 == 0) {
        for (int t = 0; t < S; ++t) dst[t] = (t % 2 == 0) ? &A : &OUT;
    } else {
        dst[0] = &A;
        if (S >= 3) { dst[1] = &B; dst[2] = &OUT; }
        for (int t = 3; t < S; ++t) dst[t] = (t % 2 == 1) ? &A : &OUT;
    }
    const PtrTab<CAP>* src = &IN;
    long long max_len = 0;
    for (int sl = 0; sl < p.ndims; ++sl) {
        long long lo, hi;
        local_slice(c, sl, &lo, &hi);
        if (hi - lo > max_len) max_len = hi - lo;
    }
    for (int t = 0; t < S; ++t) {
        LatStepArgs a;
        a.nslices = p.ndims;
        for (int sl = 0; sl < p.ndims; ++sl) {
            local_slice(c, sl, &a.s[sl].lo, &a.s[sl].hi);
            const Step& st = p.steps[sl][t];
            a.s[sl].stride = p.stride[st.dim]; a.s[sl].size = p.dims[st.dim]; a.s[sl].dist = st.dist;
        }
        dim3 grid(grid_x(max_len), n, 1);
        if (c.dtype == TRV_FLOAT32) launch_pdl(k_lat_step<float, CAP>, grid, dim3(kThreads), 0, c.st, *src, *dst[t], a);
        else launch_pdl(k_lat_step<uint32_t, CAP>, grid, dim3(kThreads), 0, c.st, *src, *dst[t], a);
        src = dst[t];
    }
    if (src != &OUT) {      // only S == 1 in place: bring the result home
        dim3 grid(grid_x((long long)c.count), n, 1);
        launch_pdl(k_copy<CAP>, grid, dim3(kThreads), 0, c.st, *src, OUT, (long long)c.count);
    }
    return cudaGetLastError() == cudaSuccess ? TRV_OK : TRV_ERR_CUDA;
}

trv_status_t run_step_latency(const Call& c) {
    g_last_kernel = "step_latency";
    if (c.scratch_bytes < step_scratch_bytes(*c.plan, c.count, c.in_place)) return TRV_ERR_SCRATCH;
    if (c.plan->n <= 32) return lat_impl<32>(c);
    if (c.plan->n <= 256) return lat_impl<256>(c);
    return lat_impl<TRV_MAX_RANKS>(c);
}

template <int CAP>
static trv_status_t bw_impl(const Call& c) {
    const Plan& p = *c.plan;
    const int n = p.n, S = p.S, D = p.ndims;
    PtrTab<CAP> IN, OUT;
    for (int r = 0; r < n; ++r) { IN.p[r] = const_cast<void*>(c.in[r]); OUT.p[r] = c.out[r]; }
    if (!c.in_place) {
        dim3 grid(grid_x((long long)c.count), n, 1);
        launch_pdl(k_copy<CAP>, grid, dim3(kThreads), 0, c.st, IN, OUT, (long long)c.count);
    }
    for (int row = 0; row < 2 * S; ++row) {
        const int t = p.step_of_row(row);
        BwStepArgs a;
        a.nslices = D; a.n = n; a.D = D;
        a.w0 = (long long)c.goff; a.w1 = (long long)(c.goff + c.count);
        long long max_len = 0;
        int nact = n;
        for (int d = 0; d < D; ++d) { a.dims[d] = p.dims[d]; a.dstride[d] = p.stride[d]; }
        for (int sl = 0; sl < D; ++sl) {
            BwSlice& s = a.s[sl];
            s.glo = slice_lo((int64_t)c.gcount, D, sl); s.ghi = slice_lo((int64_t)c.gcount, D, sl + 1);
            const Step& st = p.steps[sl][t];
            s.stride = p.stride[st.dim]; s.size = p.dims[st.dim]; s.dist = st.dist;
            int prod = 1;
            for (int d = 0; d < D; ++d) { s.mod[d] = p.mod[sl][t][d]; prod *= s.mod[d]; }
            nact = n / prod;        // the same for every slice: base^(t+1) blocks classes
            long long bl = (s.ghi - s.glo) / n + 1;
            if (bl > max_len) max_len = bl;
        }
        a.nact = nact;
        if (row < S) {
            dim3 grid(grid_x(max_len), nact, n);
            if (c.dtype == TRV_FLOAT32) launch_pdl(k_rs_step<float, CAP>, grid, dim3(kThreads), 0, c.st, OUT, a);
            else launch_pdl(k_rs_step<uint32_t, CAP>, grid, dim3(kThreads), 0, c.st, OUT, a);
        } else {
            dim3 grid(grid_x(max_len), 2 * nact, n);
            launch_pdl(k_ag_step<CAP>, grid, dim3(kThreads), 0, c.st, OUT, a);
        }
    }
    return cudaGetLastError() == cudaSuccess ? TRV_OK : TRV_ERR_CUDA;
}

trv_status_t run_step_bandwidth(const Call& c) {
    g_last_kernel = "step_bandwidth";
    if (c.plan->n <= 32) return bw_impl<32>(c);
    if (c.plan->n <= 256) return bw_impl<256>(c);
    return bw_impl<TRV_MAX_RANKS>(c);
}

}  // namespace trv
