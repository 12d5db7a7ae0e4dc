// FUSED kernels of the latency-optimal form (Sec. 4.2): all log3 n joint-reduction steps of a
// column of elements run on chip, so every element is read from HBM once and written once.
//
// Every rank has its own reduction tree (the n results differ in rounding), so the work is
// 2*S*n adds per element column and cannot be shared between ranks.  The kernels keep whole
// "closed groups" of ranks in registers: a set of ranks is closed under a group of steps if
// every step maps the set onto itself, e.g. the ranks {q + 9 i} of a ring under the steps
// with distances 9, 27, 81.  Inside a closed group a step is a compile-time permutation of
// registers plus two adds per value; between groups the column tile goes through shared
// memory once (lane = element column, so every access is bank-conflict free).
//
//   k_lat_reg   : n <= 81 (rings 3..81, tori 3x3, 9x9, 3x3x3, 3x3x3x3): one group, no shared memory
//   k_lat_ring  : rings of 243 and 729: steps {1,3} on windows of consecutive ranks with a
//                 halo of 4, then the remaining steps on the closed sets {q + 9 i}
//   k_lat_t999  : 9x9x9 torus: steps (A,1)(B,1) on 9x9 planes, then (C,1)(A,3)(B,3)(C,3) on the
//                 3x3x9 closed sets; A,B,C = the slice's dimension order
#include "trv_dev.cuh"

namespace trv {

constexpr int ipow3(int e) { return e <= 0 ? 1 : 3 * ipow3(e - 1); }
constexpr int ipow(int b, int e) { return e <= 0 ? 1 : b * ipow(b, e - 1); }
constexpr int ilog3(int n) { return n <= 1 ? 0 : 1 + ilog3(n / 3); }

// V consecutive elements of one rank
template <typename T, int V>
struct alignas(sizeof(T) * V) Elem {
    T x[V];
};

template <typename T, int V>
__device__ __forceinline__ Elem<T, V> add3(const Elem<T, V>& a, const Elem<T, V>& b, const Elem<T, V>& c) {
    Elem<T, V> r;
#pragma unroll
    for (int k = 0; k < V; ++k) r.x[k] = add3(a.x[k], b.x[k], c.x[k]);
    return r;
}

template <typename T, int V>
__device__ __forceinline__ Elem<T, V> load_elem(const T* p, long long e, long long lo, long long hi, bool full) {
    Elem<T, V> r;
    if (full) {
        r = *reinterpret_cast<const Elem<T, V>*>(p + e);
    } else {
#pragma unroll
        for (int k = 0; k < V; ++k) r.x[k] = (e + k >= lo && e + k < hi) ? p[e + k] : T(0);
    }
    return r;
}
template <typename T, int V>
__device__ __forceinline__ void store_elem(T* p, long long e, long long lo, long long hi, bool full, const Elem<T, V>& v) {
    if (full) {
        *reinterpret_cast<Elem<T, V>*>(p + e) = v;
    } else {
#pragma unroll
        for (int k = 0; k < V; ++k)
            if (e + k >= lo && e + k < hi) p[e + k] = v.x[k];
    }
}

// One joint-reduction step on a register array: along the axis with flat stride STRIDE and ring
// length L, new[i] = (old[i - DIST] + old[i]) + old[i + DIST], indices modulo L.
template <int N, int STRIDE, int L, int DIST, typename E>
__device__ __forceinline__ void reg_step(E (&v)[N]) {
#pragma unroll
    for (int base = 0; base < N; ++base) {
        if ((base / STRIDE) % L != 0) continue;
        E line[L];
#pragma unroll
        for (int i = 0; i < L; ++i) line[i] = v[base + i * STRIDE];
#pragma unroll
        for (int i = 0; i < L; ++i) v[base + i * STRIDE] = add3(line[(i - DIST + L) % L], line[i], line[(i + DIST) % L]);
    }
}

struct LatArgs {
    int nslices;
    long long lo[TRV_MAX_DIMS], hi[TRV_MAX_DIMS];   // local element range of each slice
    int rs[TRV_MAX_DIMS][4];                        // rank stride of the slice's k-th dimension in its own order
};

// ------------------------------------------------------------------ n <= 81: registers only

// steps of an A^D torus in the slice's own dimension order: axis t % D, distance 3^(t / D)
template <int A, int D, int T0, int N, typename E>
__device__ __forceinline__ void reg_all_steps(E (&v)[N]) {
    constexpr int S = D * ilog3(A);
    if constexpr (T0 < S) {
        reg_step<N, ipow(A, T0 % D), A, ipow3(T0 / D)>(v);
        reg_all_steps<A, D, T0 + 1>(v);
    }
}

template <typename T, int A, int D, int V, int THREADS, int CAP>
__global__ void __launch_bounds__(THREADS) k_lat_reg(PtrTab<CAP> in, PtrTab<CAP> out, LatArgs a) {
    constexpr int N = ipow(A, D);
    using E = Elem<T, V>;
    const int c = blockIdx.y;
    const long long lo = a.lo[c], hi = a.hi[c];
    const long long e = ((lo / V) + (long long)blockIdx.x * THREADS + threadIdx.x) * V;
    if (e >= hi) return;
    const bool full = e >= lo && e + V <= hi;
    E v[N];
#pragma unroll
    for (int idx = 0; idx < N; ++idx) {
        int rank = 0, rem = idx;
#pragma unroll
        for (int k = 0; k < D; ++k) { rank += (rem % A) * a.rs[c][k]; rem /= A; }
        v[idx] = load_elem<T, V>((const T*)in.p[rank], e, lo, hi, full);
    }
    reg_all_steps<A, D, 0>(v);
#pragma unroll
    for (int idx = 0; idx < N; ++idx) {
        int rank = 0, rem = idx;
#pragma unroll
        for (int k = 0; k < D; ++k) { rank += (rem % A) * a.rs[c][k]; rem /= A; }
        store_elem<T, V>((T*)out.p[rank], e, lo, hi, full, v[idx]);
    }
}

// ------------------------------------------------------------------ rings of 9*M ranks, M = 27 or 81

template <int M, int T0, int N, typename E>
__device__ __forceinline__ void ring_tail_steps(E (&v)[N]) {     // distances 1, 3, .. on the ring of M
    if constexpr (T0 < ilog3(M)) {
        reg_step<N, 1, M, ipow3(T0)>(v);
        ring_tail_steps<M, T0 + 1>(v);
    }
}

template <typename T, int M, int CAP>
__global__ void __launch_bounds__(288) k_lat_ring(PtrTab<CAP> in, PtrTab<CAP> out, LatArgs a) {
    constexpr int NR = 9 * M;
    extern __shared__ uint32_t slab_raw[];
    T* slab = reinterpret_cast<T*>(slab_raw);       // [NR][32]
    const int lane = threadIdx.x & 31, set = threadIdx.x >> 5;
    const long long lo = a.lo[0], hi = a.hi[0];
    const long long e = (lo & ~31LL) + (long long)blockIdx.x * 32 + lane;
    const bool valid = e >= lo && e < hi;

    // group 1: window of M consecutive ranks [set*M, set*M + M) plus a halo of 4 on each side
    T x[M + 8];
#pragma unroll
    for (int i = 0; i < M; ++i) {
        const int r = set * M + i;
        x[4 + i] = valid ? ((const T*)in.p[r])[e] : T(0);
        slab[r * 32 + lane] = x[4 + i];
    }
    __syncthreads();
#pragma unroll
    for (int k = 0; k < 4; ++k) {
        int rl = set * M - 4 + k; if (rl < 0) rl += NR;
        int rr = set * M + M + k; if (rr >= NR) rr -= NR;
        x[k] = slab[rl * 32 + lane];
        x[M + 4 + k] = slab[rr * 32 + lane];
    }
    T y[M + 8];
#pragma unroll
    for (int i = 1; i < M + 7; ++i) y[i] = add3(x[i - 1], x[i], x[i + 1]);          // distance 1
    __syncthreads();                                                                // halos read
#pragma unroll
    for (int i = 4; i < M + 4; ++i) slab[(set * M + i - 4) * 32 + lane] = add3(y[i - 3], y[i], y[i + 3]);   // distance 3
    __syncthreads();

    // group 2: ranks {set + 9 i}: closed under the distances 9, 27, .. ; a ring of M with distances 1, 3, ..
    T v[M];
#pragma unroll
    for (int i = 0; i < M; ++i) v[i] = slab[(set + 9 * i) * 32 + lane];
    ring_tail_steps<M, 0>(v);
    if (valid) {
#pragma unroll
        for (int i = 0; i < M; ++i) ((T*)out.p[set + 9 * i])[e] = v[i];
    }
}

// ------------------------------------------------------------------ 9 x 9 x 9 torus

template <typename T, int CAP>
__global__ void __launch_bounds__(288, 2) k_lat_t999(PtrTab<CAP> in, PtrTab<CAP> out, LatArgs a) {
    extern __shared__ uint32_t slab_raw[];
    T* slab = reinterpret_cast<T*>(slab_raw);       // [729][32]
    const int c = blockIdx.y;
    const int lane = threadIdx.x & 31, set = threadIdx.x >> 5;
    const long long lo = a.lo[c], hi = a.hi[c];
    const long long e = (lo & ~31LL) + (long long)blockIdx.x * 32 + lane;
    const bool valid = e >= lo && e < hi;
    const int sA = a.rs[c][0], sB = a.rs[c][1], sC = a.rs[c][2];

    T v[81];
    // group 1: plane C = set; flat index i + 9 j  <->  rank i sA + j sB + set sC; steps (A,1), (B,1)
#pragma unroll
    for (int idx = 0; idx < 81; ++idx) {
        const int rank = (idx % 9) * sA + (idx / 9) * sB + set * sC;
        v[idx] = valid ? ((const T*)in.p[rank])[e] : T(0);
    }
    reg_step<81, 1, 9, 1>(v);
    reg_step<81, 9, 9, 1>(v);
#pragma unroll
    for (int idx = 0; idx < 81; ++idx) {
        const int rank = (idx % 9) * sA + (idx / 9) * sB + set * sC;
        slab[rank * 32 + lane] = v[idx];
    }
    __syncthreads();
    // group 2: A in {a0, a0+3, a0+6}, B in {b0, b0+3, b0+6}, all of C; flat index i + 3 j + 9 k;
    // steps (C,1), (A,3), (B,3), (C,3): in this set A and B are rings of 3 with distance 1
    const int a0 = set % 3, b0 = set / 3;
#pragma unroll
    for (int idx = 0; idx < 81; ++idx) {
        const int rank = (a0 + 3 * (idx % 3)) * sA + (b0 + 3 * ((idx / 3) % 3)) * sB + (idx / 9) * sC;
        v[idx] = slab[rank * 32 + lane];
    }
    reg_step<81, 9, 9, 1>(v);
    reg_step<81, 1, 3, 1>(v);
    reg_step<81, 3, 3, 1>(v);
    reg_step<81, 9, 9, 3>(v);
    if (valid) {
#pragma unroll
        for (int idx = 0; idx < 81; ++idx) {
            const int rank = (a0 + 3 * (idx % 3)) * sA + (b0 + 3 * ((idx / 3) % 3)) * sB + (idx / 9) * sC;
            ((T*)out.p[rank])[e] = v[idx];
        }
    }
}

// ------------------------------------------------------------------ host side

enum class LatKind { None, Reg, Ring, T999 };

static LatKind classify(const Plan& p) {
    if (p.algo != TRV_ALGO_TRIVANCE || p.variant != TRV_LATENCY_OPTIMAL || !p.equal_dims) return LatKind::None;
    if (p.n <= 81 && p.ndims <= 4) return LatKind::Reg;
    if (p.ndims == 1 && (p.n == 243 || p.n == 729)) return LatKind::Ring;
    if (p.ndims == 3 && p.dims[0] == 9) return LatKind::T999;
    return LatKind::None;
}

bool fused_latency_supported(const Plan& p) { return classify(p) != LatKind::None; }

static void fill_args(const Call& c, LatArgs* a, long long* max_len) {
    const Plan& p = *c.plan;
    a->nslices = p.ndims;
    *max_len = 0;
    for (int sl = 0; sl < p.ndims; ++sl) {
        local_slice(c, sl, &a->lo[sl], &a->hi[sl]);
        for (int k = 0; k < 4; ++k) a->rs[sl][k] = k < p.ndims ? p.stride[(sl + k) % p.ndims] : 0;
    }
}

template <typename T, int A, int D, int V, int THREADS, int CAP>
static void launch_reg(const Call& c, const PtrTab<CAP>& in, const PtrTab<CAP>& out, const LatArgs& a) {
    long long tiles = 0;
    for (int sl = 0; sl < D; ++sl)
        if (a.hi[sl] > a.lo[sl]) {
            long long t = (a.hi[sl] - (a.lo[sl] / V) * V + (long long)V * THREADS - 1) / ((long long)V * THREADS);
            if (t > tiles) tiles = t;
        }
    if (tiles == 0) return;
    dim3 grid((unsigned)tiles, D, 1);
    TRV_LAUNCH((k_lat_reg<T, A, D, V, THREADS, CAP>), grid, THREADS, 0, c.st, in, out, a);
}

template <typename T, int CAP>
static trv_status_t lat_fused_impl(const Call& c) {
    const Plan& p = *c.plan;
    PtrTab<CAP> in, out;
    for (int r = 0; r < p.n; ++r) { in.p[r] = const_cast<void*>(c.in[r]); out.p[r] = c.out[r]; }
    LatArgs a;
    long long unused;
    fill_args(c, &a, &unused);
    const LatKind kind = classify(p);
    if (kind == LatKind::Reg) {
        const int A = p.dims[0], D = p.ndims;
        if constexpr (CAP == 32) {
            if (A == 3 && D == 1) { g_last_kernel = "lat_reg<3>"; launch_reg<T, 3, 1, 4, 128>(c, in, out, a); }
            else if (A == 9 && D == 1) { g_last_kernel = "lat_reg<9>"; launch_reg<T, 9, 1, 4, 128>(c, in, out, a); }
            else if (A == 27 && D == 1) { g_last_kernel = "lat_reg<27>"; launch_reg<T, 27, 1, 4, 128>(c, in, out, a); }
            else if (A == 3 && D == 2) { g_last_kernel = "lat_reg<3x3>"; launch_reg<T, 3, 2, 4, 128>(c, in, out, a); }
            else if (A == 3 && D == 3) { g_last_kernel = "lat_reg<3x3x3>"; launch_reg<T, 3, 3, 4, 128>(c, in, out, a); }
            else return TRV_ERR_UNSUPPORTED;
        } else if constexpr (CAP == 256) {
            if (A == 81 && D == 1) { g_last_kernel = "lat_reg<81>"; launch_reg<T, 81, 1, 1, 128>(c, in, out, a); }
            else if (A == 9 && D == 2) { g_last_kernel = "lat_reg<9x9>"; launch_reg<T, 9, 2, 1, 128>(c, in, out, a); }
            else if (A == 3 && D == 4) { g_last_kernel = "lat_reg<3x3x3x3>"; launch_reg<T, 3, 4, 1, 128>(c, in, out, a); }
            else return TRV_ERR_UNSUPPORTED;
        } else {
            return TRV_ERR_UNSUPPORTED;
        }
    } else if (kind == LatKind::Ring) {
        if (a.hi[0] > a.lo[0]) {
            const long long tiles = (a.hi[0] - (a.lo[0] & ~31LL) + 31) / 32;
            if (p.n == 243) {
                if constexpr (CAP == 256) {
                    g_last_kernel = "lat_ring<243>";
                    TRV_LAUNCH((k_lat_ring<T, 27, CAP>), dim3((unsigned)tiles), 288, 243 * 32 * 4, c.st, in, out, a);
                }
            } else {
                if constexpr (CAP == TRV_MAX_RANKS) {
                    g_last_kernel = "lat_ring<729>";
                    static bool attr_done[2] = {false, false};
                    auto kfn = k_lat_ring<T, 81, CAP>;
                    if (!attr_done[sizeof(T) == 4 && std::is_same<T, float>::value]) {
                        cudaFuncSetAttribute(kfn, cudaFuncAttributeMaxDynamicSharedMemorySize, 729 * 32 * 4);
                        attr_done[std::is_same<T, float>::value] = true;
                    }
                    TRV_LAUNCH(kfn, dim3((unsigned)tiles), 288, 729 * 32 * 4, c.st, in, out, a);
                }
            }
        }
    } else if (kind == LatKind::T999) {
        if constexpr (CAP == TRV_MAX_RANKS) {
            g_last_kernel = "lat_t999";
            long long tiles = 0;
            for (int sl = 0; sl < 3; ++sl)
                if (a.hi[sl] > a.lo[sl]) {
                    long long t = (a.hi[sl] - (a.lo[sl] & ~31LL) + 31) / 32;
                    if (t > tiles) tiles = t;
                }
            if (tiles > 0) {
                auto kfn = k_lat_t999<T, CAP>;
                static bool attr_done[2] = {false, false};
                if (!attr_done[std::is_same<T, float>::value]) {
                    cudaFuncSetAttribute(kfn, cudaFuncAttributeMaxDynamicSharedMemorySize, 729 * 32 * 4);
                    attr_done[std::is_same<T, float>::value] = true;
                }
                TRV_LAUNCH(kfn, dim3((unsigned)tiles, 3, 1), 288, 729 * 32 * 4, c.st, in, out, a);
            }
        }
    } else {
        return TRV_ERR_UNSUPPORTED;
    }
    return cudaGetLastError() == cudaSuccess ? TRV_OK : TRV_ERR_CUDA;
}

trv_status_t run_fused_latency(const Call& c) {
    const int n = c.plan->n;
    if (c.dtype == TRV_FLOAT32) {
        if (n <= 32) return lat_fused_impl<float, 32>(c);
        if (n <= 256) return lat_fused_impl<float, 256>(c);
        return lat_fused_impl<float, TRV_MAX_RANKS>(c);
    }
    if (n <= 32) return lat_fused_impl<uint32_t, 32>(c);
    if (n <= 256) return lat_fused_impl<uint32_t, 256>(c);
    return lat_fused_impl<uint32_t, TRV_MAX_RANKS>(c);
}

}  // namespace trv
