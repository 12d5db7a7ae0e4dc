// FUSED kernels of the latency-optimal form (Sec. 4.2): all log3 n joint-reduction steps of a
// column of elements run on chip, so every element is read from HBM once and written once.
//
// Every rank has its own reduction tree (the n results differ in rounding), so the work is
// 2*S*n adds per element column and cannot be shared between ranks.  The kernels keep whole
// "closed groups" of ranks in registers: a set of ranks is closed under a group of steps if
// every step maps the set onto itself, e.g. the ranks {q + 9 i} of a ring under the steps
// with distances 9, 27, 81.  Inside a closed group a step is a compile-time permutation of
// registers plus two adds per value; between groups the column tile goes through shared
// memory once.  A thread owns V adjacent columns, so float adds issue as packed f32x2.
//
//   k_lat_reg   : n <= 81 (rings 3..81, tori 3x3, 9x9, 3x3x3, 3x3x3x3): one group, no shared memory
//   k_lat_ring  : rings of 243 and 729: steps {1,3} on windows of consecutive ranks with a
//                 halo of 4, then the remaining steps on the closed sets {q + 9 i}
//   k_lat_t999 (trv_fused_t999.cu): 9x9x9 torus, three closed groups of two steps each
#include <type_traits>

#include "trv_dev.cuh"
#include "trv_fused_lat.cuh"

namespace trv {

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

// Tiles start on multiples of 32*V elements of the buffers (128*V bytes) so that a warp's
// access to one rank is one aligned, contiguous run.
template <typename T, int A, int D, int V, bool FULL, typename Addr>
__device__ __forceinline__ void lat_reg_body(const Addr& in, const Addr& out, const LatArgs& a, int c, long long e) {
    constexpr int N = ipow(A, D);
    using E = Elem<T, V>;
    const long long lo = a.lo[c], hi = a.hi[c];
    E v[N];
#pragma unroll
    for (int idx = 0; idx < N; ++idx) {
        int rank = 0, rem = idx;
#pragma unroll
        for (int k = 0; k < D; ++k) { rank += (rem % A) * a.rs[c][k]; rem /= A; }
        v[idx] = load_elem<T, V, FULL>(in.ptr(rank), e, lo, hi);
    }
    reg_all_steps<A, D, 0>(v);
#pragma unroll
    for (int idx = 0; idx < N; ++idx) {
        int rank = 0, rem = idx;
#pragma unroll
        for (int k = 0; k < D; ++k) { rank += (rem % A) * a.rs[c][k]; rem /= A; }
        store_elem<T, V, FULL>(out.ptr(rank), e, lo, hi, v[idx]);
    }
}

template <typename T, int A, int D, int V, int THREADS, typename Addr>
__global__ void __launch_bounds__(THREADS) k_lat_reg(Addr in, Addr out, LatArgs a) {
    pdl_trigger();
    const int c = blockIdx.y;
    const long long lo = a.lo[c], hi = a.hi[c];
    const long long t0 = (lo / (32 * V)) * (32 * V) + (long long)blockIdx.x * THREADS * V;    // first column of the tile
    pdl_wait();
    const long long e = t0 + (long long)threadIdx.x * V;
    if (t0 >= lo && t0 + (long long)THREADS * V <= hi) {
        lat_reg_body<T, A, D, V, true>(in, out, a, c, e);
    } else if (e < hi && e + V > lo) {
        lat_reg_body<T, A, D, V, false>(in, out, a, c, e);
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

// Tiles of TILE columns (32, or 64 for long vectors on the ring of 243); a thread owns V adjacent columns of one of 9
// rank sets: 9 * TILE / V threads.
template <typename T, int M, int V, int TILE, bool FULL, typename Addr>
__device__ __forceinline__ void lat_ring_body(const Addr& in, const Addr& out, const LatArgs& a, T* slab, long long t0) {
    constexpr int NR = 9 * M, LANES = TILE / V;
    using E = Elem<T, V>;
    const int lane = threadIdx.x % LANES, set = threadIdx.x / LANES;
    const long long lo = a.lo[0], hi = a.hi[0];
    const long long e = t0 + lane * V;
    auto sl = [&](int r) -> E& { return *reinterpret_cast<E*>(slab + r * TILE + lane * V); };

    // group 1: window of M consecutive ranks [set*M, set*M + M) plus a halo of 4 on each side
    E x[M + 8];
#pragma unroll
    for (int i = 0; i < M; ++i) x[4 + i] = load_elem<T, V, FULL>(in.ptr(set * M + i), e, lo, hi);
#pragma unroll
    for (int i = 0; i < M; ++i) sl(set * M + i) = x[4 + i];
    __syncthreads();
#pragma unroll
    for (int k = 0; k < 4; ++k) {
        int rl = set * M - 4 + k; if (rl < 0) rl += NR;
        int rr = set * M + M + k; if (rr >= NR) rr -= NR;
        x[k] = sl(rl);
        x[M + 4 + k] = sl(rr);
    }
    E y[M + 8];
#pragma unroll
    for (int i = 1; i < M + 7; ++i) y[i] = add3(x[i - 1], x[i], x[i + 1]);          // distance 1
    __syncthreads();                                                                // halos read
#pragma unroll
    for (int i = 4; i < M + 4; ++i) sl(set * M + i - 4) = add3(y[i - 3], y[i], y[i + 3]);   // distance 3
    __syncthreads();

    // group 2: ranks {set + 9 i}: closed under the distances 9, 27, .. ; a ring of M with distances 1, 3, ..
    E v[M];
#pragma unroll
    for (int i = 0; i < M; ++i) v[i] = sl(set + 9 * i);
    ring_tail_steps<M, 0>(v);
    if (FULL || (e < hi && e + V > lo)) {
#pragma unroll
        for (int i = 0; i < M; ++i) store_elem<T, V, FULL>(out.ptr(set + 9 * i), e, lo, hi, v[i]);
    }
}

template <typename T, int M, int V, int TILE, typename Addr>
__global__ void __launch_bounds__(9 * TILE / V, M == 27 ? (TILE == 64 ? 3 : 4) : 1) k_lat_ring(Addr in, Addr out, LatArgs a) {
    pdl_trigger();
    extern __shared__ uint4 slab_raw[];
    T* slab = reinterpret_cast<T*>(slab_raw);       // [9 M][TILE]
    const long long t0 = (a.lo[0] & ~(long long)(TILE - 1)) + (long long)blockIdx.x * TILE;
    pdl_wait();
    if (t0 >= a.lo[0] && t0 + TILE <= a.hi[0]) lat_ring_body<T, M, V, TILE, true>(in, out, a, slab, t0);   // CTA-uniform
    else lat_ring_body<T, M, V, TILE, false>(in, out, a, slab, t0);
}

// ------------------------------------------------------------------ host side

enum class LatKind { None, Reg, Ring, T999, Lines };

static LatKind classify(const Plan& p) {
    if (p.lat_kind >= 0) return (LatKind)p.lat_kind;        // decided when the plan was created
    if (p.algo != TRV_ALGO_TRIVANCE || p.variant != TRV_LATENCY_OPTIMAL) return LatKind::None;
    if (p.equal_dims) {
        if (p.n <= 81 && p.ndims <= 4) return LatKind::Reg;
        if (p.ndims == 1 && (p.n == 243 || p.n == 729)) return LatKind::Ring;
        if (p.ndims == 3 && p.dims[0] == 9) return LatKind::T999;
    }
    return fused_lines_supported(p) ? LatKind::Lines : LatKind::None;     // 27x27, unequal sides, ...
}

bool fused_latency_supported(const Plan& p) { return classify(p) != LatKind::None; }

// once per plan (prepare_launch_data)
void latency_prepare(Plan& p) {
    p.lat_kind = -1;
    const LatKind k = classify(p);
    if (k == LatKind::Lines) lines_prepare(p);
    p.lat_kind = (int)k;
}

static void fill_args(const Call& c, LatArgs* a) {
    const Plan& p = *c.plan;
    a->nslices = p.ndims;
    for (int sl = 0; sl < p.ndims; ++sl) {
        local_slice(c, sl, &a->lo[sl], &a->hi[sl]);
        for (int k = 0; k < 4; ++k) a->rs[sl][k] = k < p.ndims ? p.stride[(sl + k) % p.ndims] : 0;
    }
}

// number of tiles of `tile` elements, starting at a multiple of `align`, that cover the longest slice
static long long tiles_for(const LatArgs& a, int nslices, long long tile, long long align) {
    long long tiles = 0;
    for (int sl = 0; sl < nslices; ++sl)
        if (a.hi[sl] > a.lo[sl]) {
            const long long t = (a.hi[sl] - (a.lo[sl] / align) * align + tile - 1) / tile;
            if (t > tiles) tiles = t;
        }
    return tiles;
}

template <typename T, int A, int D, int V, int THREADS, typename Addr>
static void launch_reg(const Call& c, const Addr& in, const Addr& out, const LatArgs& a) {
    const long long tiles = tiles_for(a, D, (long long)V * THREADS, 32 * V);
    if (tiles == 0) return;
    launch_pdl(k_lat_reg<T, A, D, V, THREADS, Addr>, dim3((unsigned)tiles, D, 1), dim3(THREADS), 0, c.st, in, out, a);
}

template <typename T, typename Addr>
static trv_status_t lat_fused_launch(const Call& c, const Addr& in, const Addr& out) {
    const Plan& p = *c.plan;
    LatArgs a;
    fill_args(c, &a);
    const LatKind kind = classify(p);
    if (kind == LatKind::Reg) {
        const int A = p.dims[0], D = p.ndims;
        if (A == 3 && D == 1) { g_last_kernel = "lat_reg<3>"; launch_reg<T, 3, 1, 4, 64>(c, in, out, a); }
        else if (A == 9 && D == 1) { g_last_kernel = "lat_reg<9>"; launch_reg<T, 9, 1, 4, 64>(c, in, out, a); }
        else if (A == 27 && D == 1) { g_last_kernel = "lat_reg<27>"; launch_reg<T, 27, 1, 2, 128>(c, in, out, a); }
        else if (A == 3 && D == 2) { g_last_kernel = "lat_reg<3x3>"; launch_reg<T, 3, 2, 4, 64>(c, in, out, a); }
        else if (A == 3 && D == 3) { g_last_kernel = "lat_reg<3x3x3>"; launch_reg<T, 3, 3, 4, 64>(c, in, out, a); }
        else if (A == 81 && D == 1) { g_last_kernel = "lat_reg<81>"; launch_reg<T, 81, 1, 2, 64>(c, in, out, a); }
        else if (A == 9 && D == 2) { g_last_kernel = "lat_reg<9x9>"; launch_reg<T, 9, 2, 2, 64>(c, in, out, a); }
        else if (A == 3 && D == 4) { g_last_kernel = "lat_reg<3x3x3x3>"; launch_reg<T, 3, 4, 2, 64>(c, in, out, a); }
        else return TRV_ERR_UNSUPPORTED;
    } else if (kind == LatKind::Ring) {
        if (p.n == 729) {               // long vectors, equally spaced rank buffers: the persistent 64-column kernel
            trv_status_t st = TRV_OK;
            if (run_fused_r729_wide(c, a, &st)) return st;
        }
        // Ring of 243, long vectors: tiles of 64 columns (256 bytes per rank and tile), three CTAs per SM (72 registers).
        // Every tile touches all 243 input and all 243 output rows, and the 32-column kernel loses bandwidth as the rows
        // get longer (0.93 of the copy bandwidth at 2 MiB per rank, 0.85 at 8 MiB, 0.83 at 32 MiB) while the 64-column
        // one holds 0.93 - 0.94 (8 MiB: 730 -> 664 us, 32 MiB: 3013 -> 2648 us).  Up to 2 MiB per rank the two are
        // within a percent of each other; the 32-column kernel (four CTAs per SM, 96 registers) keeps the short vectors.
        if (p.n == 243 && a.hi[0] - a.lo[0] >= (1LL << 20)) {
            const long long tiles = tiles_for(a, 1, 64, 64);
            g_last_kernel = "lat_ring<243,64>";
            auto kfn = k_lat_ring<T, 27, 2, 64, Addr>;
            if (!allow_big_smem(kfn, 243 * 64 * 4)) return TRV_ERR_CUDA;
            launch_pdl(kfn, dim3((unsigned)tiles), dim3(288), 243 * 64 * 4, c.st, in, out, a);
        } else {
            const long long tiles = tiles_for(a, 1, 32, 32);
            if (tiles > 0) {
                if (p.n == 243) {
                    g_last_kernel = "lat_ring<243>";
                    launch_pdl(k_lat_ring<T, 27, 2, 32, Addr>, dim3((unsigned)tiles), dim3(144), 243 * 32 * 4, c.st, in, out, a);
                } else {
                    g_last_kernel = "lat_ring<729>";
                    auto kfn = k_lat_ring<T, 81, 1, 32, Addr>;
                    if (!allow_big_smem(kfn, 729 * 32 * 4)) return TRV_ERR_CUDA;
                    launch_pdl(kfn, dim3((unsigned)tiles), dim3(288), 729 * 32 * 4, c.st, in, out, a);
                }
            }
        }
    } else if (kind == LatKind::T999) {
        // equally spaced rank buffers: the tile arrives by TMA; else per-thread loads
        trv_status_t st = TRV_OK;
        if (run_fused_t999_wide(c, a, &st)) return st;
        if (run_fused_t999_tma(c, a, &st)) return st;
        g_last_kernel = "lat_t999";
        return run_fused_t999(c, a);
    } else if (kind == LatKind::Lines) {
        trv_status_t st = TRV_OK;
        if (run_fused_t2727_wide(c, a, &st)) return st;       // 27 x 27, long vectors, equally spaced rank buffers
        if (run_fused_t981_wide(c, a, &st)) return st;        // 9 x 81, likewise
        g_last_kernel = "lat_lines";
        return run_fused_lines(c, a);
    } else {
        return TRV_ERR_UNSUPPORTED;
    }
    return cudaGetLastError() == cudaSuccess ? TRV_OK : TRV_ERR_CUDA;
}

template <typename T>
static trv_status_t lat_fused_addr(const Call& c) {
    const int n = c.plan->n;
    StrideAddr sin, sout;
    if (uniform_stride(c.in, n, &sin) && uniform_stride((const void* const*)c.out, n, &sout))
        return lat_fused_launch<T, StrideAddr>(c, sin, sout);
    if (n <= 81) {      // k_lat_reg shapes
        TabAddr<81> in, out;
        for (int r = 0; r < n; ++r) { in.t.p[r] = const_cast<void*>(c.in[r]); out.t.p[r] = c.out[r]; }
        return lat_fused_launch<T, TabAddr<81>>(c, in, out);
    }
    TabAddr<729> in, out;
    for (int r = 0; r < n; ++r) { in.t.p[r] = const_cast<void*>(c.in[r]); out.t.p[r] = c.out[r]; }
    return lat_fused_launch<T, TabAddr<729>>(c, in, out);
}

trv_status_t run_fused_latency(const Call& c) {
    return c.dtype == TRV_FLOAT32 ? lat_fused_addr<float>(c) : lat_fused_addr<uint32_t>(c);
}

}  // namespace trv
