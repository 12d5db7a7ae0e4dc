// FUSED latency-optimal kernel for the 9 x 9 x 9 torus (Sec. 4.2, Sec. 5).
//
// A tile is 32 element columns x 729 ranks (93 KB of shared memory, two CTAs per SM).  A, B, C are
// the slice's dimensions in its own order (Sec. 5: collective c starts on dimension c); their rank
// strides are compile-time (ROT = slice number), so every rank offset inside a closed set is an
// immediate.  The six steps of a slice run as three groups of two, each on sets of ranks closed
// under its steps:
//   group 1: (A,1) (B,1) on the 9x9 plane C = set, streamed row by row (row = 9 values along A):
//            (A,1) inside a row, (B,1) over a sliding window of three rows
//   group 2: (C,1) (A,3) on the sets {A in a0+3i, B = j, all C}            (27 values, 3 sets per thread)
//   group 3: (B,3) (C,3) on the sets {A = i, B in b0+3j, C in c0+3k}        (9 values, 9 sets per thread)
// Between groups the tile stays in shared memory; inside a group every set is read and written by
// one thread only, so the two barriers between the groups are the only synchronisation.
// A thread owns V adjacent columns (V = 1: 288 threads; V = 2: packed adds, 144 threads) of one
// ninth of the sets.  Measured on B200 (729 x 32 MiB): V = 1 9.96 ms, V = 2 10.8 ms; staging the
// plane with asynchronous global->shared copies, two groups with an 81-value register set,
// persistent and warp-specialised variants were all slower (10.8 - 14 ms): what counts is the
// number of warps that have loads in flight, not the instruction count.  With 288 threads the
// register file allows two CTAs per SM only up to 96 registers per thread.
#include "trv_dev.cuh"
#include "trv_fused_lat.cuh"

namespace trv {

template <int ROT>
struct Rot {
    static constexpr int sA = ROT == 0 ? 1 : (ROT == 1 ? 9 : 81);
    static constexpr int sB = ROT == 0 ? 9 : (ROT == 1 ? 81 : 1);
    static constexpr int sC = ROT == 0 ? 81 : (ROT == 1 ? 1 : 9);
};

template <typename T, int ROT, int V, bool FULL, typename Addr>
__device__ __forceinline__ void t999_body(const Addr& in, const Addr& out, const LatArgs& a, T* slab, long long t0) {
    using R = Rot<ROT>;
    using E = Elem<T, V>;
    constexpr int LANES = 32 / V;
    const int lane = threadIdx.x % LANES, set = threadIdx.x / LANES;
    const long long lo = a.lo[ROT], hi = a.hi[ROT];
    const long long e = t0 + lane * V;
    T* const mine = slab + lane * V;
    auto sl = [&](int r) -> E& { return *reinterpret_cast<E*>(mine + r * 32); };
    {   // ---- group 1: (A,1) (B,1) on the plane C = set
        const int r0 = set * R::sC;
        auto load_row = [&](int j, E (&row)[9]) {
#pragma unroll
            for (int i = 0; i < 9; ++i) row[i] = load_elem<T, V, FULL>(in.ptr(r0 + i * R::sA + j * R::sB), e, lo, hi);
            reg_step<9, 1, 9, 1>(row);                                      // (A,1)
        };
        auto emit = [&](int j, const E (&p)[9], const E (&q)[9], const E (&r)[9]) {     // (B,1) for row j
#pragma unroll
            for (int i = 0; i < 9; ++i) sl(r0 + i * R::sA + j * R::sB) = add3(p[i], q[i], r[i]);
        };
        E first[9], second[9], prev[9], cur[9], next[9];
        load_row(0, first);
        load_row(1, second);
#pragma unroll
        for (int i = 0; i < 9; ++i) { prev[i] = first[i]; cur[i] = second[i]; }
#pragma unroll
        for (int j = 1; j < 8; ++j) {
            load_row(j + 1, next);
            emit(j, prev, cur, next);
#pragma unroll
            for (int i = 0; i < 9; ++i) { prev[i] = cur[i]; cur[i] = next[i]; }
        }
        emit(8, prev, cur, first);      // row 8 needs rows 7, 8, 0
        emit(0, cur, first, second);    // row 0 needs rows 8, 0, 1
    }
    __syncthreads();
    // ---- group 2: (C,1) (A,3); flat index k + 9 i  <->  rank (a0 + 3 i) sA + j sB + k sC
#pragma unroll 1
    for (int m = 0; m < 3; ++m) {
        const int q = set + 9 * m, r0 = (q % 3) * R::sA + (q / 3) * R::sB;
        E v[27];
#pragma unroll
        for (int idx = 0; idx < 27; ++idx) v[idx] = sl(r0 + 3 * (idx / 9) * R::sA + (idx % 9) * R::sC);
        reg_step<27, 1, 9, 1>(v);       // (C,1)
        reg_step<27, 9, 3, 1>(v);       // (A,3): inside this set a ring of three with distance one
#pragma unroll
        for (int idx = 0; idx < 27; ++idx) sl(r0 + 3 * (idx / 9) * R::sA + (idx % 9) * R::sC) = v[idx];
    }
    __syncthreads();
    // ---- group 3: (B,3) (C,3); flat index jj + 3 kk  <->  rank i sA + (b0 + 3 jj) sB + (c0 + 3 kk) sC
    const bool any = FULL || (e < hi && e + V > lo);
#pragma unroll 1
    for (int m = 0; m < 9; ++m) {
        const int q = set + 9 * m, r0 = (q % 9) * R::sA + ((q / 9) % 3) * R::sB + (q / 27) * R::sC;
        E v[9];
#pragma unroll
        for (int idx = 0; idx < 9; ++idx) v[idx] = sl(r0 + 3 * (idx % 3) * R::sB + 3 * (idx / 3) * R::sC);
        reg_step<9, 1, 3, 1>(v);        // (B,3)
        reg_step<9, 3, 3, 1>(v);        // (C,3)
        if (any) {
#pragma unroll
            for (int idx = 0; idx < 9; ++idx)
                store_elem<T, V, FULL>(out.ptr(r0 + 3 * (idx % 3) * R::sB + 3 * (idx / 3) * R::sC), e, lo, hi, v[idx]);
        }
    }
}

template <typename T, int V, typename Addr>
__global__ void __launch_bounds__(288 / V, 2) k_lat_t999(Addr in, Addr out, LatArgs a) {
    pdl_trigger();
    extern __shared__ uint4 slab_raw[];
    T* slab = reinterpret_cast<T*>(slab_raw);       // [729][32]
    const int c = blockIdx.y;                       // everything below is CTA-uniform
    const long long t0 = (a.lo[c] & ~31LL) + (long long)blockIdx.x * 32;
    if (t0 >= a.hi[c]) return;
    pdl_wait();
    const bool full = t0 >= a.lo[c] && t0 + 32 <= a.hi[c];
    if (c == 0) { if (full) t999_body<T, 0, V, true>(in, out, a, slab, t0); else t999_body<T, 0, V, false>(in, out, a, slab, t0); }
    else if (c == 1) { if (full) t999_body<T, 1, V, true>(in, out, a, slab, t0); else t999_body<T, 1, V, false>(in, out, a, slab, t0); }
    else { if (full) t999_body<T, 2, V, true>(in, out, a, slab, t0); else t999_body<T, 2, V, false>(in, out, a, slab, t0); }
}

template <typename T, int V, typename Addr>
static trv_status_t launch_t999_v(const Call& c, const Addr& in, const Addr& out, const LatArgs& a, long long tiles_x) {
    auto kfn = k_lat_t999<T, V, Addr>;
    constexpr size_t smem = 729 * 32 * sizeof(T);
    if (!allow_big_smem(kfn, (int)smem)) return TRV_ERR_CUDA;
    launch_pdl(kfn, dim3((unsigned)tiles_x, 3, 1), dim3(288 / V), smem, c.st, in, out, a);
    return TRV_OK;
}

template <typename T, typename Addr>
static trv_status_t launch_t999(const Call& c, const Addr& in, const Addr& out, const LatArgs& a) {
    long long tiles_x = 0;
    for (int sl = 0; sl < 3; ++sl)
        if (a.hi[sl] > a.lo[sl]) {
            const long long t = (a.hi[sl] - (a.lo[sl] & ~31LL) + 31) / 32;
            if (t > tiles_x) tiles_x = t;
        }
    if (tiles_x == 0) return TRV_OK;
    if (tiles_x > (1LL << 30)) return TRV_ERR_UNSUPPORTED;
    // One column per thread and direct loads measured fastest on B200: 18 warps per SM matter more
    // than packed adds or asynchronous staging here.
    return launch_t999_v<T, 1>(c, in, out, a, tiles_x);
}

trv_status_t run_fused_t999(const Call& c, const LatArgs& a) {
    const int n = c.plan->n;
    StrideAddr sin, sout;
    const bool strided = uniform_stride(c.in, n, &sin) && uniform_stride((const void* const*)c.out, n, &sout);
    trv_status_t st;
    if (strided) {
        st = c.dtype == TRV_FLOAT32 ? launch_t999<float>(c, sin, sout, a) : launch_t999<uint32_t>(c, sin, sout, a);
    } else {
        TabAddr<729> in, out;
        for (int r = 0; r < n; ++r) { in.t.p[r] = const_cast<void*>(c.in[r]); out.t.p[r] = c.out[r]; }
        st = c.dtype == TRV_FLOAT32 ? launch_t999<float>(c, in, out, a) : launch_t999<uint32_t>(c, in, out, a);
    }
    if (st != TRV_OK) return st;
    return cudaGetLastError() == cudaSuccess ? TRV_OK : TRV_ERR_CUDA;
}

}  // namespace trv
