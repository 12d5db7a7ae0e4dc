// FUSED kernel of the bandwidth-optimal form (Sec. 4.1): Reduce-Scatter + AllGather in one pass.
//
// The Reduce-Scatter phase follows the same communication pattern as the latency-optimal form
// (Sec. 4.2) and only restricts every message to the blocks of the closed-form set Pi
// (Sec. 4.3).  The partial of block j that rank q holds after step t is therefore the
// latency-form partial of rank q after step t, restricted to block j; the owner j ends with
//      T_S(j),   T_t(p) = (T_{t-1}(p - dist_t) + T_{t-1}(p)) + T_{t-1}(p + dist_t),   T_0(p) = input of p,
// and the AllGather copies that value to every rank.  T_S(j) is a balanced ternary tree whose
// 3^S leaves, read left to right, are the ranks j + sum_t eps_t dist_t with the digit of the
// LAST step most significant and eps = -1, 0, +1 in that order.  A thread streams the n inputs
// of its element column(s) in exactly that order, nine at a time, through an S-level carry
// stack (n - 1 adds, the association of the schedule), then writes the value to all n ranks:
// n*count elements read once, n*count written once, no shared-memory staging of data.
#include "trv_dev.cuh"

namespace trv {

constexpr int kBwThreads = 128;
constexpr int kBwMaxD = 4;
constexpr int kBwMaxS = 6;

struct BwArgs {
    int n;
    long long w0;                               // global index of local element 0
    long long lo[kBwMaxD], hi[kBwMaxD];         // local element range of each slice
    long long glo[kBwMaxD], ghi[kBwMaxD];       // global element range of each slice
    int dims[kBwMaxD], dstride[kBwMaxD];
    int ldim[kBwMaxD][kBwMaxS], ldist[kBwMaxD][kBwMaxS];   // per slice, per step: dimension, distance
};

__device__ __forceinline__ int wrap(int x, int a) { return x < 0 ? x + a : (x >= a ? x - a : x); }

// rank -> buffer start: a pointer table staged in shared memory, or base + rank * stride
template <typename T>
struct SmemTabs {
    const T* const* sin;
    T* const* sout;
    __device__ __forceinline__ const T* in(int r) const { return sin[r]; }
    __device__ __forceinline__ T* out(int r) const { return sout[r]; }
};
template <typename T>
struct StrideTabs {
    StrideAddr i, o;
    __device__ __forceinline__ const T* in(int r) const { return reinterpret_cast<const T*>(i.ptr(r)); }
    __device__ __forceinline__ T* out(int r) const { return reinterpret_cast<T*>(o.ptr(r)); }
};

// Value of block owner j for the V columns starting at local element e, written to all ranks.
template <typename T, int V, int S, int D, typename Tabs>
__device__ __forceinline__ void column_tree(const BwArgs& a, int c, const Tabs& tabs, long long e, int j) {
    using P = Elem<T, V>;
    int base[D];    // coordinates of the centre of the current nine-leaf chunk
#pragma unroll
    for (int d = 0; d < D; ++d) base[d] = (j / a.dstride[d]) % a.dims[d];
    P res;
    if constexpr (S == 1) {
        const int d0 = a.ldim[c][0], x0 = a.ldist[c][0];
        int bd = 0, ad = 1, sd = 1;
#pragma unroll
        for (int d = 0; d < D; ++d) if (d == d0) { bd = base[d]; ad = a.dims[d]; sd = a.dstride[d]; }
        const P l = *reinterpret_cast<const P*>(tabs.in(j + (wrap(bd - x0, ad) - bd) * sd) + e);
        const P m = *reinterpret_cast<const P*>(tabs.in(j) + e);
        const P r = *reinterpret_cast<const P*>(tabs.in(j + (wrap(bd + x0, ad) - bd) * sd) + e);
        res = add3(l, m, r);
    } else {
        // start at the leftmost chunk: every step >= 2 at eps = -1
#pragma unroll
        for (int t = 2; t < S; ++t) {
            const int dt = a.ldim[c][t], xt = a.ldist[c][t];
#pragma unroll
            for (int d = 0; d < D; ++d) if (d == dt) base[d] = wrap(base[d] - xt, a.dims[d]);
        }
        const int d0 = a.ldim[c][0], x0 = a.ldist[c][0], d1 = a.ldim[c][1], x1 = a.ldist[c][1];
        // the nine leaves of the chunk centred at base[]: leaf m <-> (eps_1, eps_0) = (m / 3 - 1, m % 3 - 1)
        auto load_chunk = [&](P (&l)[9]) {
            int rank_c = 0, b0 = 0, a0 = 1, s0 = 1, b1 = 0, a1 = 1, s1 = 1;
#pragma unroll
            for (int d = 0; d < D; ++d) {
                rank_c += base[d] * a.dstride[d];
                if (d == d0) { b0 = base[d]; a0 = a.dims[d]; s0 = a.dstride[d]; }
                if (d == d1) { b1 = base[d]; a1 = a.dims[d]; s1 = a.dstride[d]; }
            }
            int rk[9];
            if (d0 != d1) {
                int X0[3], X1[3];
#pragma unroll
                for (int q = 0; q < 3; ++q) {
                    X0[q] = (wrap(b0 + (q - 1) * x0, a0) - b0) * s0;
                    X1[q] = (wrap(b1 + (q - 1) * x1, a1) - b1) * s1;
                }
#pragma unroll
                for (int m = 0; m < 9; ++m) rk[m] = rank_c + X1[m / 3] + X0[m % 3];
            } else {
#pragma unroll
                for (int m = 0; m < 9; ++m) rk[m] = rank_c + (wrap(b0 + (m / 3 - 1) * x1 + (m % 3 - 1) * x0, a0) - b0) * s0;
            }
#pragma unroll
            for (int m = 0; m < 9; ++m) l[m] = *reinterpret_cast<const P*>(tabs.in(rk[m]) + e);
        };
        int pd[S], vd[S];   // position / value digit (child number) of each level >= 2
        P acc[S];
#pragma unroll
        for (int t = 0; t < S; ++t) { pd[t] = 0; vd[t] = 0; }
        constexpr int CHUNKS = (S == 2) ? 1 : (S == 3 ? 3 : (S == 4 ? 9 : (S == 5 ? 27 : 81)));
        P nxt[9];
        load_chunk(nxt);
        for (int ch = 0; ch < CHUNKS; ++ch) {
            P l[9];
#pragma unroll
            for (int m = 0; m < 9; ++m) l[m] = nxt[m];
            // move to the next chunk and start its loads before reducing this one
            bool go = true;
#pragma unroll
            for (int t = 2; t < S; ++t) {
                if (go) {
                    const int dt = a.ldim[c][t], xt = a.ldist[c][t];
                    int delta;
                    if (pd[t] < 2) { pd[t]++; delta = xt; go = false; }
                    else { pd[t] = 0; delta = -2 * xt; }
#pragma unroll
                    for (int d = 0; d < D; ++d) if (d == dt) base[d] = wrap(base[d] + delta, a.dims[d]);
                }
            }
            if (ch + 1 < CHUNKS) load_chunk(nxt);
            P r = add3(add3(l[0], l[1], l[2]), add3(l[3], l[4], l[5]), add3(l[6], l[7], l[8]));
            // carry the finished 9-leaf subtree up the tree: (first + second) + third at every level
            bool carry = true;
#pragma unroll
            for (int t = 2; t < S; ++t) {
                if (carry) {
                    if (vd[t] == 0) { acc[t] = r; vd[t] = 1; carry = false; }
                    else if (vd[t] == 1) { acc[t] = add2(acc[t], r); vd[t] = 2; carry = false; }
                    else { r = add2(acc[t], r); vd[t] = 0; }
                }
            }
            res = r;    // after the last chunk the carry has run through every level
        }
    }
    // AllGather: the owner's value goes to every rank
#pragma unroll 9
    for (int r = 0; r < a.n; ++r) *reinterpret_cast<P*>(tabs.out(r) + e) = res;
}

// Short vectors: too few columns to fill the GPU with one thread per column, and a thread walking
// all n leaves needs n / 9 dependent memory round trips.  Here G = 3^(S-L) threads share a column:
// thread g reduces the g-th subtree of 3^L leaves (one round of independent loads), the G subtree
// values are combined in tree order through shared memory (S - L rounds of (first + second) +
// third over neighbours at distance 1, 3, 9), and every thread stores the result to n / G ranks.
// Block = 32 columns x G threads; a warp reads 128 contiguous bytes of one rank.
constexpr int coop_L(int S) { return S >= 5 ? 3 : 2; }
constexpr int coop_G(int S) { return S == 6 ? 27 : (S == 5 ? 9 : (S == 4 ? 9 : 3)); }

template <typename T, int S, int D, typename Tabs>
__device__ __forceinline__ void bw_coop_tile(const BwArgs& a, const Tabs& tabs, T* xch) {
    constexpr int L = coop_L(S), G = coop_G(S), LEAVES = (L == 3 ? 27 : 9);
    const int lane = threadIdx.x, g = threadIdx.y;
    const int c = blockIdx.y;
    const long long lo = a.lo[c], hi = a.hi[c];
    const long long e = (lo / 32) * 32 + (long long)blockIdx.x * 32 + lane;
    const bool live = e >= lo && e < hi;            // every thread takes part in the barriers
    T val = T(0);
    if (live) {
        const unsigned long long len = (unsigned long long)(a.ghi[c] - a.glo[c]);
        const unsigned long long x0 = (unsigned long long)(a.w0 + e - a.glo[c]);
        const int j = (int)(((x0 + 1) * (unsigned)a.n - 1) / len);      // owner of the column's block
        int base[D];
#pragma unroll
        for (int d = 0; d < D; ++d) base[d] = (j / a.dstride[d]) % a.dims[d];
        int gg = g;
#pragma unroll
        for (int t = L; t < S; ++t) {               // centre of this thread's subtree: digits of g, level L lowest
            const int eps = gg % 3 - 1, dt = a.ldim[c][t], xt = a.ldist[c][t];
            gg /= 3;
#pragma unroll
            for (int d = 0; d < D; ++d) if (d == dt) base[d] = wrap(base[d] + eps * xt, a.dims[d]);
        }
        int ldm[L], ldx[L];
#pragma unroll
        for (int t = 0; t < L; ++t) { ldm[t] = a.ldim[c][t]; ldx[t] = a.ldist[c][t]; }
        T l[LEAVES];
#pragma unroll
        for (int m = 0; m < LEAVES; ++m) {          // leaf m <-> eps_t = (m / 3^t) % 3 - 1
            const int eps[3] = {m % 3 - 1, (m / 3) % 3 - 1, m / 9 - 1};
            int rank = 0;
#pragma unroll
            for (int d = 0; d < D; ++d) {
                int off = 0;
#pragma unroll
                for (int t = 0; t < L; ++t) off += (ldm[t] == d) ? eps[t] * ldx[t] : 0;
                rank += wrap(base[d] + off, a.dims[d]) * a.dstride[d];   // |off| < a_d
            }
            l[m] = tabs.in(rank)[e];
        }
        T r9[LEAVES / 9];
#pragma unroll
        for (int q = 0; q < LEAVES / 9; ++q)
            r9[q] = add3(add3(l[9 * q], l[9 * q + 1], l[9 * q + 2]), add3(l[9 * q + 3], l[9 * q + 4], l[9 * q + 5]),
                         add3(l[9 * q + 6], l[9 * q + 7], l[9 * q + 8]));
        if constexpr (L == 3) val = add3(r9[0], r9[1], r9[2]);
        else val = r9[0];
    }
    xch[g * 32 + lane] = val;
    __syncthreads();
#pragma unroll
    for (int step = 1; step < G; step *= 3) {
        if (g % (3 * step) == 0) xch[g * 32 + lane] = add3(xch[g * 32 + lane], xch[(g + step) * 32 + lane], xch[(g + 2 * step) * 32 + lane]);
        __syncthreads();
    }
    const T res = xch[lane];
    if (live)
        for (int r = g; r < a.n; r += G) tabs.out(r)[e] = res;
}

template <typename T, int S, int D, int CAP>
__global__ void __launch_bounds__(32 * coop_G(S)) k_bw_coop(PtrTab<CAP> in, PtrTab<CAP> out, BwArgs a) {
    pdl_trigger();
    __shared__ const T* sin[CAP];
    __shared__ T* sout[CAP];
    __shared__ T xch[coop_G(S) * 32];
    for (int r = threadIdx.y * 32 + threadIdx.x; r < a.n; r += 32 * coop_G(S)) { sin[r] = (const T*)in.p[r]; sout[r] = (T*)out.p[r]; }
    __syncthreads();
    pdl_wait();
    bw_coop_tile<T, S, D>(a, SmemTabs<T>{sin, sout}, xch);
}

template <typename T, int S, int D>
__global__ void __launch_bounds__(32 * coop_G(S)) k_bw_coop_strided(StrideAddr in, StrideAddr out, BwArgs a) {
    pdl_trigger();
    __shared__ T xch[coop_G(S) * 32];
    pdl_wait();
    bw_coop_tile<T, S, D>(a, StrideTabs<T>{in, out}, xch);
}

template <typename T, int V, int S, int D, typename Tabs>
__device__ __forceinline__ void bw_tile(const BwArgs& a, const Tabs& tabs) {
    const int c = blockIdx.y;
    const long long lo = a.lo[c], hi = a.hi[c];
    // tiles start on multiples of 32*V elements: a warp's access to one rank is one aligned run
    const long long e = (lo / (32 * V)) * (32 * V) + ((long long)blockIdx.x * kBwThreads + threadIdx.x) * V;
    if (e >= hi || e + V <= lo) return;
    const unsigned long long L = (unsigned long long)(a.ghi[c] - a.glo[c]);
    auto owner = [&](long long el) -> int {
        const unsigned long long x = (unsigned long long)(a.w0 + el - a.glo[c]);
        return (int)(((x + 1) * (unsigned)a.n - 1) / L);
    };
    if constexpr (V == 1) {
        column_tree<T, 1, S, D>(a, c, tabs, e, owner(e));
    } else {
        const bool inside = e >= lo && e + V <= hi;
        int j0 = 0;
        bool same = false;
        if (inside) { j0 = owner(e); same = owner(e + V - 1) == j0; }
        if (same) {
            column_tree<T, V, S, D>(a, c, tabs, e, j0);
        } else {
            for (int k = 0; k < V; ++k)
                if (e + k >= lo && e + k < hi) column_tree<T, 1, S, D>(a, c, tabs, e + k, owner(e + k));
        }
    }
}

template <typename T, int V, int S, int D, int CAP>
__global__ void __launch_bounds__(kBwThreads) k_bw_fused(PtrTab<CAP> in, PtrTab<CAP> out, BwArgs a) {
    pdl_trigger();
    __shared__ const T* sin[CAP];
    __shared__ T* sout[CAP];
    for (int r = threadIdx.x; r < a.n; r += kBwThreads) { sin[r] = (const T*)in.p[r]; sout[r] = (T*)out.p[r]; }
    __syncthreads();
    pdl_wait();
    bw_tile<T, V, S, D>(a, SmemTabs<T>{sin, sout});
}

template <typename T, int V, int S, int D>
__global__ void __launch_bounds__(kBwThreads) k_bw_fused_strided(StrideAddr in, StrideAddr out, BwArgs a) {
    pdl_trigger();
    pdl_wait();
    bw_tile<T, V, S, D>(a, StrideTabs<T>{in, out});
}

// ------------------------------------------------------------------ host side

bool fused_bandwidth_supported(const Plan& p) {
    return p.algo == TRV_ALGO_TRIVANCE && p.variant == TRV_BANDWIDTH_OPTIMAL && p.ndims <= kBwMaxD && p.S <= kBwMaxS;
}

template <typename T, int V, int S, int D>
static void launch_bw(const Call& c, const BwArgs& a) {
    constexpr int CAP = S <= 3 ? 32 : (S <= 5 ? 256 : TRV_MAX_RANKS);
    const Plan& p = *c.plan;
    long long tiles = 0;
    for (int sl = 0; sl < D; ++sl)
        if (a.hi[sl] > a.lo[sl]) {
            long long t = (a.hi[sl] - (a.lo[sl] / (32 * V)) * (32 * V) + (long long)V * kBwThreads - 1) / ((long long)V * kBwThreads);
            if (t > tiles) tiles = t;
        }
    if (tiles == 0) return;
    StrideAddr sin, sout;
    const bool strided = uniform_stride(c.in, p.n, &sin) && uniform_stride((const void* const*)c.out, p.n, &sout);
    if constexpr (V == 1 && S >= 3) {       // short vectors: several threads per column
        long long ct = 0;
        for (int sl = 0; sl < D; ++sl)
            if (a.hi[sl] > a.lo[sl]) {
                const long long t = (a.hi[sl] - (a.lo[sl] / 32) * 32 + 31) / 32;
                if (t > ct) ct = t;
            }
        const dim3 grid((unsigned)ct, D, 1), block(32, coop_G(S), 1);
        if (strided) {
            launch_pdl(k_bw_coop_strided<T, S, D>, grid, block, 0, c.st, sin, sout, a);
        } else {
            PtrTab<CAP> in, out;
            for (int r = 0; r < p.n; ++r) { in.p[r] = const_cast<void*>(c.in[r]); out.p[r] = c.out[r]; }
            launch_pdl(k_bw_coop<T, S, D, CAP>, grid, block, 0, c.st, in, out, a);
        }
    } else if (strided) {
        launch_pdl(k_bw_fused_strided<T, V, S, D>, dim3((unsigned)tiles, D, 1), dim3(kBwThreads), 0, c.st, sin, sout, a);
    } else {
        PtrTab<CAP> in, out;
        for (int r = 0; r < p.n; ++r) { in.p[r] = const_cast<void*>(c.in[r]); out.p[r] = c.out[r]; }
        launch_pdl(k_bw_fused<T, V, S, D, CAP>, dim3((unsigned)tiles, D, 1), dim3(kBwThreads), 0, c.st, in, out, a);
    }
}

template <typename T, int V, int S>
static trv_status_t bw_by_d(const Call& c, const BwArgs& a) {
    switch (c.plan->ndims) {
        case 1: launch_bw<T, V, S, 1>(c, a); return TRV_OK;
        case 2: if constexpr (S >= 2) { launch_bw<T, V, S, 2>(c, a); return TRV_OK; } break;
        case 3: if constexpr (S >= 3) { launch_bw<T, V, S, 3>(c, a); return TRV_OK; } break;
        case 4: if constexpr (S >= 4) { launch_bw<T, V, S, 4>(c, a); return TRV_OK; } break;
    }
    return TRV_ERR_UNSUPPORTED;
}

template <typename T, int V>
static trv_status_t bw_by_s(const Call& c, const BwArgs& a) {
    switch (c.plan->S) {
        case 1: return bw_by_d<T, V, 1>(c, a);
        case 2: return bw_by_d<T, V, 2>(c, a);
        case 3: return bw_by_d<T, V, 3>(c, a);
        case 4: return bw_by_d<T, V, 4>(c, a);
        case 5: return bw_by_d<T, V, 5>(c, a);
        case 6: return bw_by_d<T, V, 6>(c, a);
    }
    return TRV_ERR_UNSUPPORTED;
}

trv_status_t run_fused_bandwidth(const Call& c) {
    const Plan& p = *c.plan;
    if (!fused_bandwidth_supported(p)) return TRV_ERR_UNSUPPORTED;
    BwArgs a;
    a.n = p.n;
    a.w0 = (long long)c.goff;
    long long min_block = -1;
    for (int d = 0; d < kBwMaxD; ++d) { a.dims[d] = d < p.ndims ? p.dims[d] : 1; a.dstride[d] = d < p.ndims ? p.stride[d] : 1; }
    for (int sl = 0; sl < p.ndims; ++sl) {
        local_slice(c, sl, &a.lo[sl], &a.hi[sl]);
        a.glo[sl] = slice_lo((int64_t)c.gcount, p.ndims, sl);
        a.ghi[sl] = slice_lo((int64_t)c.gcount, p.ndims, sl + 1);
        const long long bl = (a.ghi[sl] - a.glo[sl]) / p.n;
        if (min_block < 0 || bl < min_block) min_block = bl;
        for (int t = 0; t < p.S; ++t) { a.ldim[sl][t] = p.steps[sl][t].dim; a.ldist[sl][t] = p.steps[sl][t].dist; }
    }
    // Two columns per thread (8-byte accesses, packed adds) when blocks are long enough that few
    // threads straddle a block boundary and the vector is long enough to fill the GPU with such
    // threads; otherwise several threads per column (k_bw_coop; n <= 9: one thread per column).
    // Measured on B200: two columns beat four at every size (shorter thread lifetimes, more warps).
    const bool wide = min_block >= 256 && c.count >= ((size_t)1 << 20);
    g_last_kernel = wide ? "bw_fused<V=2>" : (p.S >= 3 ? "bw_coop" : "bw_fused<V=1>");
    trv_status_t st;
    if (c.dtype == TRV_FLOAT32) st = wide ? bw_by_s<float, 2>(c, a) : bw_by_s<float, 1>(c, a);
    else st = wide ? bw_by_s<uint32_t, 2>(c, a) : bw_by_s<uint32_t, 1>(c, a);
    if (st != TRV_OK) return st;
    return cudaGetLastError() == cudaSuccess ? TRV_OK : TRV_ERR_CUDA;
}

}  // namespace trv
