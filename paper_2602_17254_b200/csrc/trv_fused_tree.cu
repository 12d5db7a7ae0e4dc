// FUSED kernel for rings and tori with a side that is no power of three (Sec. 4.4, Sec. 5), bandwidth-optimal form.
//
// Every block of a collective follows the same reduction tree up to translation (Plan::gstep / gsgn).  The owner's
// final value of a block is that tree evaluated bottom-up; the AllGather hands it to every rank.
// The host flattens the tree into a PROGRAM: the nodes in the order a depth-first walk first
// meets them (a node, then for every step in ascending order its left child's subtree and its
// right child's subtree), each with the number of additions that follow it.  A thread runs the
// program for its element column(s) as a small stack machine:
//     visit node      : push the input of rank block + offset (coordinate by coordinate, modulo the sides)
//     after a subtree : pop it and add it to the value below  (own <- own + child)
// which performs exactly the additions of the schedule in the schedule's association
// ((from_left + own) + from_right at every step; binary32 addition is commutative, so which
// operand comes first does not change a bit).  Loads are issued a chunk of program entries
// ahead of the additions that consume them; the stack lives in shared memory (one slot column
// per thread) with its top in registers.  n*count elements read once, n*count written once.
// On a torus every collective (slice of the vector) has its own program (grid.y = collective) and block + offset
// needs one modular addition per dimension: the CTA tabulates it once for the block its first column lies in
// (shared memory, 2 bytes per node); the threads of the few CTAs that straddle a block boundary compute it.
#include <algorithm>
#include <type_traits>
#include <vector>

#include "trv_dev.cuh"

namespace trv {

constexpr int kTreeThreads = 128;
constexpr int kTreeChunk = 8;       // program entries whose loads are in flight together
constexpr int kTreeDepth = 10;      // stack slots: tree height <= steps + 1 <= 8 for n <= 1024

// entry: offset from the block's owner (bits 0..9) | additions after this node (bits 10..13); one program per collective
constexpr int kTreeMaxSlices = 4;
template <int CAP>
struct TreeProg {
    unsigned short e[kTreeMaxSlices][CAP];
};
struct TreeArgs {
    int n;
    long long w0, count;                                // global index of local element 0; local elements
    long long slo[kTreeMaxSlices], shi[kTreeMaxSlices]; // the collectives' slices of the global vector
    TorusGeo geo;
};

template <typename T, int CAP>
struct TreeSmemTabs {
    const T* const* sin;
    T* const* sout;
    __device__ __forceinline__ const T* in(int r) const { return sin[r]; }
    __device__ __forceinline__ T* out(int r) const { return sout[r]; }
};
template <typename T>
struct TreeStrideTabs {
    StrideAddr i, o;
    __device__ __forceinline__ const T* in(int r) const { return reinterpret_cast<const T*>(i.ptr(r)); }
    __device__ __forceinline__ T* out(int r) const { return reinterpret_cast<T*>(o.ptr(r)); }
};

// V columns starting at local element e, all inside block b: evaluate the tree, store to all ranks.
// `stack` is this thread's slot of level 0; levels are kTreeThreads * SLOT elements apart, SLOT being
// the slot width of the kernel (its own V) also when a thread walks single columns, so that the
// slots of different threads never overlap.
template <typename T, int V, int SLOT, typename Tabs, typename RankOf>
__device__ __forceinline__ void tree_column(const TreeArgs& a, const unsigned short* prog, const Tabs& tabs, long long e,
                                            RankOf rank_of, T* stack) {
    static_assert(V <= SLOT, "slot too narrow");
    using P = Elem<T, V>;
    const int n = a.n;
    auto load_chunk = [&](int i0, P (&v)[kTreeChunk]) {
#pragma unroll
        for (int m = 0; m < kTreeChunk; ++m) {
            const int idx = i0 + m;
            if (idx < n) v[m] = *reinterpret_cast<const P*>(tabs.in(rank_of(prog[idx] & 1023)) + e);
        }
    };
    P nxt[kTreeChunk];
    P tos;
    int sp = 0;
    load_chunk(0, nxt);
    for (int i0 = 0; i0 < n; i0 += kTreeChunk) {
        P cur[kTreeChunk];
#pragma unroll
        for (int m = 0; m < kTreeChunk; ++m) cur[m] = nxt[m];
        if (i0 + kTreeChunk < n) load_chunk(i0 + kTreeChunk, nxt);
#pragma unroll
        for (int m = 0; m < kTreeChunk; ++m) {
            const int idx = i0 + m;
            if (idx < n) {
                int k = prog[idx] >> 10;
                if (k == 0) {           // an inner node: its subtrees follow
                    if (idx > 0) *reinterpret_cast<P*>(stack + (sp++) * (kTreeThreads * SLOT)) = tos;
                    tos = cur[m];
                } else {                // a leaf closes at once: add it to the value on top, no stack traffic
                    tos = add2(tos, cur[m]);
                    for (--k; k > 0; --k) tos = add2(*reinterpret_cast<const P*>(stack + (--sp) * (kTreeThreads * SLOT)), tos);
                }
            }
        }
    }
#pragma unroll 8
    for (int r = 0; r < n; ++r) *reinterpret_cast<P*>(tabs.out(r) + e) = tos;
}

template <typename T, int V, int CAP, typename Tabs>
__device__ __forceinline__ void tree_tile(const TreeArgs& a, const TreeProg<CAP>& progs, const Tabs& tabs, void* stack_raw,
                                          unsigned short* rk) {
    const int c = blockIdx.y, n = a.n;                  // CTA-uniform: the collective
    const unsigned short* prog = progs.e[c];
    const long long slo = a.slo[c], shi = a.shi[c];
    // local range of the collective inside the window, tiles aligned to V elements of the buffers
    long long llo = slo - a.w0, lhi = shi - a.w0;
    if (llo < 0) llo = 0;
    if (lhi > a.count) lhi = a.count;
    const long long t0 = (llo / V) * V + (long long)blockIdx.x * kTreeThreads * V;
    if (t0 >= lhi) return;
    auto owner = [&](long long el) -> int {
        const unsigned long long x = (unsigned long long)(a.w0 + el - slo);
        return (int)(((x + 1) * (unsigned)n - 1) / (unsigned long long)(shi - slo));
    };
    // block + offset for the block the CTA's first column lies in
    const int b0 = owner(t0 < llo ? llo : t0);
    if (a.geo.nd > 1) {
        for (int o = threadIdx.x; o < n; o += kTreeThreads) rk[o] = (unsigned short)geo_add(a.geo, b0, o);
        __syncthreads();
    }
    const long long e = t0 + (long long)threadIdx.x * V;
    if (e >= lhi) return;
    T* const stack = reinterpret_cast<T*>(stack_raw) + threadIdx.x * V;
    auto run = [&](auto width, long long el, int b) {
        constexpr int W = decltype(width)::value;
        if (a.geo.nd == 1) {
            tree_column<T, W, V>(a, prog, tabs, el, [&](int o) { int r = b + o; return r >= n ? r - n : r; }, stack);
        } else if (b == b0) {
            tree_column<T, W, V>(a, prog, tabs, el, [&](int o) { return (int)rk[o]; }, stack);
        } else {
            tree_column<T, W, V>(a, prog, tabs, el, [&](int o) { return geo_add(a.geo, b, o); }, stack);
        }
    };
    if constexpr (V == 1) {
        run(std::integral_constant<int, 1>{}, e, owner(e));
    } else {
        const bool inside = e >= llo && e + V <= lhi;
        int bf = 0;
        bool same = false;
        if (inside) { bf = owner(e); same = owner(e + V - 1) == bf; }
        if (same) {
            run(std::integral_constant<int, V>{}, e, bf);
        } else {
            for (int k = 0; k < V; ++k)
                if (e + k >= llo && e + k < lhi) run(std::integral_constant<int, 1>{}, e + k, owner(e + k));
        }
    }
}

template <typename T, int V, int CAP>
__global__ void __launch_bounds__(kTreeThreads) k_bw_tree(PtrTab<CAP> in, PtrTab<CAP> out, TreeProg<CAP> prog, TreeArgs a) {
    pdl_trigger();
    __shared__ const T* sin[CAP];
    __shared__ T* sout[CAP];
    __shared__ __align__(16) unsigned char stack[kTreeDepth * kTreeThreads * V * sizeof(T)];
    __shared__ unsigned short rk[CAP];
    for (int r = threadIdx.x; r < a.n; r += kTreeThreads) { sin[r] = (const T*)in.p[r]; sout[r] = (T*)out.p[r]; }
    __syncthreads();
    pdl_wait();
    tree_tile<T, V, CAP>(a, prog, TreeSmemTabs<T, CAP>{sin, sout}, stack, rk);
}

template <typename T, int V, int CAP>
__global__ void __launch_bounds__(kTreeThreads) k_bw_tree_strided(StrideAddr in, StrideAddr out, TreeProg<CAP> prog, TreeArgs a) {
    pdl_trigger();
    __shared__ __align__(16) unsigned char stack[kTreeDepth * kTreeThreads * V * sizeof(T)];
    __shared__ unsigned short rk[CAP];
    pdl_wait();
    tree_tile<T, V, CAP>(a, prog, TreeStrideTabs<T>{in, out}, stack, rk);
}

// ------------------------------------------------------------------ host side

// Depth-first flattening of collective c's tree stored by offsets; returns the deepest stack it needs.
static int build_program(const Plan& p, int c, std::vector<unsigned short>& prog) {
    int depth = 0, max_depth = 0;
    struct Walk {
        const Plan& p; int c; std::vector<unsigned short>& prog; int& depth; int& max_depth;
        void visit(int v) {
            prog.push_back((unsigned short)v);
            if (++depth > max_depth) max_depth = depth;
            const int upto = v == 0 ? p.S : p.gstep[c][v];
            for (int t = 0; t < upto; ++t) {
                const int d = p.steps[c][t].dim, dist = p.steps[c][t].dist;
                const int l = p.shift(v, d, -dist), r = p.shift(v, d, dist);
                if (p.gstep[c][l] == t && p.gsgn[c][l] > 0) { visit(l); prog.back() += 1 << 10; --depth; }
                if (r != l && p.gstep[c][r] == t && p.gsgn[c][r] < 0) { visit(r); prog.back() += 1 << 10; --depth; }
            }
        }
    } w{p, c, prog, depth, max_depth};
    w.visit(0);
    return max_depth;
}

template <typename T, int V, int CAP>
static trv_status_t launch_tree(const Call& c, const std::vector<std::vector<unsigned short>>& progs) {
    const Plan& p = *c.plan;
    static thread_local TreeProg<CAP> pg;
    TreeArgs a;
    a.n = p.n; a.w0 = (long long)c.goff; a.count = (long long)c.count;
    a.geo = make_geo(p);
    long long tiles = 0;
    for (int sl = 0; sl < kTreeMaxSlices; ++sl) {
        a.slo[sl] = a.shi[sl] = 0;
        if (sl >= p.nslices) continue;
        for (int i = 0; i < p.n; ++i) pg.e[sl][i] = progs[sl][i];
        a.slo[sl] = slice_lo((int64_t)c.gcount, p.nslices, sl);
        a.shi[sl] = slice_lo((int64_t)c.gcount, p.nslices, sl + 1);
        long long lo, hi;
        local_slice(c, sl, &lo, &hi);
        if (hi > lo) tiles = std::max(tiles, (hi - (lo / V) * V + (long long)V * kTreeThreads - 1) / ((long long)V * kTreeThreads));
    }
    if (tiles == 0) return TRV_OK;
    const dim3 grid((unsigned)tiles, p.nslices, 1);
    StrideAddr sin, sout;
    if (uniform_stride(c.in, p.n, &sin) && uniform_stride((const void* const*)c.out, p.n, &sout)) {
        launch_pdl(k_bw_tree_strided<T, V, CAP>, grid, dim3(kTreeThreads), 0, c.st, sin, sout, pg, a);
    } else {
        PtrTab<CAP> in, out;
        for (int r = 0; r < p.n; ++r) { in.p[r] = const_cast<void*>(c.in[r]); out.p[r] = c.out[r]; }
        launch_pdl(k_bw_tree<T, V, CAP>, grid, dim3(kTreeThreads), 0, c.st, in, out, pg, a);
    }
    return cudaGetLastError() == cudaSuccess ? TRV_OK : TRV_ERR_CUDA;
}

template <typename T, int V>
static trv_status_t tree_by_cap(const Call& c, const std::vector<std::vector<unsigned short>>& prog) {
    if (c.plan->n <= 32) return launch_tree<T, V, 32>(c, prog);
    if (c.plan->n <= 256) return launch_tree<T, V, 256>(c, prog);
    return launch_tree<T, V, TRV_MAX_RANKS>(c, prog);
}

bool fused_tree_supported(const Plan& p) {
    return p.general && p.n <= TRV_MAX_RANKS && p.nslices <= kTreeMaxSlices && p.ndims <= 4 && p.S + 2 <= kTreeDepth;
}

trv_status_t run_fused_tree(const Call& c) {
    const Plan& p = *c.plan;
    if (!fused_tree_supported(p)) return TRV_ERR_UNSUPPORTED;
    std::vector<std::vector<unsigned short>> progs(p.nslices);
    for (int sl = 0; sl < p.nslices; ++sl) {
        progs[sl].reserve(p.n);
        const int depth = build_program(p, sl, progs[sl]);
        if ((int)progs[sl].size() != p.n || depth > kTreeDepth) return TRV_ERR_UNSUPPORTED;
    }
    // two columns per thread when blocks are long (few threads straddle a block boundary) and the
    // vector is long enough to fill the GPU with such threads.  Measured on B200 at 8 MiB per rank:
    // four columns per thread are slower from 53 ranks up (0.82 against 0.89 of the copy bandwidth
    // at 100 ranks) and no faster below, but for 32 ranks.
    const bool wide = (long long)(c.gcount / p.nslices / p.n) >= 256 && c.count >= ((size_t)1 << 20);
    g_last_kernel = wide ? "bw_tree<V=2>" : "bw_tree<V=1>";
    if (c.dtype == TRV_FLOAT32) return wide ? tree_by_cap<float, 2>(c, progs) : tree_by_cap<float, 1>(c, progs);
    return wide ? tree_by_cap<uint32_t, 2>(c, progs) : tree_by_cap<uint32_t, 1>(c, progs);
}

}  // namespace trv
