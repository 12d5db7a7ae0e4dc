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
// Few ranks leave a thread little to do (n loads, n stores): a ring of 8 reaches 0.77 - 0.82 of the copy bandwidth, 32 ranks
// 0.95.  Letting a CTA work through 2 - 8 consecutive tiles made that worse (ring of 8: 0.50, 32 ranks: 0.80): what these
// sizes lack is loads in flight, and a CTA that runs its tiles one after the other has fewer of them than eight CTAs side by side.
#include <algorithm>
#include <type_traits>
#include <vector>

#include "trv_dev.cuh"

namespace trv {

constexpr int kTreeThreads = 128;
constexpr int kTreeChunk = 8;       // program entries whose loads are in flight together
constexpr int kTreeDepth = 12;      // stack slots: tree height <= steps + 1 <= 11 for n <= 1024 in up to four dimensions
constexpr int kTreeAlign = 64;      // tiles start on multiples of 64 elements of the buffers: a warp's access is whole 128-byte lines

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
    int two_blocks;                                     // every block is at least a CTA's span long
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

// V columns starting at local element e: evaluate the tree, store to all ranks.  rank_of(o, k) = the rank at offset o
// from the block that column k lies in.  SPLIT = false: both columns lie in one block and are loaded and stored as one
// vector.  SPLIT = true (V = 2): the columns may lie in different blocks, or one of them outside the collective
// (live[k] = false): one scalar access per column, same walk.  A warp takes ONE of the two forms as a whole, so a
// block boundary inside a warp costs no second pass.
// `stack` is this thread's slot of level 0; levels are kTreeThreads * V elements apart.
template <typename T, int V, bool SPLIT, typename Tabs, typename RankOf>
__device__ __forceinline__ void tree_column(const TreeArgs& a, const unsigned short* prog, const Tabs& tabs, long long e,
                                            RankOf rank_of, T* stack, bool live0, bool live1) {
    using P = Elem<T, V>;
    const int n = a.n;
    const long long e0 = live0 ? e : e + 1, e1 = live1 ? e + 1 : e;     // a column that is not live re-reads the live one
    auto load_chunk = [&](int i0, P (&v)[kTreeChunk]) {
#pragma unroll
        for (int m = 0; m < kTreeChunk; ++m) {
            const int idx = i0 + m;
            if (idx < n) {
                const int o = prog[idx] & 1023;
                if constexpr (!SPLIT) {
                    v[m] = *reinterpret_cast<const P*>(tabs.in(rank_of(o, 0)) + e);
                } else {
                    v[m].x[0] = tabs.in(rank_of(o, 0))[e0];
                    v[m].x[1] = tabs.in(rank_of(o, 1))[e1];
                }
            }
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
                    if (idx > 0) *reinterpret_cast<P*>(stack + (sp++) * (kTreeThreads * V)) = tos;
                    tos = cur[m];
                } else {                // a leaf closes at once: add it to the value on top, no stack traffic
                    tos = add2(tos, cur[m]);
                    for (--k; k > 0; --k) tos = add2(*reinterpret_cast<const P*>(stack + (--sp) * (kTreeThreads * V)), tos);
                }
            }
        }
    }
    if constexpr (!SPLIT) {
#pragma unroll 8
        for (int r = 0; r < n; ++r) *reinterpret_cast<P*>(tabs.out(r) + e) = tos;
    } else {
#pragma unroll 4
        for (int r = 0; r < n; ++r) {
            if (live0) tabs.out(r)[e] = tos.x[0];
            if (live1) tabs.out(r)[e + 1] = tos.x[1];
        }
    }
}

template <typename T, int V, int CAP, typename Tabs>
__device__ __forceinline__ void tree_tile(const TreeArgs& a, const TreeProg<CAP>& progs, const Tabs& tabs, void* stack_raw,
                                          unsigned short* rk, unsigned* oc) {
    const int c = blockIdx.y, n = a.n;                  // CTA-uniform: the collective
    const unsigned short* prog = progs.e[c];
    const long long slo = a.slo[c], shi = a.shi[c];
    // local range of the collective inside the window; tiles aligned to whole lines of the buffers (a collective
    // that starts inside a line leaves the columns before its start to the previous collective's last tile)
    long long llo = slo - a.w0, lhi = shi - a.w0;
    if (llo < 0) llo = 0;
    if (lhi > a.count) lhi = a.count;
    const long long t0 = (llo / kTreeAlign) * kTreeAlign + (long long)blockIdx.x * kTreeThreads * V;
    if (t0 >= lhi) return;
    auto owner = [&](long long el) -> int {
        const unsigned long long x = (unsigned long long)(a.w0 + el - slo);
        return (int)(((x + 1) * (unsigned)n - 1) / (unsigned long long)(shi - slo));
    };
    // Torus: block + offset is tabulated for the block the CTA's first column lies in and for the next one; where
    // blocks are at least a CTA's span long (a.two_blocks) no CTA reaches a third.  Otherwise (short vectors) it is
    // computed from the packed coordinates oc of the offsets.
    const bool torus = a.geo.nd > 1;
    const int b0 = owner(t0 < llo ? llo : t0), b1 = b0 + 1 < n ? b0 + 1 : b0;
    if (torus) {
        for (int o = threadIdx.x; o < n; o += kTreeThreads) oc[o] = geo_pack(a.geo, o);
        __syncthreads();
        if (a.two_blocks) {
            const unsigned c0 = geo_pack(a.geo, b0), c1 = geo_pack(a.geo, b1);
            for (int o = threadIdx.x; o < n; o += kTreeThreads) {
                rk[o] = (unsigned short)geo_add_packed(a.geo, c0, oc[o]);
                rk[CAP + o] = (unsigned short)geo_add_packed(a.geo, c1, oc[o]);
            }
            __syncthreads();
        }
    }
    const long long e = t0 + (long long)threadIdx.x * V;
    T* const stack = reinterpret_cast<T*>(stack_raw) + threadIdx.x * V;
    if constexpr (V == 1) {
        if (e >= lhi || e < llo) return;
        const int b = owner(e);
        if (!torus) {
            tree_column<T, 1, false>(a, prog, tabs, e, [&](int o, int) { int r = b + o; return r >= n ? r - n : r; }, stack, true, true);
        } else if (a.two_blocks) {
            const unsigned short* tab = b == b0 ? rk : rk + CAP;
            tree_column<T, 1, false>(a, prog, tabs, e, [&](int o, int) { return (int)tab[o]; }, stack, true, true);
        } else {
            const unsigned cb = geo_pack(a.geo, b);
            tree_column<T, 1, false>(a, prog, tabs, e, [&](int o, int) { return geo_add_packed(a.geo, cb, oc[o]); }, stack, true, true);
        }
    } else {
        static_assert(V == 2, "one or two columns per thread");
        const bool live0 = e >= llo && e < lhi, live1 = e + 1 >= llo && e + 1 < lhi;
        const bool dead = !(live0 || live1);
        const int bA = dead ? 0 : owner(live0 ? e : e + 1), bB = dead ? 0 : owner(live1 ? e + 1 : e);
        // all 32 lanes are here (every return above is CTA-uniform): the warp picks one form
        const bool vec = __all_sync(0xffffffffu, dead || (live0 && live1 && bA == bB));
        if (dead) return;
        if (!torus) {
            auto rank_of = [&](int o, int k) { int r = (k ? bB : bA) + o; return r >= n ? r - n : r; };
            if (vec) tree_column<T, 2, false>(a, prog, tabs, e, rank_of, stack, true, true);
            else tree_column<T, 2, true>(a, prog, tabs, e, rank_of, stack, live0, live1);
        } else {        // the host takes this kernel only where a.two_blocks holds
            const unsigned short* tA = bA == b0 ? rk : rk + CAP;
            const unsigned short* tB = bB == b0 ? rk : rk + CAP;
            auto rank_of = [&](int o, int k) { return (int)(k ? tB : tA)[o]; };
            if (vec) tree_column<T, 2, false>(a, prog, tabs, e, rank_of, stack, true, true);
            else tree_column<T, 2, true>(a, prog, tabs, e, rank_of, stack, live0, live1);
        }
    }
}

template <typename T, int V, int CAP>
__global__ void __launch_bounds__(kTreeThreads) k_bw_tree(PtrTab<CAP> in, PtrTab<CAP> out, TreeProg<CAP> prog, TreeArgs a) {
    pdl_trigger();
    __shared__ const T* sin[CAP];
    __shared__ T* sout[CAP];
    __shared__ __align__(16) unsigned char stack[kTreeDepth * kTreeThreads * V * sizeof(T)];
    __shared__ unsigned short rk[2 * CAP];
    __shared__ unsigned oc[CAP];
    for (int r = threadIdx.x; r < a.n; r += kTreeThreads) { sin[r] = (const T*)in.p[r]; sout[r] = (T*)out.p[r]; }
    __syncthreads();
    pdl_wait();
    tree_tile<T, V, CAP>(a, prog, TreeSmemTabs<T, CAP>{sin, sout}, stack, rk, oc);
}

template <typename T, int V, int CAP>
__global__ void __launch_bounds__(kTreeThreads) k_bw_tree_strided(StrideAddr in, StrideAddr out, TreeProg<CAP> prog, TreeArgs a) {
    pdl_trigger();
    __shared__ __align__(16) unsigned char stack[kTreeDepth * kTreeThreads * V * sizeof(T)];
    __shared__ unsigned short rk[2 * CAP];
    __shared__ unsigned oc[CAP];
    pdl_wait();
    tree_tile<T, V, CAP>(a, prog, TreeStrideTabs<T>{in, out}, stack, rk, oc);
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
    a.two_blocks = (long long)(c.gcount / p.nslices / p.n) >= (long long)V * kTreeThreads ? 1 : 0;
    long long tiles = 0;
    for (int sl = 0; sl < kTreeMaxSlices; ++sl) {
        a.slo[sl] = a.shi[sl] = 0;
        if (sl >= p.nslices) continue;
        for (int i = 0; i < p.n; ++i) pg.e[sl][i] = progs[sl][i];
        a.slo[sl] = slice_lo((int64_t)c.gcount, p.nslices, sl);
        a.shi[sl] = slice_lo((int64_t)c.gcount, p.nslices, sl + 1);
        long long lo, hi;
        local_slice(c, sl, &lo, &hi);
        if (hi > lo)
            tiles = std::max(tiles, (hi - (lo / kTreeAlign) * kTreeAlign + (long long)V * kTreeThreads - 1) / ((long long)V * kTreeThreads));
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
    if (p.tree_ready) return true;
    return p.general && p.n <= TRV_MAX_RANKS && p.nslices <= kTreeMaxSlices && p.ndims <= 4 && p.S + 2 <= kTreeDepth;
}

// once per plan (prepare_launch_data): the depth-first programs of all collectives
void tree_prepare(Plan& p) {
    p.tree_ready = false;
    p.tree_progs.clear();
    if (!fused_tree_supported(p)) return;
    std::vector<std::vector<unsigned short>> progs(p.nslices);
    for (int sl = 0; sl < p.nslices; ++sl) {
        progs[sl].reserve(p.n);
        const int depth = build_program(p, sl, progs[sl]);
        if ((int)progs[sl].size() != p.n || depth > kTreeDepth) return;
    }
    p.tree_progs.swap(progs);
    p.tree_ready = true;
}

trv_status_t run_fused_tree(const Call& c) {
    const Plan& p = *c.plan;
    if (!p.tree_ready) return TRV_ERR_UNSUPPORTED;
    const std::vector<std::vector<unsigned short>>& progs = p.tree_progs;
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
