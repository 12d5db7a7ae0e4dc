// FUSED kernel for rings whose size is no power of three (Sec. 4.4), bandwidth-optimal form.
//
// Every block follows the same reduction tree up to rotation (Plan::gstep / gsgn).  The owner's
// final value of a block is that tree evaluated bottom-up; the AllGather hands it to every rank.
// The host flattens the tree into a PROGRAM: the nodes in the order a depth-first walk first
// meets them (a node, then for every step in ascending order its left child's subtree and its
// right child's subtree), each with the number of additions that follow it.  A thread runs the
// program for its element column(s) as a small stack machine:
//     visit node      : push the input of rank (block + offset) mod n
//     after a subtree : pop it and add it to the value below  (own <- own + child)
// which performs exactly the additions of the schedule in the schedule's association
// ((from_left + own) + from_right at every step; binary32 addition is commutative, so which
// operand comes first does not change a bit).  Loads are issued a chunk of program entries
// ahead of the additions that consume them; the stack lives in shared memory (one slot column
// per thread) with its top in registers.  n*count elements read once, n*count written once.
#include <vector>

#include "trv_dev.cuh"

namespace trv {

constexpr int kTreeThreads = 128;
constexpr int kTreeChunk = 8;       // program entries whose loads are in flight together
constexpr int kTreeDepth = 10;      // stack slots: tree height <= steps + 1 <= 8 for n <= 1024

// entry: offset from the block's owner (bits 0..9) | additions after this node (bits 10..13)
template <int CAP>
struct TreeProg {
    unsigned short e[CAP];
};
struct TreeArgs {
    int n;
    long long w0, gcount;       // global index of local element 0; global vector length
    long long count;            // local elements
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
template <typename T, int V, int SLOT, int CAP, typename Tabs>
__device__ __forceinline__ void tree_column(const TreeArgs& a, const TreeProg<CAP>& prog, const Tabs& tabs, long long e,
                                            int b, T* stack) {
    static_assert(V <= SLOT, "slot too narrow");
    using P = Elem<T, V>;
    const int n = a.n;
    auto load_chunk = [&](int i0, P (&v)[kTreeChunk]) {
#pragma unroll
        for (int m = 0; m < kTreeChunk; ++m) {
            const int idx = i0 + m;
            if (idx < n) {
                int r = b + (prog.e[idx] & 1023);
                if (r >= n) r -= n;
                v[m] = *reinterpret_cast<const P*>(tabs.in(r) + e);
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
                int k = prog.e[idx] >> 10;
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
__device__ __forceinline__ void tree_tile(const TreeArgs& a, const TreeProg<CAP>& prog, const Tabs& tabs, void* stack_raw) {
    const long long e = ((long long)blockIdx.x * kTreeThreads + threadIdx.x) * V;
    if (e >= a.count) return;
    auto owner = [&](long long el) -> int {
        const unsigned long long x = (unsigned long long)(a.w0 + el);
        return (int)(((x + 1) * (unsigned)a.n - 1) / (unsigned long long)a.gcount);
    };
    T* const stack = reinterpret_cast<T*>(stack_raw) + threadIdx.x * V;
    if constexpr (V == 1) {
        tree_column<T, 1, 1, CAP>(a, prog, tabs, e, owner(e), stack);
    } else {
        const bool inside = e + V <= a.count;
        int b0 = 0;
        bool same = false;
        if (inside) { b0 = owner(e); same = owner(e + V - 1) == b0; }
        if (same) {
            tree_column<T, V, V, CAP>(a, prog, tabs, e, b0, stack);
        } else {
            for (int k = 0; k < V; ++k)
                if (e + k < a.count)
                    tree_column<T, 1, V, CAP>(a, prog, tabs, e + k, owner(e + k), stack);
        }
    }
}

template <typename T, int V, int CAP>
__global__ void __launch_bounds__(kTreeThreads) k_bw_tree(PtrTab<CAP> in, PtrTab<CAP> out, TreeProg<CAP> prog, TreeArgs a) {
    pdl_trigger();
    __shared__ const T* sin[CAP];
    __shared__ T* sout[CAP];
    __shared__ __align__(16) unsigned char stack[kTreeDepth * kTreeThreads * V * sizeof(T)];
    for (int r = threadIdx.x; r < a.n; r += kTreeThreads) { sin[r] = (const T*)in.p[r]; sout[r] = (T*)out.p[r]; }
    __syncthreads();
    pdl_wait();
    tree_tile<T, V, CAP>(a, prog, TreeSmemTabs<T, CAP>{sin, sout}, stack);
}

template <typename T, int V, int CAP>
__global__ void __launch_bounds__(kTreeThreads) k_bw_tree_strided(StrideAddr in, StrideAddr out, TreeProg<CAP> prog, TreeArgs a) {
    pdl_trigger();
    __shared__ __align__(16) unsigned char stack[kTreeDepth * kTreeThreads * V * sizeof(T)];
    pdl_wait();
    tree_tile<T, V, CAP>(a, prog, TreeStrideTabs<T>{in, out}, stack);
}

// ------------------------------------------------------------------ host side

// Depth-first flattening of the tree stored by offsets; returns the deepest stack it needs.
static int build_program(const Plan& p, std::vector<unsigned short>& prog) {
    const int n = p.n, S = p.S;
    int depth = 0, max_depth = 0;
    struct Walk {
        const Plan& p; std::vector<unsigned short>& prog; int n, S; int& depth; int& max_depth;
        void visit(int v) {
            prog.push_back((unsigned short)v);
            if (++depth > max_depth) max_depth = depth;
            const int upto = v == 0 ? S : p.gstep[v];
            for (int t = 0; t < upto; ++t) {
                const int dist = p.steps[0][t].dist;
                const int l = ((v - dist) % n + n) % n, r = (v + dist) % n;
                if (p.gstep[l] == t && p.gsgn[l] > 0) { visit(l); prog.back() += 1 << 10; --depth; }
                if (r != l && p.gstep[r] == t && p.gsgn[r] < 0) { visit(r); prog.back() += 1 << 10; --depth; }
            }
        }
    } w{p, prog, n, S, depth, max_depth};
    w.visit(0);
    return max_depth;
}

template <typename T, int V, int CAP>
static trv_status_t launch_tree(const Call& c, const std::vector<unsigned short>& prog) {
    const Plan& p = *c.plan;
    TreeProg<CAP> pg;
    for (int i = 0; i < p.n; ++i) pg.e[i] = prog[i];
    TreeArgs a;
    a.n = p.n; a.w0 = (long long)c.goff; a.gcount = (long long)c.gcount; a.count = (long long)c.count;
    const long long tiles = ((long long)c.count + (long long)V * kTreeThreads - 1) / ((long long)V * kTreeThreads);
    StrideAddr sin, sout;
    if (uniform_stride(c.in, p.n, &sin) && uniform_stride((const void* const*)c.out, p.n, &sout)) {
        launch_pdl(k_bw_tree_strided<T, V, CAP>, dim3((unsigned)tiles), dim3(kTreeThreads), 0, c.st, sin, sout, pg, a);
    } else {
        PtrTab<CAP> in, out;
        for (int r = 0; r < p.n; ++r) { in.p[r] = const_cast<void*>(c.in[r]); out.p[r] = c.out[r]; }
        launch_pdl(k_bw_tree<T, V, CAP>, dim3((unsigned)tiles), dim3(kTreeThreads), 0, c.st, in, out, pg, a);
    }
    return cudaGetLastError() == cudaSuccess ? TRV_OK : TRV_ERR_CUDA;
}

template <typename T, int V>
static trv_status_t tree_by_cap(const Call& c, const std::vector<unsigned short>& prog) {
    if (c.plan->n <= 32) return launch_tree<T, V, 32>(c, prog);
    if (c.plan->n <= 256) return launch_tree<T, V, 256>(c, prog);
    return launch_tree<T, V, TRV_MAX_RANKS>(c, prog);
}

bool fused_tree_supported(const Plan& p) { return p.general && p.n <= TRV_MAX_RANKS && p.S + 2 <= kTreeDepth; }

trv_status_t run_fused_tree(const Call& c) {
    const Plan& p = *c.plan;
    if (!fused_tree_supported(p)) return TRV_ERR_UNSUPPORTED;
    std::vector<unsigned short> prog;
    prog.reserve(p.n);
    const int depth = build_program(p, prog);
    if ((int)prog.size() != p.n || depth > kTreeDepth) return TRV_ERR_UNSUPPORTED;
    // two columns per thread when blocks are long (few threads straddle a block boundary) and the
    // vector is long enough to fill the GPU with such threads.  Measured on B200 at 8 MiB per rank:
    // four columns per thread are slower from 53 ranks up (0.82 against 0.89 of the copy bandwidth
    // at 100 ranks) and no faster below, but for 32 ranks.
    const bool wide = (long long)(c.gcount / p.n) >= 256 && c.count >= ((size_t)1 << 20);
    g_last_kernel = wide ? "bw_tree<V=2>" : "bw_tree<V=1>";
    if (c.dtype == TRV_FLOAT32) return wide ? tree_by_cap<float, 2>(c, prog) : tree_by_cap<float, 1>(c, prog);
    return wide ? tree_by_cap<uint32_t, 2>(c, prog) : tree_by_cap<uint32_t, 1>(c, prog);
}

}  // namespace trv
