// FUSED latency-optimal kernel for ANY torus with power-of-three sides up to 81 and at most 729
// ranks (Sec. 4.2, Sec. 5) that has no hand-shaped kernel: 27x27, 3x9, 27x3, 3x3x9, 9x81, ...
//
// A tile is 32 element columns x n ranks in shared memory.  The slice's steps are cut into GROUPS
// of consecutive steps whose closed rank sets are small enough for registers:
//   LINE  : steps of one dimension with distances d, 3d, 9d, ...: closed on the lines
//           {r0 + d*stride*i, i < L}, L = side / d; inside a line the steps have distances 1, 3, ...
//   PLANE : one step in each of two dimensions, closed on {r0 + dA*sA*i + dB*sB*j}, LA x LB <= 81
// Each thread owns one element column and every ninth set of a group; a set is read and written
// by one thread only, so one barrier between groups is all the synchronisation.  The first group
// reads global memory directly and the last one writes it directly: 2 (groups - 1) shared-memory
// passes per tile.  The host builds the group list and the base rank r0 of every set (integer work)
// and passes both by value.
//
// The file is compiled five times (build.py): TRV_LN_PART = 0 gives the host side, 1..4 the kernels of one
// (element type, tile width) pair each, so that the long straight-line bodies compile in parallel.
#include "trv_dev.cuh"
#include "trv_fused_lat.cuh"

#ifndef TRV_LN_PART
#error "compile with -DTRV_LN_PART=0..4 (see build.py)"
#endif

namespace trv {

constexpr int kLnSets = 9;              // sets worked on concurrently per column: 9 x 32 = 288 threads
constexpr int kLnMaxGroups = 8;
constexpr int kLnMaxBases = 1536;
constexpr int kLnMaxD = 4;

enum LnKind : short { LN_LINE = 0, LN_PLANE = 1 };

struct LnGroup {
    short kind, la, lb, nsteps;         // LINE: la = L, nsteps = steps inside the line; PLANE: la x lb
    int stride_a, stride_b;             // rank stride between neighbours along the set's axes
    int nsets, base_off;                // sets of the group, offset of their base ranks in `bases`
};
struct LnProgram {
    int n, cg;                          // cg = column groups of 32 per tile: 9 for n <= 81, else 1
    int ngroups[kLnMaxD];
    LnGroup g[kLnMaxD][kLnMaxGroups];
    short bases[kLnMaxD][kLnMaxBases];
};

#if TRV_LN_PART > 0
template <typename T, int N, bool FULL, typename Addr, typename RankOf>
__device__ __forceinline__ void ln_load(Elem<T, 1> (&v)[N], bool from_global, const Addr& in, const T* mine, int pitch, long long e,
                                        long long lo, long long hi, RankOf rank_of) {
    if (from_global) {
#pragma unroll
        for (int i = 0; i < N; ++i) v[i] = load_elem<T, 1, FULL>(in.ptr(rank_of(i)), e, lo, hi);
    } else {
#pragma unroll
        for (int i = 0; i < N; ++i) v[i].x[0] = mine[rank_of(i) * pitch];
    }
}
template <typename T, int N, bool FULL, typename Addr, typename RankOf>
__device__ __forceinline__ void ln_store(const Elem<T, 1> (&v)[N], bool to_global, const Addr& out, T* mine, int pitch, long long e,
                                         long long lo, long long hi, RankOf rank_of) {
    if (to_global) {
        if (FULL || (e >= lo && e < hi)) {
#pragma unroll
            for (int i = 0; i < N; ++i) store_elem<T, 1, FULL>(out.ptr(rank_of(i)), e, lo, hi, v[i]);
        }
    } else {
#pragma unroll
        for (int i = 0; i < N; ++i) mine[rank_of(i) * pitch] = v[i].x[0];
    }
}

template <int L, int K, int T0, typename E>
__device__ __forceinline__ void ln_line_steps(E (&v)[L]) {      // distances 1, 3, .. (K of them) on a ring of L
    if constexpr (T0 < K) {
        reg_step<L, 1, L, ipow3(T0)>(v);
        ln_line_steps<L, K, T0 + 1>(v);
    }
}

template <typename T, int L, int K, bool FULL, typename Addr>
__device__ __forceinline__ void ln_line(const LnGroup& g, const short* bases, bool fg, bool tg, const Addr& in, const Addr& out,
                                        T* mine, int pitch, long long e, long long lo, long long hi, int set, int nslots) {   // pitch, nslots: constants after inlining
    for (int q = set; q < g.nsets; q += nslots) {
        const int r0 = bases[g.base_off + q], sa = g.stride_a;
        auto rank_of = [&](int i) { return r0 + i * sa; };
        Elem<T, 1> v[L];
        ln_load<T, L, FULL>(v, fg, in, mine, pitch, e, lo, hi, rank_of);
        ln_line_steps<L, K, 0>(v);
        ln_store<T, L, FULL>(v, tg, out, mine, pitch, e, lo, hi, rank_of);
    }
}

template <typename T, int LA, int LB, bool FULL, typename Addr>
__device__ __forceinline__ void ln_plane(const LnGroup& g, const short* bases, bool fg, bool tg, const Addr& in, const Addr& out,
                                         T* mine, int pitch, long long e, long long lo, long long hi, int set, int nslots) {   // pitch, nslots: constants after inlining
    for (int q = set; q < g.nsets; q += nslots) {
        const int r0 = bases[g.base_off + q], sa = g.stride_a, sb = g.stride_b;
        auto rank_of = [&](int idx) { return r0 + (idx % LA) * sa + (idx / LA) * sb; };
        Elem<T, 1> v[LA * LB];
        ln_load<T, LA * LB, FULL>(v, fg, in, mine, pitch, e, lo, hi, rank_of);
        reg_step<LA * LB, 1, LA, 1>(v);         // the step along the first dimension comes first in the schedule
        reg_step<LA * LB, LA, LB, 1>(v);
        ln_store<T, LA * LB, FULL>(v, tg, out, mine, pitch, e, lo, hi, rank_of);
    }
}

// The 9 x 9 plane group, streamed: rows of nine values along the first axis, the first step inside a row, the second
// over a sliding window of three rows -- 45 live values instead of 81 (which spill at two CTAs of 288 threads per SM).
// In place: row j + 1 is read before row j is overwritten, rows 0 and 1 are kept for the last two outputs.
template <typename T, bool FULL, typename Addr>
__device__ __forceinline__ void ln_plane99(const LnGroup& g, const short* bases, bool fg, bool tg, const Addr& in, const Addr& out,
                                           T* mine, int pitch, long long e, long long lo, long long hi, int set, int nslots) {
    using E = Elem<T, 1>;
    for (int q = set; q < g.nsets; q += nslots) {
        const int r0 = bases[g.base_off + q], sa = g.stride_a, sb = g.stride_b;
        auto load_row = [&](int j, E (&row)[9]) {
#pragma unroll
            for (int i = 0; i < 9; ++i) {
                const int rank = r0 + i * sa + j * sb;
                if (fg) row[i] = load_elem<T, 1, FULL>(in.ptr(rank), e, lo, hi);
                else row[i].x[0] = mine[rank * pitch];
            }
            reg_step<9, 1, 9, 1>(row);
        };
        auto emit = [&](int j, const E (&a)[9], const E (&b)[9], const E (&c)[9]) {
#pragma unroll
            for (int i = 0; i < 9; ++i) {
                const int rank = r0 + i * sa + j * sb;
                const E v = add3(a[i], b[i], c[i]);
                if (tg) { if (FULL || (e >= lo && e < hi)) store_elem<T, 1, FULL>(out.ptr(rank), e, lo, hi, v); }
                else mine[rank * pitch] = v.x[0];
            }
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
        emit(8, prev, cur, first);
        emit(0, cur, first, second);
    }
}

template <typename T, int CG, bool FULL, typename Addr>
__device__ __forceinline__ void ln_tile(const LnProgram& p, int c, const Addr& in, const Addr& out, T* slab, long long t0,
                                        long long lo, long long hi) {
    // thread = (lane, column group, set slot): tiles are 32 * cg columns wide so that a CTA has enough
    // work when n is small; the 9 warps split into cg column groups x 9 / cg set slots
    constexpr int cg = CG, nslots = kLnSets / cg, pitch = 32 * cg;
    const int lane = threadIdx.x % 32, col = (threadIdx.x / 32) % cg, set = threadIdx.x / (32 * cg);
    const long long e = t0 + col * 32 + lane;
    T* const mine = slab + col * 32 + lane;
    const int ng = p.ngroups[c];
    for (int gi = 0; gi < ng; ++gi) {
        const LnGroup& g = p.g[c][gi];
        const bool fg = gi == 0, tg = gi == ng - 1;
        const short* bases = p.bases[c];
#define LN_ARGS g, bases, fg, tg, in, out, mine, pitch, e, lo, hi, set, nslots
        if (g.kind == LN_LINE) {
            switch (g.la * 8 + g.nsteps) {
                case 3 * 8 + 1: ln_line<T, 3, 1, FULL>(LN_ARGS); break;
                case 9 * 8 + 1: ln_line<T, 9, 1, FULL>(LN_ARGS); break;
                case 9 * 8 + 2: ln_line<T, 9, 2, FULL>(LN_ARGS); break;
                case 27 * 8 + 1: ln_line<T, 27, 1, FULL>(LN_ARGS); break;
                case 27 * 8 + 2: ln_line<T, 27, 2, FULL>(LN_ARGS); break;
                case 27 * 8 + 3: ln_line<T, 27, 3, FULL>(LN_ARGS); break;
                case 81 * 8 + 1: ln_line<T, 81, 1, FULL>(LN_ARGS); break;
                case 81 * 8 + 2: ln_line<T, 81, 2, FULL>(LN_ARGS); break;
                case 81 * 8 + 3: ln_line<T, 81, 3, FULL>(LN_ARGS); break;
                case 81 * 8 + 4: ln_line<T, 81, 4, FULL>(LN_ARGS); break;
            }
        } else {
            switch (g.la * 100 + g.lb) {
                case 303: ln_plane<T, 3, 3, FULL>(LN_ARGS); break;
                case 309: ln_plane<T, 3, 9, FULL>(LN_ARGS); break;
                case 903: ln_plane<T, 9, 3, FULL>(LN_ARGS); break;
                case 909: ln_plane99<T, FULL>(LN_ARGS); break;
                case 327: ln_plane<T, 3, 27, FULL>(LN_ARGS); break;
                case 2703: ln_plane<T, 27, 3, FULL>(LN_ARGS); break;
            }
        }
#undef LN_ARGS
        if (!tg) __syncthreads();
    }
}

template <typename T, int CG, typename Addr>
__global__ void __launch_bounds__(32 * kLnSets, 2) k_lat_lines(Addr in, Addr out, LatArgs a, LnProgram p) {
    pdl_trigger();
    extern __shared__ uint4 slab_raw[];
    T* slab = reinterpret_cast<T*>(slab_raw);       // [n][32]
    const int c = blockIdx.y;                       // CTA-uniform from here on
    const long long lo = a.lo[c], hi = a.hi[c];
    constexpr int tw = 32 * CG;
    const long long t0 = (lo & ~31LL) + (long long)blockIdx.x * tw;
    if (t0 >= hi) return;
    pdl_wait();
    if (t0 >= lo && t0 + tw <= hi) ln_tile<T, CG, true>(p, c, in, out, slab, t0, lo, hi);
    else ln_tile<T, CG, false>(p, c, in, out, slab, t0, lo, hi);
}

template <typename T, int CG, typename Addr>
static trv_status_t launch_lines_cg(const Call& c, const Addr& in, const Addr& out, const LatArgs& a, const LnProgram& prog) {
    const Plan& p = *c.plan;
    long long tiles = 0;
    for (int sl = 0; sl < p.ndims; ++sl)
        if (a.hi[sl] > a.lo[sl]) {
            const long long tw = 32 * CG;
            const long long t = (a.hi[sl] - (a.lo[sl] & ~31LL) + tw - 1) / tw;
            if (t > tiles) tiles = t;
        }
    if (tiles == 0) return TRV_OK;
    auto kfn = k_lat_lines<T, CG, Addr>;
    if (!allow_big_smem(kfn, 729 * 32 * 4)) return TRV_ERR_CUDA;
    launch_pdl(kfn, dim3((unsigned)tiles, p.ndims, 1), dim3(32 * kLnSets), (size_t)p.n * 32 * CG * sizeof(T), c.st, in, out, a, prog);
    return TRV_OK;
}
#endif  // TRV_LN_PART > 0

// ------------------------------------------------------------------ host side

#if TRV_LN_PART == 0
static bool build_program(const Plan& p, LnProgram* prog);

bool fused_lines_supported(const Plan& p) {
    if (p.lines_prog) return true;
    if (p.general || p.algo != TRV_ALGO_TRIVANCE || p.variant != TRV_LATENCY_OPTIMAL) return false;
    if (p.n > 729 || p.ndims > kLnMaxD) return false;
    for (int d = 0; d < p.ndims; ++d)
        if (p.dims[d] > 81) return false;
    static thread_local LnProgram probe;        // every group of the plan must be one the kernel carries
    return build_program(p, &probe);
}

// The (kind, shape) pairs the kernel's dispatch switches carry; build_program refuses anything else, so a shape that
// a raised limit would let through can never fall through a switch unnoticed.
static bool plane_ok(int la, int lb) {
    return (la == 3 && (lb == 3 || lb == 9 || lb == 27)) || (la == 9 && (lb == 3 || lb == 9)) || (la == 27 && lb == 3);
}
static bool line_ok(int la, int nsteps) {
    int s = 0;
    for (int v = la; v > 1; v /= 3) { if (v % 3) return false; ++s; }
    return (la == 3 || la == 9 || la == 27 || la == 81) && nsteps >= 1 && nsteps <= s;
}

// base ranks of the sets {r0 + da*sa*i + db*sb*j}: all ranks whose coordinate along the set's
// dimensions is below the step distance (the other coordinates are free)
static int set_bases(const Plan& p, int dim_a, int dist_a, int dim_b, int dist_b, short* out) {
    int cnt = 0;
    for (int r = 0; r < p.n; ++r) {
        if (p.coord(r, dim_a) >= dist_a) continue;
        if (dim_b >= 0 && p.coord(r, dim_b) >= dist_b) continue;
        out[cnt++] = (short)r;
    }
    return cnt;
}

static bool build_program(const Plan& p, LnProgram* prog) {
    prog->n = p.n;
    prog->cg = p.n <= 81 ? 9 : 1;       // measured: 243 ranks run faster with 32-column tiles
    for (int c = 0; c < p.ndims; ++c) {
        const std::vector<Step>& st = p.steps[c];
        int ng = 0, nb = 0, i = 0;
        while (i < p.S) {
            if (ng >= kLnMaxGroups) return false;
            LnGroup& g = prog->g[c][ng];
            const int da = st[i].dim, xa = st[i].dist, la = p.dims[da] / xa;
            // steps of the same dimension that follow directly stay inside the same lines
            int k = 1;
            while (i + k < p.S && st[i + k].dim == da) ++k;
            if (k == 1 && i + 1 < p.S && st[i + 1].dim != da) {
                const int db = st[i + 1].dim, xb = st[i + 1].dist, lb = p.dims[db] / xb;
                const bool next_alone = !(i + 2 < p.S && st[i + 2].dim == db);     // else the next LINE would take it
                if (plane_ok(la, lb) && next_alone) {
                    g.kind = LN_PLANE; g.la = (short)la; g.lb = (short)lb; g.nsteps = 2;
                    g.stride_a = xa * p.stride[da]; g.stride_b = xb * p.stride[db];
                    g.base_off = nb;
                    if (nb + p.n / (la * lb) > kLnMaxBases) return false;
                    g.nsets = set_bases(p, da, xa, db, xb, prog->bases[c] + nb);
                    nb += g.nsets; ++ng; i += 2;
                    continue;
                }
            }
            if (!line_ok(la, k)) return false;
            g.kind = LN_LINE; g.la = (short)la; g.lb = 1; g.nsteps = (short)k;
            g.stride_a = xa * p.stride[da]; g.stride_b = 0;
            g.base_off = nb;
            if (nb + p.n / la > kLnMaxBases) return false;
            g.nsets = set_bases(p, da, xa, -1, 0, prog->bases[c] + nb);
            nb += g.nsets; ++ng; i += k;
        }
        prog->ngroups[c] = ng;
    }
    return true;
}
#endif  // TRV_LN_PART == 0

// one (element type, tile width) pair per translation unit
template <typename T, int CG>
trv_status_t launch_lines_part(const Call& c, const LatArgs& a, const LnProgram& prog);

#if TRV_LN_PART > 0
template <typename T, int CG>
trv_status_t launch_lines_part(const Call& c, const LatArgs& a, const LnProgram& prog) {
    const Plan& p = *c.plan;
    StrideAddr sin, sout;
    if (uniform_stride(c.in, p.n, &sin) && uniform_stride((const void* const*)c.out, p.n, &sout))
        return launch_lines_cg<T, CG>(c, sin, sout, a, prog);
    TabAddr<729> in, out;
    for (int r = 0; r < p.n; ++r) { in.t.p[r] = const_cast<void*>(c.in[r]); out.t.p[r] = c.out[r]; }
    return launch_lines_cg<T, CG>(c, in, out, a, prog);
}
#if TRV_LN_PART == 1
template trv_status_t launch_lines_part<float, 9>(const Call&, const LatArgs&, const LnProgram&);
#elif TRV_LN_PART == 2
template trv_status_t launch_lines_part<float, 1>(const Call&, const LatArgs&, const LnProgram&);
#elif TRV_LN_PART == 3
template trv_status_t launch_lines_part<uint32_t, 9>(const Call&, const LatArgs&, const LnProgram&);
#else
template trv_status_t launch_lines_part<uint32_t, 1>(const Call&, const LatArgs&, const LnProgram&);
#endif
#endif  // TRV_LN_PART > 0

#if TRV_LN_PART == 0
// once per plan (prepare_launch_data): the group list and the base ranks of all sets
void lines_prepare(Plan& p) {
    p.lines_prog.reset();
    if (!fused_lines_supported(p)) return;
    auto prog = std::make_shared<LnProgram>();
    if (build_program(p, prog.get())) p.lines_prog = prog;
}

trv_status_t run_fused_lines(const Call& c, const LatArgs& a) {
    const Plan& p = *c.plan;
    if (!p.lines_prog) return TRV_ERR_UNSUPPORTED;
    const LnProgram& prog = *static_cast<const LnProgram*>(p.lines_prog.get());
    trv_status_t st;
    if (c.dtype == TRV_FLOAT32) st = prog.cg == 9 ? launch_lines_part<float, 9>(c, a, prog) : launch_lines_part<float, 1>(c, a, prog);
    else st = prog.cg == 9 ? launch_lines_part<uint32_t, 9>(c, a, prog) : launch_lines_part<uint32_t, 1>(c, a, prog);
    if (st != TRV_OK) return st;
    return cudaGetLastError() == cudaSuccess ? TRV_OK : TRV_ERR_CUDA;
}
#endif

}  // namespace trv
