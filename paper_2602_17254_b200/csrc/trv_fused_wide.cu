// FUSED latency-optimal kernels for the 729-rank shapes 9 x 9 x 9, 27 x 27, 9 x 81 / 81 x 9 and the ring of 729 (Sec. 4.2,
// Sec. 5) on tiles of 64 element columns, for long vectors: one persistent kernel, a shape policy for each.
//
// Why 64 columns: every tile touches all 729 input rows and all 729 output rows.  A plain copy that moves 128 bytes
// per row visit (32 columns) stops at 0.89 - 0.90 of the copy bandwidth on this part however many CTAs are resident,
// one that moves 256 bytes per visit reaches all of it; the 32-column kernels (trv_fused_t999_tma.cu) sit at that
// lower ceiling.  A 64-column tile of 729 ranks is 182 KB, so only one fits an SM, and the overlap that two resident
// CTAs gave for free has to come from inside one persistent CTA:
//   * a thread owns two adjacent columns (packed adds), a warp one row of 256 bytes;
//   * the tile arrives as nine plane copies of the copy engine on nine mbarriers (group 1 starts plane by plane);
//   * group 3 runs in three phases; a phase first pulls its three planes into registers, and as soon as every thread
//     has done so the copy engine refills those planes with the NEXT tile -- the slab never waits for the stores;
//   * the results go to HBM from registers (one 256-byte run per warp and rank) and drain while the next tile's
//     group 1 and 2 run.
// So loads are in flight during group 3 and the wait for the first planes, stores during groups 1 and 2.
// 729 x 32 MiB: 8.5 ms in a 0.6 s timed region under the power cap (1.7 GHz), against 9.05 ms for the 32-column kernel.
// Measured on the way and dropped: all of group 3's 81 values in registers before a single refill of nine planes
// (spills at 168 registers, 8.56 ms); eleven plane slots with the planes 2 and 5 of the tile after the next loading
// early (8.75 ms: the run-time slot arithmetic costs more than the two planes' head start gains).
// Asking the copy engine to bring the next tile's planes into L2 while groups 1 and 2 run (bulk tensor prefetch): slower
// on the same box (8.22 - 8.31 -> 8.62 - 8.64 ms).
// 9 x 9 x 9: the same three closed groups as the other 9 x 9 x 9 kernels: (A,1)(B,1) per C-plane, (C,1)(A,3), (B,3)(C,3).
// 27 x 27 (steps A1 B1 A3 B3 A9 B9): a plane is three A-lines (81 ranks); four groups: (A,1) on the 27-rank A-lines of a
// plane, (B,1) on the B-lines, (A,3)(B,3) on the nine 9 x 9 sets {A = a0 + 3 i, B = b0 + 3 j} streamed row by row, and
// (A,9)(B,9) on 3 x 3 sets in three phases whose planes are k0, k0 + 3, k0 + 6 -- the phase structure the refill needs.
// 27 x 27, 729 x 8 MiB: 3132 us with the line-group kernel -> 2400 us.  9 x 81 and the ring of 729: see their sections below.
// Every wait on a copy's mbarrier is bounded; a CTA that gives up counts it (trv_tma.cuh) and leaves without
// storing the tile it waited for.
#include <map>
#include <mutex>

#include "trv_dev.cuh"
#include "trv_fused_lat.cuh"
#include "trv_tma.cuh"

namespace trv {

// Tile scheduling.  With a fixed assignment (tile t, t + grid, ...) the slowest SM ends the kernel; handing out tiles from a
// counter instead is worth half a percent (three alternating runs each: 8.53 - 8.57 -> 8.50 - 8.51 ms).  The counter must
// belong to one launch at a time, and the call may allocate nothing, so the library keeps a small pool of counters per device and gives every (device, stream) pair its own:
// launches of one stream run one after the other, and the last CTA of a launch puts the counter back to zero.  Calls
// on the per-thread default stream (one handle, many streams), calls being captured into a graph (the graph may later
// run on any stream) and streams beyond the pool take the fixed assignment.
struct WideSched {
    unsigned next, done;
};
constexpr int kWideSchedSlots = 256;
__device__ WideSched g_wide_sched[kWideSchedSlots];

constexpr int kWideCols = 64;
constexpr unsigned kWidePlaneBytes = 81 * kWideCols * 4;
constexpr unsigned kWideTileBytes = 9 * kWidePlaneBytes;

struct WideTiles {
    long long nx[3];        // tiles of each slice
    long long total;
};

__device__ __forceinline__ void wide_locate(const WideTiles& w, const LatArgs& a, long long t, int* c, long long* t0) {
    int s = 0;
    while (s < 2 && t >= w.nx[s]) { t -= w.nx[s]; ++s; }        // nx[s] = 0 for slices the shape does not have
    *c = s;
    *t0 = (a.lo[s] & ~(long long)(kWideCols - 1)) + t * kWideCols;
}

__device__ __forceinline__ int wide_cpos(int c) { return c == 0 ? 3 : (c == 1 ? 1 : 2); }   // where C sits in the slice's maps

// one thread: plane k of the tile (c, t0) into its place in the slab, completing on bars[k]
__device__ __forceinline__ void wide_fetch_plane(const PlaneMaps& maps, int c, long long t0, int k, unsigned slab_s,
                                                 unsigned long long* bars) {
    const unsigned bar_s = smem_u32(bars + k);
    const int cpos = wide_cpos(c);
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar_s), "r"(kWidePlaneBytes) : "memory");
    asm volatile(
        "cp.async.bulk.tensor.4d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3, %4, %5}], [%6];" ::"r"(
            slab_s + k * kWidePlaneBytes),
        "l"(&maps.in[c]), "r"((int)t0), "r"(cpos == 1 ? k : 0), "r"(cpos == 2 ? k : 0), "r"(cpos == 3 ? k : 0), "r"(bar_s)
        : "memory");
}

// One tile.  PA = 1: inside a plane the A coordinate runs fastest, PA = 9: B does (see encode_planes).
// Returns false when a wait ran out (CTA-uniform).
template <typename T, int PA, bool FULL>
__device__ __forceinline__ bool wide_tile(const PlaneMaps& maps, const StrideAddr& out, const LatArgs& a, int c, long long t0,
                                          unsigned parity, bool has_next, int nc, long long nt0, T* slab, unsigned long long* bars,
                                          int* gave_up) {
    constexpr int PB = PA == 1 ? 9 : 1, PC = 81;
    using E = Elem<T, 2>;
    const int lane = threadIdx.x % 32, set = threadIdx.x / 32;
    const long long lo = a.lo[c], hi = a.hi[c];
    const long long e = t0 + 2 * lane;
    E* const mine = reinterpret_cast<E*>(slab) + lane;
    auto sl = [&](int r) -> E& { return mine[r * (kWideCols / 2)]; };
    {   // ---- group 1: (A,1) (B,1) on the plane C = set, as soon as it has arrived
        unsigned done = 0;
        const unsigned bar_s = smem_u32(bars + set);
        for (unsigned spins = 0; spins < kTmaWaitLimit; ++spins) {
            asm volatile(
                "{\n\t.reg .pred p;\n\tmbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\tselp.u32 %0, 1, 0, p;\n\t}"
                : "=r"(done)
                : "r"(bar_s), "r"(parity)
                : "memory");
            if (done) break;
        }
        if (!done) *gave_up = 1;
        const int r0 = set * PC;
        auto load_row = [&](int j, E (&row)[9]) {
#pragma unroll
            for (int i = 0; i < 9; ++i) row[i] = sl(r0 + i * PA + j * PB);
            reg_step<9, 1, 9, 1>(row);                                      // (A,1)
        };
        auto emit = [&](int j, const E (&p)[9], const E (&q)[9], const E (&r)[9]) {     // (B,1) for row j
#pragma unroll
            for (int i = 0; i < 9; ++i) sl(r0 + i * PA + j * PB) = add3(p[i], q[i], r[i]);
        };
        E first[9], second[9], prev[9], cur[9], next[9];
        load_row(0, first);
        load_row(1, second);
#pragma unroll
        for (int i = 0; i < 9; ++i) { prev[i] = first[i]; cur[i] = second[i]; }
#pragma unroll
        for (int j = 1; j < 8; ++j) {
            load_row(j + 1, next);          // row j + 1 is read before row j is overwritten
            emit(j, prev, cur, next);
#pragma unroll
            for (int i = 0; i < 9; ++i) { prev[i] = cur[i]; cur[i] = next[i]; }
        }
        emit(8, prev, cur, first);
        emit(0, cur, first, second);
    }
    __syncthreads();
    if (*gave_up) return false;
    // ---- group 2: (C,1) (A,3) on the sets {A in a0 + 3 i, B = j, all C}; flat index k + 9 i
#pragma unroll
    for (int m = 0; m < 3; ++m) {
        const int q = set + 9 * m, r0 = (q % 3) * PA + (q / 3) * PB;
        E v[27];
#pragma unroll
        for (int idx = 0; idx < 27; ++idx) v[idx] = sl(r0 + 3 * (idx / 9) * PA + (idx % 9) * PC);
        reg_step<27, 1, 9, 1>(v);       // (C,1)
        reg_step<27, 9, 3, 1>(v);       // (A,3)
#pragma unroll
        for (int idx = 0; idx < 27; ++idx) sl(r0 + 3 * (idx / 9) * PA + (idx % 9) * PC) = v[idx];
    }
    __syncthreads();
    // ---- group 3: (B,3) (C,3) on the sets {A = i, B in b0 + 3 jj, C in c0 + 3 kk}, phase by phase in c0
    const int sA = a.rs[c][0], sB = a.rs[c][1], sC = a.rs[c][2];
    const long long dB = 3LL * sB * out.stride, dC = 3LL * sC * out.stride;       // bytes between the rows of a set
    const unsigned slab_s = smem_u32(slab);
#pragma unroll                  // unrolled: a phase's slab reads move up past the previous phase's stores (8.30 -> 8.16 ms on one box)
    for (int c0 = 0; c0 < 3; ++c0) {
        E v[3][9];
#pragma unroll
        for (int m = 0; m < 3; ++m) {
            const int q = set + 9 * m, r0 = (q % 9) * PA + (q / 9) * PB + c0 * PC;
#pragma unroll
            for (int idx = 0; idx < 9; ++idx) v[m][idx] = sl(r0 + 3 * (idx % 3) * PB + 3 * (idx / 3) * PC);
        }
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");      // this thread's slab accesses before the engine's writes
        __syncthreads();                    // everybody holds its part of the planes c0, c0 + 3, c0 + 6: they may be refilled
        if (threadIdx.x == 0 && has_next) {
            for (int kk = 0; kk < 3; ++kk) wide_fetch_plane(maps, nc, nt0, c0 + 3 * kk, slab_s, bars);
        }
#pragma unroll
        for (int m = 0; m < 3; ++m) {
            const int q = set + 9 * m, g0 = (q % 9) * sA + (q / 9) * sB + c0 * sC;
            reg_step<9, 1, 3, 1>(v[m]);     // (B,3)
            reg_step<9, 3, 3, 1>(v[m]);     // (C,3)
            if (FULL || (e < hi && e + 2 > lo)) {
                // nine rows at rank offsets 3 jj sB + 3 kk sC: one base pointer per set, the rest by two byte strides
                char* row = out.ptr(g0);
#pragma unroll
                for (int kk = 0; kk < 3; ++kk) {
                    char* r = row;
#pragma unroll
                    for (int jj = 0; jj < 3; ++jj) {
                        store_elem<T, 2, FULL>(r, e, lo, hi, v[m][jj + 3 * kk]);
                        r += dB;
                    }
                    row += dC;
                }
            }
        }
    }
    return true;
}


// bounded wait of a warp for its plane of the current tile
__device__ __forceinline__ void wide_wait_plane(unsigned long long* bars, int k, unsigned parity, int* gave_up) {
    unsigned done = 0;
    const unsigned bar_s = smem_u32(bars + k);
    for (unsigned spins = 0; spins < kTmaWaitLimit; ++spins) {
        asm volatile(
            "{\n\t.reg .pred p;\n\tmbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\tselp.u32 %0, 1, 0, p;\n\t}"
            : "=r"(done)
            : "r"(bar_s), "r"(parity)
            : "memory");
        if (done) break;
    }
    if (!done) *gave_up = 1;
}

struct ShapeT999 {
    static constexpr int kSlices = 3;
    static bool encode(const StrideAddr& base, size_t count, const LatArgs& a, int sl, CUtensorMap* out) {
        return encode_planes(base, count, a.rs[sl], kWideCols, out);
    }
    __device__ static __forceinline__ void fetch(const PlaneMaps& maps, int c, long long t0, int k, unsigned slab_s,
                                                 unsigned long long* bars) {
        wide_fetch_plane(maps, c, t0, k, slab_s, bars);
    }
    template <typename T>
    __device__ static __forceinline__ bool tile(const PlaneMaps& maps, const StrideAddr& out, const LatArgs& a, int c, long long t0,
                                                bool full, unsigned parity, bool has_next, int nc, long long nt0, T* slab,
                                                unsigned long long* bars, int* gave_up) {
        if (c == 2)
            return full ? wide_tile<T, 9, true>(maps, out, a, c, t0, parity, has_next, nc, nt0, slab, bars, gave_up)
                        : wide_tile<T, 9, false>(maps, out, a, c, t0, parity, has_next, nc, nt0, slab, bars, gave_up);
        return full ? wide_tile<T, 1, true>(maps, out, a, c, t0, parity, has_next, nc, nt0, slab, bars, gave_up)
                    : wide_tile<T, 1, false>(maps, out, a, c, t0, parity, has_next, nc, nt0, slab, bars, gave_up);
    }
};

// ------------------------------------------------------------------ 27 x 27
//
// Slice c runs the steps (A,1) (B,1) (A,3) (B,3) (A,9) (B,9) with A = dimension c, B = the other one (Sec. 5).  Plane
// k = the three A-lines with B in 3k .. 3k + 2.  The slice's tensor map has the dimension with the smaller rank stride
// first, so a plane lands as [B - 3k][A] for slice 0 (PA = 1, PB = 27) and as [A][B - 3k] for slice 1 (PA = 3, PB = 1).
__device__ __forceinline__ void wide_fetch_plane_2727(const PlaneMaps& maps, int c, long long t0, int k, unsigned slab_s,
                                                      unsigned long long* bars) {
    const unsigned bar_s = smem_u32(bars + k);
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar_s), "r"(kWidePlaneBytes) : "memory");
    asm volatile(
        "cp.async.bulk.tensor.3d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3, %4}], [%5];" ::"r"(
            slab_s + k * kWidePlaneBytes),
        "l"(&maps.in[c]), "r"((int)t0), "r"(c == 1 ? 3 * k : 0), "r"(c == 0 ? 3 * k : 0), "r"(bar_s)
        : "memory");
}

template <typename T, int PA, bool FULL>
__device__ __forceinline__ bool wide_tile_2727(const PlaneMaps& maps, const StrideAddr& out, const LatArgs& a, int c, long long t0,
                                               unsigned parity, bool has_next, int nc, long long nt0, T* slab,
                                               unsigned long long* bars, int* gave_up) {
    constexpr int PB = PA == 1 ? 27 : 1, PK = 81;       // row of (A, B) in the slab: (B / 3) * PK + A * PA + (B % 3) * PB
    using E = Elem<T, 2>;
    const int lane = threadIdx.x % 32, set = threadIdx.x / 32;
    const long long lo = a.lo[c], hi = a.hi[c];
    const long long e = t0 + 2 * lane;
    E* const mine = reinterpret_cast<E*>(slab) + lane;
    auto sl = [&](int r) -> E& { return mine[r * (kWideCols / 2)]; };
    // ---- group 1: (A,1) on the three A-lines of the plane `set`, as soon as it has arrived
    wide_wait_plane(bars, set, parity, gave_up);
#pragma unroll 1
    for (int b = 0; b < 3; ++b) {
        const int r0 = set * PK + b * PB;
        E v[27];
#pragma unroll
        for (int i = 0; i < 27; ++i) v[i] = sl(r0 + i * PA);
        reg_step<27, 1, 27, 1>(v);
#pragma unroll
        for (int i = 0; i < 27; ++i) sl(r0 + i * PA) = v[i];
    }
    __syncthreads();
    if (*gave_up) return false;
    // ---- group 2: (B,1) on the B-lines A = set + 9 m
#pragma unroll 1
    for (int m = 0; m < 3; ++m) {
        const int r0 = (set + 9 * m) * PA;
        E v[27];
#pragma unroll
        for (int j = 0; j < 27; ++j) v[j] = sl(r0 + (j / 3) * PK + (j % 3) * PB);
        reg_step<27, 1, 27, 1>(v);
#pragma unroll
        for (int j = 0; j < 27; ++j) sl(r0 + (j / 3) * PK + (j % 3) * PB) = v[j];
    }
    __syncthreads();
    {   // ---- group 3: (A,3) (B,3) on the set {A = a0 + 3 i, B = b0 + 3 j}: a 9 x 9 torus, row j = plane j, streamed
        const int r0 = (set % 3) * PA + (set / 3) * PB;
        auto load_row = [&](int j, E (&row)[9]) {
#pragma unroll
            for (int i = 0; i < 9; ++i) row[i] = sl(r0 + 3 * i * PA + j * PK);
            reg_step<9, 1, 9, 1>(row);                                      // (A,3)
        };
        auto emit = [&](int j, const E (&p)[9], const E (&q)[9], const E (&r)[9]) {     // (B,3) for row j
#pragma unroll
            for (int i = 0; i < 9; ++i) sl(r0 + 3 * i * PA + j * PK) = add3(p[i], q[i], r[i]);
        };
        E first[9], second[9], prev[9], cur[9], next[9];
        load_row(0, first);
        load_row(1, second);
#pragma unroll
        for (int i = 0; i < 9; ++i) { prev[i] = first[i]; cur[i] = second[i]; }
#pragma unroll
        for (int j = 1; j < 8; ++j) {
            load_row(j + 1, next);          // row j + 1 is read before row j is overwritten
            emit(j, prev, cur, next);
#pragma unroll
            for (int i = 0; i < 9; ++i) { prev[i] = cur[i]; cur[i] = next[i]; }
        }
        emit(8, prev, cur, first);
        emit(0, cur, first, second);
    }
    __syncthreads();
    // ---- group 4: (A,9) (B,9) on the sets {A = a + 9 i, B = b + 9 j}; phase k0 takes the b with b / 3 = k0, whose planes are
    // k0, k0 + 3, k0 + 6; flat index i + 3 j
    const int sA = a.rs[c][0], sB = a.rs[c][1];
    const long long dA = 9LL * sA * out.stride, dB = 9LL * sB * out.stride;
    const unsigned slab_s = smem_u32(slab);
#pragma unroll
    for (int k0 = 0; k0 < 3; ++k0) {
        E v[3][9];
#pragma unroll
        for (int m = 0; m < 3; ++m) {
            const int q = set + 9 * m, r0 = (q % 9) * PA + (q / 9) * PB + k0 * PK;      // a = q % 9, b = 3 k0 + q / 9
#pragma unroll
            for (int idx = 0; idx < 9; ++idx) v[m][idx] = sl(r0 + 9 * (idx % 3) * PA + 3 * (idx / 3) * PK);
        }
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");      // this thread's slab accesses before the engine's writes
        __syncthreads();                    // everybody holds its part of the planes k0, k0 + 3, k0 + 6: they may be refilled
        if (threadIdx.x == 0 && has_next) {
            for (int kk = 0; kk < 3; ++kk) wide_fetch_plane_2727(maps, nc, nt0, k0 + 3 * kk, slab_s, bars);
        }
#pragma unroll
        for (int m = 0; m < 3; ++m) {
            const int q = set + 9 * m, g0 = (q % 9) * sA + (3 * k0 + q / 9) * sB;
            reg_step<9, 1, 3, 1>(v[m]);     // (A,9)
            reg_step<9, 3, 3, 1>(v[m]);     // (B,9)
            if (FULL || (e < hi && e + 2 > lo)) {
                char* row = out.ptr(g0);        // nine rows at rank offsets 9 i sA + 9 j sB: two byte strides from one base
#pragma unroll
                for (int j = 0; j < 3; ++j) {
                    char* r = row;
#pragma unroll
                    for (int i = 0; i < 3; ++i) {
                        store_elem<T, 2, FULL>(r, e, lo, hi, v[m][i + 3 * j]);
                        r += dA;
                    }
                    row += dB;
                }
            }
        }
    }
    return true;
}

static bool encode_planes_2727(const StrideAddr& base, size_t count, int slice, CUtensorMap* out);
struct Shape2727 {
    static constexpr int kSlices = 2;
    static bool encode(const StrideAddr& base, size_t count, const LatArgs&, int sl, CUtensorMap* out) { return encode_planes_2727(base, count, sl, out); }
    __device__ static __forceinline__ void fetch(const PlaneMaps& maps, int c, long long t0, int k, unsigned slab_s,
                                                 unsigned long long* bars) {
        wide_fetch_plane_2727(maps, c, t0, k, slab_s, bars);
    }
    template <typename T>
    __device__ static __forceinline__ bool tile(const PlaneMaps& maps, const StrideAddr& out, const LatArgs& a, int c, long long t0,
                                                bool full, unsigned parity, bool has_next, int nc, long long nt0, T* slab,
                                                unsigned long long* bars, int* gave_up) {
        if (c == 1)
            return full ? wide_tile_2727<T, 3, true>(maps, out, a, c, t0, parity, has_next, nc, nt0, slab, bars, gave_up)
                        : wide_tile_2727<T, 3, false>(maps, out, a, c, t0, parity, has_next, nc, nt0, slab, bars, gave_up);
        return full ? wide_tile_2727<T, 1, true>(maps, out, a, c, t0, parity, has_next, nc, nt0, slab, bars, gave_up)
                    : wide_tile_2727<T, 1, false>(maps, out, a, c, t0, parity, has_next, nc, nt0, slab, bars, gave_up);
    }
};

// ------------------------------------------------------------------ 9 x 81 and 81 x 9
//
// 9 x 81: rank = A + 9 B with A < 9, B < 81; write B = Bl + 9 Bh: the ranks form a 9 x 9 x 9 index space (A, Bl, Bh) with
// rank strides 1, 9, 81, and plane k = the ranks with Bl = k lands as [Bh][A] (row Bh * 9 + A: PA = 1).  81 x 9: rank =
// B + 81 A, strides 81, 1, 9, the plane lands as [A][Bh] (PA = 9).  The slice that starts with the side of 9 runs the steps
// A1 B1 A3 B3 B9 B27, the other one B1 A1 B3 A3 B9 B27 (Sec. 5).  Steps along B with distance 1 or 3 walk a ring of 81 or 27
// positions that crosses the planes: they are streamed as three-point stencils, nine positions at a time, in place.
// Groups: (A,1) on the 9-rank A-lines of a plane; (B,1) on the nine B-lines; (A,3)(B,3) on the nine sets
// {A = a0 + 3 i, B = b0 + 3 j}, streamed along j; (B,9)(B,27) on the 9-rank sets {A, Bl fixed}, which lie inside ONE plane:
// three phases of three planes each, as the refill wants them.
template <bool SWAP>
__device__ __forceinline__ void wide_fetch_plane_981(const PlaneMaps& maps, long long t0, int k, unsigned slab_s, unsigned long long* bars) {
    const unsigned bar_s = smem_u32(bars + k);
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar_s), "r"(kWidePlaneBytes) : "memory");
    asm volatile(
        "cp.async.bulk.tensor.4d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3, %4, %5}], [%6];" ::"r"(
            slab_s + k * kWidePlaneBytes),
        "l"(&maps.in[0]), "r"((int)t0), "r"(SWAP ? k : 0), "r"(SWAP ? 0 : k), "r"(0), "r"(bar_s)
        : "memory");
}

// One distance-1 step on a ring of L positions (L a multiple of 9), each position a row of W values, in place:
// out[i] = (row[i - 1] + row[i]) + row[i + 1] where row[i] = what load(i, .) delivers (the stored values BEFORE this step,
// possibly with a step of their own applied), handed to store(i, .).  Nine positions at a time: position i is stored
// only after positions up to i + 1 have been loaded, and positions 0 and 1 are kept for the wrap-around.
template <int L, int W, typename E, typename Load, typename Store>
__device__ __forceinline__ void wide_ring_stencil(Load load, Store store) {
    E first[W], second[W], a[W], b[W];
    load(0, first);
    load(1, second);
#pragma unroll
    for (int w = 0; w < W; ++w) { a[w] = first[w]; b[w] = second[w]; }
#pragma unroll
    for (int k = 0; k < L / 9; ++k) {
        E x[11][W];
#pragma unroll
        for (int w = 0; w < W; ++w) { x[0][w] = a[w]; x[1][w] = b[w]; }
#pragma unroll
        for (int m = 0; m < 9; ++m) {
            const int i = 9 * k + 2 + m;
            if (i < L) load(i, x[2 + m]);
            else {
#pragma unroll
                for (int w = 0; w < W; ++w) x[2 + m][w] = i == L ? first[w] : second[w];
            }
        }
#pragma unroll
        for (int m = 0; m < 9; ++m) {
            E o[W];
#pragma unroll
            for (int w = 0; w < W; ++w) o[w] = add3(x[m][w], x[m + 1][w], x[m + 2][w]);
            store((9 * k + 1 + m) % L, o);
        }
#pragma unroll
        for (int w = 0; w < W; ++w) { a[w] = x[9][w]; b[w] = x[10][w]; }
    }
}

// BFIRST = false: the slice A1 B1 A3 B3 B9 B27; true: B1 A1 B3 A3 B9 B27.  PA = 1: 9 x 81, PA = 9: 81 x 9.
template <typename T, int PA, bool BFIRST, bool FULL>
__device__ __forceinline__ bool wide_tile_981(const PlaneMaps& maps, const StrideAddr& out, const LatArgs& a, int c, long long t0,
                                              unsigned parity, bool has_next, long long nt0, T* slab, unsigned long long* bars,
                                              int* gave_up) {
    constexpr int PK = 81, PH = PA == 1 ? 9 : 1;        // row of (A, B) in the slab: (B % 9) * PK + (B / 9) * PH + A * PA
    using E = Elem<T, 2>;
    const int lane = threadIdx.x % 32, set = threadIdx.x / 32;
    const long long lo = a.lo[c], hi = a.hi[c];
    const long long e = t0 + 2 * lane;
    E* const mine = reinterpret_cast<E*>(slab) + lane;
    auto sl = [&](int r) -> E& { return mine[r * (kWideCols / 2)]; };
    auto a_lines = [&]() {              // (A,1) on the nine A-lines of the plane `set`
#pragma unroll 3
        for (int h = 0; h < 9; ++h) {
            E v[9];
#pragma unroll
            for (int i = 0; i < 9; ++i) v[i] = sl(set * PK + h * PH + i * PA);
            reg_step<9, 1, 9, 1>(v);
#pragma unroll
            for (int i = 0; i < 9; ++i) sl(set * PK + h * PH + i * PA) = v[i];
        }
    };
    auto b_lines = [&]() {              // (B,1) on the B-line A = set: a ring of 81 positions across the planes
        wide_ring_stencil<81, 1, E>([&](int i, E (&row)[1]) { row[0] = sl((i % 9) * PK + (i / 9) * PH + set * PA); },
                                    [&](int i, const E (&row)[1]) { sl((i % 9) * PK + (i / 9) * PH + set * PA) = row[0]; });
    };
    if (!BFIRST) {
        wide_wait_plane(bars, set, parity, gave_up);
        a_lines();
        __syncthreads();
        if (*gave_up) return false;
        b_lines();
    } else {
#pragma unroll 1
        for (int k = 0; k < 9; ++k) wide_wait_plane(bars, k, parity, gave_up);     // a B-line crosses every plane
        __syncthreads();
        if (*gave_up) return false;
        b_lines();
        __syncthreads();
        a_lines();
    }
    __syncthreads();
    {   // ---- (A,3) (B,3), or (B,3) (A,3), on the set {A = a0 + 3 i, B = b0 + 3 j}: rows of three values, ring of 27 rows
        const int a0 = set % 3, b0 = set / 3;
        auto row_at = [&](int j) { return (b0 + 3 * (j % 3)) * PK + (j / 3) * PH + a0 * PA; };       // B = b0 + 3 j
        wide_ring_stencil<27, 3, E>(
            [&](int j, E (&row)[3]) {
#pragma unroll
                for (int i = 0; i < 3; ++i) row[i] = sl(row_at(j) + 3 * i * PA);
                if (!BFIRST) reg_step<3, 1, 3, 1>(row);        // (A,3) comes before (B,3)
            },
            [&](int j, const E (&row)[3]) {
                E o[3];
#pragma unroll
                for (int i = 0; i < 3; ++i) o[i] = row[i];
                if (BFIRST) reg_step<3, 1, 3, 1>(o);           // (A,3) comes after (B,3)
#pragma unroll
                for (int i = 0; i < 3; ++i) sl(row_at(j) + 3 * i * PA) = o[i];
            });
    }
    __syncthreads();
    // ---- (B,9) (B,27) on the sets {A, Bl fixed, Bh = 0 .. 8}: inside the plane Bl; phase k0 takes the planes k0, k0 + 3, k0 + 6
    const int sA = a.rs[c][BFIRST ? 1 : 0], sB = a.rs[c][BFIRST ? 0 : 1];       // rank strides of the side of 9 and of the side of 81
    const long long d9 = 9LL * sB * out.stride;         // bytes between the rows of a set
    const unsigned slab_s = smem_u32(slab);
#pragma unroll
    for (int k0 = 0; k0 < 3; ++k0) {
        E v[3][9];
#pragma unroll
        for (int m = 0; m < 3; ++m) {
            const int q = set + 9 * m, r0 = (k0 + 3 * (q / 9)) * PK + (q % 9) * PA;     // A = q % 9, Bl = k0 + 3 (q / 9)
#pragma unroll
            for (int idx = 0; idx < 9; ++idx) v[m][idx] = sl(r0 + PH * idx);
        }
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");      // this thread's slab accesses before the engine's writes
        __syncthreads();                    // everybody holds its part of the planes k0, k0 + 3, k0 + 6: they may be refilled
        if (threadIdx.x == 0 && has_next) {
            for (int kk = 0; kk < 3; ++kk) wide_fetch_plane_981<PA == 9>(maps, nt0, k0 + 3 * kk, slab_s, bars);
        }
#pragma unroll
        for (int m = 0; m < 3; ++m) {
            const int q = set + 9 * m, g0 = (q % 9) * sA + (k0 + 3 * (q / 9)) * sB;
            reg_step<9, 1, 9, 1>(v[m]);     // (B,9): distance 1 in Bh
            reg_step<9, 1, 9, 3>(v[m]);     // (B,27): distance 3 in Bh
            if (FULL || (e < hi && e + 2 > lo)) {
                {
                    char* row = out.ptr(g0);
#pragma unroll
                    for (int idx = 0; idx < 9; ++idx) {
                        store_elem<T, 2, FULL>(row, e, lo, hi, v[m][idx]);
                        row += d9;
                    }
                }
            }
        }
    }
    return true;
}

template <bool SWAP>          // false: 9 x 81, true: 81 x 9
struct Shape981 {
    static constexpr int kSlices = 2;
    static bool encode(const StrideAddr& base, size_t count, const LatArgs&, int, CUtensorMap* out) {
        const int s981[3] = {1, 81, 9}, s819[3] = {81, 9, 1};       // A, Bh, and Bl in the place of the plane coordinate
        return encode_planes(base, count, SWAP ? s819 : s981, kWideCols, out);
    }
    __device__ static __forceinline__ void fetch(const PlaneMaps& maps, int c, long long t0, int k, unsigned slab_s,
                                                 unsigned long long* bars) {
        wide_fetch_plane_981<SWAP>(maps, t0, k, slab_s, bars);  // both slices read the same map
    }
    template <typename T>
    __device__ static __forceinline__ bool tile(const PlaneMaps& maps, const StrideAddr& out, const LatArgs& a, int c, long long t0,
                                                bool full, unsigned parity, bool has_next, int nc, long long nt0, T* slab,
                                                unsigned long long* bars, int* gave_up) {
        constexpr int PA = SWAP ? 9 : 1;
        if ((c == 1) != SWAP)           // the slice that starts with the side of 81
            return full ? wide_tile_981<T, PA, true, true>(maps, out, a, c, t0, parity, has_next, nt0, slab, bars, gave_up)
                        : wide_tile_981<T, PA, true, false>(maps, out, a, c, t0, parity, has_next, nt0, slab, bars, gave_up);
        return full ? wide_tile_981<T, PA, false, true>(maps, out, a, c, t0, parity, has_next, nt0, slab, bars, gave_up)
                    : wide_tile_981<T, PA, false, false>(maps, out, a, c, t0, parity, has_next, nt0, slab, bars, gave_up);
    }
};

// ------------------------------------------------------------------ ring of 729
//
// rank r = a + 9 b + 81 c: the index space and the plane (the ranks with b = k, landing as [c][a]) of the 9 x 81 shape.
// Steps 1 3 9 27 81 243.  Distance 1 and 3 walk the whole ring: warp w takes the 81 positions with c = w as an open
// segment whose halo (four positions on either side, the neighbouring warps' values) it reads before anybody stores, and
// runs both steps in one pass.  Distance 9 and 27 walk the ring of the 81 positions {a + 9 m} of one a (distance 1 and 3
// in m = b + 9 c): one ring per warp, the same two-step pass with the ring's own other end as the halo.  Distance 81 and 243 stay inside the 9-rank sets {a, b fixed}, which lie inside ONE plane:
// three phases of three planes.
//
// Two steps at once on an open segment of L positions (L a multiple of 9) with four halo positions on either side, in
// place: t[i] = (old[i - 1] + old[i]) + old[i + 1], then out[i] = (t[i - 3] + t[i]) + t[i + 3] -- a distance-1 step followed
// by a distance-3 step, both roundings as the two separate steps have them.  Nine outputs at a time; out[i] is stored
// after old[i + 12] has been loaded, and nothing at or before i is read again.
template <int L, typename E, typename Load, typename Store>
__device__ __forceinline__ void wide_seg_stencil13(Load load, Store store, const E (&left)[4], const E (&right)[4]) {
    auto old_at = [&](int i) { return i < 0 ? left[i + 4] : (i < L ? load(i) : right[i - L]); };     // i known at compile time
    E t6[6], o2[2];         // t[9k - 3 .. 9k + 2] and old[9k + 2], old[9k + 3]
    {
        E o[8];
#pragma unroll
        for (int i = 0; i < 8; ++i) o[i] = old_at(i - 4);
#pragma unroll
        for (int i = 0; i < 6; ++i) t6[i] = add3(o[i], o[i + 1], o[i + 2]);
        o2[0] = o[6]; o2[1] = o[7];
    }
#pragma unroll
    for (int k = 0; k < L / 9; ++k) {
        E o[11], t[15];
        o[0] = o2[0]; o[1] = o2[1];
#pragma unroll
        for (int m = 0; m < 9; ++m) o[2 + m] = old_at(9 * k + 4 + m);
#pragma unroll
        for (int i = 0; i < 6; ++i) t[i] = t6[i];
#pragma unroll
        for (int m = 0; m < 9; ++m) t[6 + m] = add3(o[m], o[m + 1], o[m + 2]);         // t[9k + 3 + m]
#pragma unroll
        for (int m = 0; m < 9; ++m) store(9 * k + m, add3(t[m], t[m + 3], t[m + 6]));  // t[9k + m - 3], t[9k + m], t[9k + m + 3]
#pragma unroll
        for (int i = 0; i < 6; ++i) t6[i] = t[9 + i];
        o2[0] = o[9]; o2[1] = o[10];
    }
}

template <typename T, bool FULL>
__device__ __forceinline__ bool wide_tile_729(const PlaneMaps& maps, const StrideAddr& out, const LatArgs& a, long long t0,
                                              unsigned parity, bool has_next, long long nt0, T* slab, unsigned long long* bars,
                                              int* gave_up) {
    constexpr int PK = 81;              // row of rank a + 9 b + 81 c in the slab: b * PK + c * 9 + a
    using E = Elem<T, 2>;
    const int lane = threadIdx.x % 32, set = threadIdx.x / 32;
    const long long lo = a.lo[0], hi = a.hi[0];
    const long long e = t0 + 2 * lane;
    E* const mine = reinterpret_cast<E*>(slab) + lane;
    auto sl = [&](int r) -> E& { return mine[r * (kWideCols / 2)]; };
    const int prev_c = (set + 8) % 9, next_c = (set + 1) % 9;
#pragma unroll 1
    for (int k = 0; k < 9; ++k) wide_wait_plane(bars, k, parity, gave_up);     // the ring crosses every plane
    {   // ---- distance 1, then 3: segment c = set, positions i = a + 9 b; halo: the last four positions of c - 1, the first four of c + 1
        E left[4], right[4];
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            left[i] = sl(8 * PK + prev_c * 9 + 5 + i);
            right[i] = sl(next_c * 9 + i);
        }
        __syncthreads();                // every halo is read before any segment is written
        if (*gave_up) return false;
        auto at = [&](int i) { return (i / 9) * PK + set * 9 + i % 9; };
        wide_seg_stencil13<81, E>([&](int i) { return sl(at(i)); }, [&](int i, const E& v) { sl(at(i)) = v; }, left, right);
    }
    __syncthreads();
    {   // ---- distance 9, then 27: the ring of the 81 positions m = b + 9 c with a = set -- a segment whose halo is its own other end
        auto at = [&](int m) { return (m % 9) * PK + (m / 9) * 9 + set; };
        E left[4], right[4];
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            left[i] = sl(at(77 + i));
            right[i] = sl(at(i));
        }
        wide_seg_stencil13<81, E>([&](int m) { return sl(at(m)); }, [&](int m, const E& v) { sl(at(m)) = v; }, left, right);
    }
    __syncthreads();
    // ---- distance 81, then 243, on the sets {a, b fixed, c = 0 .. 8}: inside the plane b; phase k0 takes the planes k0, k0 + 3, k0 + 6
    const long long d81 = 81LL * out.stride;            // bytes between the rows of a set
    const unsigned slab_s = smem_u32(slab);
#pragma unroll 1
    for (int k0 = 0; k0 < 3; ++k0) {       // not unrolled: with the two-step passes above this shape would spill
        E v[3][9];
#pragma unroll
        for (int m = 0; m < 3; ++m) {
            const int q = set + 9 * m, r0 = (k0 + 3 * (q / 9)) * PK + q % 9;       // a = q % 9, b = k0 + 3 (q / 9)
#pragma unroll
            for (int idx = 0; idx < 9; ++idx) v[m][idx] = sl(r0 + 9 * idx);
        }
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");      // this thread's slab accesses before the engine's writes
        __syncthreads();                    // everybody holds its part of the planes k0, k0 + 3, k0 + 6: they may be refilled
        if (threadIdx.x == 0 && has_next) {
            for (int kk = 0; kk < 3; ++kk) wide_fetch_plane_981<false>(maps, nt0, k0 + 3 * kk, slab_s, bars);
        }
#pragma unroll
        for (int m = 0; m < 3; ++m) {
            const int q = set + 9 * m, g0 = q % 9 + 9 * (k0 + 3 * (q / 9));
            reg_step<9, 1, 9, 1>(v[m]);     // distance 81
            reg_step<9, 1, 9, 3>(v[m]);     // distance 243
            if (FULL || (e < hi && e + 2 > lo)) {
                {
                    char* row = out.ptr(g0);
#pragma unroll
                    for (int idx = 0; idx < 9; ++idx) {
                        store_elem<T, 2, FULL>(row, e, lo, hi, v[m][idx]);
                        row += d81;
                    }
                }
            }
        }
    }
    return true;
}

struct Shape729 {
    static constexpr int kSlices = 1;
    static bool encode(const StrideAddr& base, size_t count, const LatArgs&, int, CUtensorMap* out) {
        const int strides[3] = {1, 81, 9};      // a, c, and b in the place of the plane coordinate
        return encode_planes(base, count, strides, kWideCols, out);
    }
    __device__ static __forceinline__ void fetch(const PlaneMaps& maps, int c, long long t0, int k, unsigned slab_s,
                                                 unsigned long long* bars) {
        wide_fetch_plane_981<false>(maps, t0, k, slab_s, bars);
    }
    template <typename T>
    __device__ static __forceinline__ bool tile(const PlaneMaps& maps, const StrideAddr& out, const LatArgs& a, int c, long long t0,
                                                bool full, unsigned parity, bool has_next, int nc, long long nt0, T* slab,
                                                unsigned long long* bars, int* gave_up) {
        return full ? wide_tile_729<T, true>(maps, out, a, t0, parity, has_next, nt0, slab, bars, gave_up)
                    : wide_tile_729<T, false>(maps, out, a, t0, parity, has_next, nt0, slab, bars, gave_up);
    }
};

template <typename T, typename Shape>
__global__ void __launch_bounds__(288, 1) k_lat_wide(const __grid_constant__ PlaneMaps maps, StrideAddr out, LatArgs a,
                                                     WideTiles w, unsigned* giveups, WideSched* sched) {
    extern __shared__ __align__(128) unsigned char smem_raw[];
    T* slab = reinterpret_cast<T*>(smem_raw);                           // [9 planes][81][64]
    unsigned long long* bars = reinterpret_cast<unsigned long long*>(smem_raw + kWideTileBytes);
    int* gave_up = reinterpret_cast<int*>(bars + 9);
    long long* next_tile = reinterpret_cast<long long*>(bars + 10);
    long long t = blockIdx.x;                                           // everything below is CTA-uniform
    if (t >= w.total) return;
    int c;
    long long t0;
    wide_locate(w, a, t, &c, &t0);
    if (threadIdx.x == 0) {
        *gave_up = 0;
        for (int k = 0; k < 9; ++k) asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(bars + k)), "r"(1) : "memory");
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
        for (int k = 0; k < 9; ++k) Shape::fetch(maps, c, t0, k, smem_u32(slab), bars);
    }
    __syncthreads();                    // the barriers are initialised before anybody polls them
    // the first tile is the CTA's own number; further ones are drawn from the counter (or t + grid without one), always one
    // tile ahead: what thread 0 draws at the top of an iteration is read at the top of the next, many barriers later
    auto draw = [&]() { return (long long)gridDim.x + atomicAdd(&sched->next, 1u); };
    auto leave = [&]() {                // the last CTA of the launch hands the counter back as it found it
        if (sched && threadIdx.x == 0 && atomicAdd(&sched->done, 1u) == gridDim.x - 1) {
            sched->next = 0;
            sched->done = 0;
        }
    };
    if (sched && threadIdx.x == 0) next_tile[0] = draw();
    __syncthreads();
    for (unsigned parity = 0;; parity ^= 1) {
        const long long tn = sched ? next_tile[parity] : t + gridDim.x;
        if (sched && threadIdx.x == 0) next_tile[parity ^ 1] = draw();
        const bool has_next = tn < w.total;
        int nc = 0;
        long long nt0 = 0;
        if (has_next) wide_locate(w, a, tn, &nc, &nt0);
        const bool full = t0 >= a.lo[c] && t0 + kWideCols <= a.hi[c];
        const bool ok = Shape::template tile<T>(maps, out, a, c, t0, full, parity, has_next, nc, nt0, slab, bars, gave_up);
        if (!ok) {                      // a wait ran out: counted once, this tile is not stored
            if (threadIdx.x == 0) atomicAdd(giveups, 1u);
            leave();
            return;
        }
        if (!has_next) {
            leave();
            return;
        }
        t = tn; c = nc; t0 = nt0;
    }
}

// The counter of (current device, stream), or NULL (fixed assignment).  Host-side bookkeeping only.
static WideSched* wide_sched_for(int dev, cudaStream_t st) {
    if (st == cudaStreamPerThread) return nullptr;
    cudaStreamCaptureStatus cap = cudaStreamCaptureStatusNone;
    if (cudaStreamIsCapturing(st, &cap) != cudaSuccess) { (void)cudaGetLastError(); return nullptr; }
    if (cap != cudaStreamCaptureStatusNone) return nullptr;
    if (st == cudaStreamLegacy) st = nullptr;                   // both name the legacy default stream
    void* base = nullptr;               // asked for in every call: a pointer kept from before a device reset would dangle
    if (cudaGetSymbolAddress(&base, g_wide_sched) != cudaSuccess) { (void)cudaGetLastError(); return nullptr; }
    static std::mutex mu;
    static std::map<int, std::map<cudaStream_t, int>> slots;    // per device: stream -> counter number
    std::lock_guard<std::mutex> lock(mu);
    std::map<cudaStream_t, int>& d = slots[dev];
    auto it = d.find(st);
    if (it == d.end()) {
        if ((int)d.size() >= kWideSchedSlots) return nullptr;
        it = d.emplace(st, (int)d.size()).first;
    }
    return (WideSched*)base + it->second;
}

// false: this call cannot use the wide kernel (the caller goes on to the 32-column kernels)
template <typename Shape>
static bool run_wide(const Call& c, const LatArgs& a, const char* name, trv_status_t* status) {
    constexpr int NS = Shape::kSlices;
    StrideAddr sin, sout;
    if (!uniform_stride(c.in, 729, &sin) || !uniform_stride((const void* const*)c.out, 729, &sout)) return false;
    if ((sout.stride & 7) || ((uintptr_t)sout.base & 7)) return false;      // two-column stores
    WideTiles w;
    w.total = 0;
    long long local = 0;            // elements of this call's window, all slices
    for (int sl = 0; sl < 3; ++sl) {
        w.nx[sl] = 0;
        if (sl >= NS || a.hi[sl] <= a.lo[sl]) continue;
        local += a.hi[sl] - a.lo[sl];
        w.nx[sl] = (a.hi[sl] - (a.lo[sl] & ~(long long)(kWideCols - 1)) + kWideCols - 1) / kWideCols;
        w.total += w.nx[sl];
    }
    int dev = 0, sms = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || sms < 1)
        return false;
    // From about 3 MiB per rank on (9 x 9 x 9: 4 MiB per rank 1155 -> 1084 us, 8 MiB 2314 -> 2156 us, 32 MiB 9.05 -> 8.5 ms; at
    // 2 MiB the two kernels tie, below it the 32-column kernels win: more, smaller tiles to spread over the SMs).
    // 27 x 27 has no 32-column TMA kernel to fall back to, only the line-group kernel, and wins from 256 KiB per rank on
    // (64 Ki elements: 114 -> 91 us; 512 Ki: 811 -> 611 us; 2 Mi: 3132 -> 2400 us; 8 Mi: 9.44 ms, 0.79 of the copy bandwidth).
    if (local < (NS == 3 ? (3LL << 18) : (1LL << 16)) || w.total < 2LL * sms || w.total > (1LL << 30)) return false;
    unsigned* giveups = tma_giveup_counter();
    if (!giveups) return false;
    PlaneMaps maps;
    for (int sl = 0; sl < NS; ++sl) {
        if (!Shape::encode(sin, c.count, a, sl, &maps.in[sl])) return false;
    }
    *status = TRV_OK;
    constexpr int smem = (int)kWideTileBytes + 9 * 8 + 16 + 24;
    g_last_kernel = name;
    const unsigned grid = (unsigned)(w.total < sms ? w.total : sms);
    WideSched* sched = wide_sched_for(dev, c.st);
    if (c.dtype == TRV_FLOAT32) {
        if (!allow_big_smem(k_lat_wide<float, Shape>, smem)) { *status = TRV_ERR_CUDA; return true; }
        TRV_LAUNCH((k_lat_wide<float, Shape>), dim3(grid), 288, smem, c.st, maps, sout, a, w, giveups, sched);
    } else {
        if (!allow_big_smem(k_lat_wide<uint32_t, Shape>, smem)) { *status = TRV_ERR_CUDA; return true; }
        TRV_LAUNCH((k_lat_wide<uint32_t, Shape>), dim3(grid), 288, smem, c.st, maps, sout, a, w, giveups, sched);
    }
    if (cudaGetLastError() != cudaSuccess) *status = TRV_ERR_CUDA;
    return true;
}

bool run_fused_t999_wide(const Call& c, const LatArgs& a, trv_status_t* status) { return run_wide<ShapeT999>(c, a, "lat_t999_wide", status); }

// 27 x 27 with rank = x0 + 27 x1 (the plan's layout); false: not this shape or not this call
bool run_fused_t2727_wide(const Call& c, const LatArgs& a, trv_status_t* status) {
    const Plan& p = *c.plan;
    if (p.ndims != 2 || p.dims[0] != 27 || p.dims[1] != 27 || p.stride[0] != 1 || p.stride[1] != 27) return false;
    return run_wide<Shape2727>(c, a, "lat_t27x27_wide", status);
}

// the ring of 729; false: not this shape or not this call
bool run_fused_r729_wide(const Call& c, const LatArgs& a, trv_status_t* status) {
    const Plan& p = *c.plan;
    if (p.ndims != 1 || p.n != 729) return false;
    return run_wide<Shape729>(c, a, "lat_ring729_wide", status);
}

// 9 x 81 (rank = x0 + 9 x1) and 81 x 9 (rank = x0 + 81 x1); false: not these shapes or not this call
bool run_fused_t981_wide(const Call& c, const LatArgs& a, trv_status_t* status) {
    const Plan& p = *c.plan;
    if (p.ndims != 2 || p.stride[0] != 1) return false;
    if (p.dims[0] == 9 && p.dims[1] == 81 && p.stride[1] == 9) return run_wide<Shape981<false>>(c, a, "lat_t9x81_wide", status);
    if (p.dims[0] == 81 && p.dims[1] == 9 && p.stride[1] == 81) return run_wide<Shape981<true>>(c, a, "lat_t81x9_wide", status);
    return false;
}

// Tensor map of one slice of the 27 x 27 torus over equally spaced rank buffers: dimensions (column, then the two torus
// dimensions by increasing rank stride), boxes of 64 columns x 27 along the slice's own dimension x 3 along the other.
static bool encode_planes_2727(const StrideAddr& base, size_t count, int slice, CUtensorMap* out) {
    if ((base.stride & 15) || ((uintptr_t)base.base & 15) || count == 0 || count >= ((size_t)1 << 31)) return false;
    if ((size_t)base.stride < count * 4) return false;
    const cuuint64_t gdim[3] = {(cuuint64_t)count, 27, 27};
    const cuuint64_t gstride[2] = {(cuuint64_t)base.stride, (cuuint64_t)27 * base.stride};
    const cuuint32_t box[3] = {(cuuint32_t)kWideCols, slice == 0 ? 27u : 3u, slice == 0 ? 3u : 27u};
    return tma_encode_raw(out, 3, base.base, gdim, gstride, box);
}

}  // namespace trv
