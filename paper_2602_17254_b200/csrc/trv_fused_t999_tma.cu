// FUSED latency-optimal kernels for the 9 x 9 x 9 torus (Sec. 4.2, Sec. 5) whose tile moves by TMA.
//
// Same three closed groups as k_lat_t999 (trv_fused_t999.cu); both kernels need equally spaced rank buffers (tensor
// maps describe them as a matrix); other callers keep k_lat_t999.  Vectors from about 3 MiB per rank go to the
// persistent kernel on 64-column tiles (trv_fused_wide.cu) instead.
//   k_lat_t999_planes : the 32-column x 729-rank tile arrives as nine bulk tensor copies, one C-plane each, on nine
//                       mbarriers, so group 1 starts plane by plane; the results leave through bulk tensor stores,
//                       three planes after each phase of group 3.  729 x 32 MiB: 9.07 ms in a 0.7 s timed region under
//                       the power cap (1.8 GHz), 8.4 ms in a burst of five calls at 1.965 GHz.
//   k_lat_t999_tma    : three copies of 243 ranks on one mbarrier, results stored from registers (9.25 ms / 8.4 ms);
//                       kept for the case that the four-dimensional tensor maps cannot be encoded.
// Measured on the way (same workload, 0.7 s regions): the copy engine moving the tile in and straight out again with
// no arithmetic at all takes 8.16 ms with two 93 KB tiles per SM: that, not the adds, bounds this design.  Two columns
// per thread with packed adds and half the instructions: 9.35 ms.  Tiles of 64 columns, one persistent CTA per SM,
// with no overlap between a tile's arithmetic and the next tile's copies: 9.9 ms (with that overlap: the wide kernel).
// L2 prefetch of 1 KB-wide boxes ahead of the tiles, clusters of 2 to 8 adjacent tiles: no gain or worse.
// The plane-wise kernel made persistent, a tenth warp storing each finished phase and refilling its three planes with
// the NEXT tile at once (so that a CTA's copies in flight never drop to nothing between tiles): 11.6 ms -- the copy
// thread's wait for the engine to have read a phase before it may refill it serialises what two independent CTAs
// overlap by themselves.
// Every wait on a copy's mbarrier is bounded; a waiter that gives up counts it in a device-side counter (trv_tma.cuh)
// and the CTA leaves without storing.
#include "trv_dev.cuh"
#include "trv_fused_lat.cuh"
#include "trv_tma.cuh"

namespace trv {

__device__ unsigned int g_tma_giveups = 0;

template <int ROT>
struct RotT {
    static constexpr int sA = ROT == 0 ? 1 : (ROT == 1 ? 9 : 81);
    static constexpr int sB = ROT == 0 ? 9 : (ROT == 1 ? 81 : 1);
    static constexpr int sC = ROT == 0 ? 81 : (ROT == 1 ? 1 : 9);
};

template <typename T, int ROT, bool FULL, typename Addr>
__device__ __forceinline__ void t999_tma_body(const Addr& out, const LatArgs& a, T* slab, long long t0) {
    using R = RotT<ROT>;
    const int lane = threadIdx.x % 32, set = threadIdx.x / 32;
    const long long lo = a.lo[ROT], hi = a.hi[ROT];
    const long long e = t0 + lane;
    T* const mine = slab + lane;
    auto sl = [&](int r) -> T& { return mine[r * 32]; };
    {   // ---- group 1: (A,1) (B,1) on the plane C = set, row by row, in place
        const int r0 = set * R::sC;
        auto load_row = [&](int j, T (&row)[9]) {
#pragma unroll
            for (int i = 0; i < 9; ++i) row[i] = sl(r0 + i * R::sA + j * R::sB);
            reg_step<9, 1, 9, 1>(row);                                      // (A,1)
        };
        auto emit = [&](int j, const T (&p)[9], const T (&q)[9], const T (&r)[9]) {     // (B,1) for row j
#pragma unroll
            for (int i = 0; i < 9; ++i) sl(r0 + i * R::sA + j * R::sB) = add3(p[i], q[i], r[i]);
        };
        T first[9], second[9], prev[9], cur[9], next[9];
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
        emit(8, prev, cur, first);      // row 8 needs rows 7, 8, 0
        emit(0, cur, first, second);    // row 0 needs rows 8, 0, 1
    }
    __syncthreads();
    // ---- group 2: (C,1) (A,3); flat index k + 9 i  <->  rank (a0 + 3 i) sA + j sB + k sC
#pragma unroll 1
    for (int m = 0; m < 3; ++m) {
        const int q = set + 9 * m, r0 = (q % 3) * R::sA + (q / 3) * R::sB;
        T v[27];
#pragma unroll
        for (int idx = 0; idx < 27; ++idx) v[idx] = sl(r0 + 3 * (idx / 9) * R::sA + (idx % 9) * R::sC);
        reg_step<27, 1, 9, 1>(v);       // (C,1)
        reg_step<27, 9, 3, 1>(v);       // (A,3)
#pragma unroll
        for (int idx = 0; idx < 27; ++idx) sl(r0 + 3 * (idx / 9) * R::sA + (idx % 9) * R::sC) = v[idx];
    }
    __syncthreads();
    // ---- group 3: (B,3) (C,3); flat index jj + 3 kk  <->  rank i sA + (b0 + 3 jj) sB + (c0 + 3 kk) sC
    const bool live = FULL || (e >= lo && e < hi);
#pragma unroll 1
    for (int m = 0; m < 9; ++m) {
        const int q = set + 9 * m, r0 = (q % 9) * R::sA + ((q / 9) % 3) * R::sB + (q / 27) * R::sC;
        T v[9];
#pragma unroll
        for (int idx = 0; idx < 9; ++idx) v[idx] = sl(r0 + 3 * (idx % 3) * R::sB + 3 * (idx / 3) * R::sC);
        reg_step<9, 1, 3, 1>(v);        // (B,3)
        reg_step<9, 3, 3, 1>(v);        // (C,3)
        if (live) {
#pragma unroll
            for (int idx = 0; idx < 9; ++idx)
                reinterpret_cast<T*>(out.ptr(r0 + 3 * (idx % 3) * R::sB + 3 * (idx / 3) * R::sC))[e] = v[idx];
        }
    }
}

constexpr unsigned kTmaTileBytes = 729 * 32 * 4;

template <typename T>
__global__ void __launch_bounds__(288, 2) k_lat_t999_tma(const __grid_constant__ CUtensorMap tmap, StrideAddr out, LatArgs a,
                                                         unsigned* giveups) {
    extern __shared__ __align__(128) unsigned char smem_raw[];
    T* slab = reinterpret_cast<T*>(smem_raw);                           // [729][32]
    unsigned long long* bar = reinterpret_cast<unsigned long long*>(smem_raw + kTmaTileBytes);
    const int c = blockIdx.y;                                           // everything below is CTA-uniform
    const long long t0 = (a.lo[c] & ~31LL) + (long long)blockIdx.x * 32;
    if (t0 >= a.hi[c]) return;
    if (!tma_fetch_tile(&tmap, slab, bar, (int)t0, 3, 243, giveups)) return;     // gave up: counted, nothing stored
    const bool full = t0 >= a.lo[c] && t0 + 32 <= a.hi[c];
    if (c == 0) { if (full) t999_tma_body<T, 0, true>(out, a, slab, t0); else t999_tma_body<T, 0, false>(out, a, slab, t0); }
    else if (c == 1) { if (full) t999_tma_body<T, 1, true>(out, a, slab, t0); else t999_tma_body<T, 1, false>(out, a, slab, t0); }
    else { if (full) t999_tma_body<T, 2, true>(out, a, slab, t0); else t999_tma_body<T, 2, false>(out, a, slab, t0); }
}

// ------------------------------------------------------------------ plane by plane in, plane by plane out
//
// Same groups again, but the copy engine works plane by plane in both directions.  Each slice has its own tensor
// maps whose dimensions are ordered by increasing rank stride, with boxes of one C-plane (32 columns x 81 ranks):
// the tile lands plane-major, plane k = ranks with C = k, whatever the slice's rotation; inside a plane the A
// coordinate runs fastest (PA = 1, PB = 9) for the slices whose A stride is below their B stride, else B does
// (PA = 9, PB = 1).  Nine copies on nine mbarriers: warp k starts group 1 on plane k as soon as THAT plane is
// there.  Group 3 runs in three phases c0 = 0, 1, 2; a phase finishes the planes c0, c0 + 3, c0 + 6, writes them
// back into the slab and one thread hands them to the copy engine (bulk tensor stores), which drains them while
// the next phase computes.  The CTA leaves when the engine has read the last planes from shared memory.
// Tiles that are not wholly inside their slice store from registers with per-column masks instead.
template <typename T, int PA, bool FULL>
__device__ __forceinline__ void t999_planes_body(const CUtensorMap* omap, const StrideAddr& out, const LatArgs& a, int c, int cpos,
                                                 T* slab, unsigned long long* bars, long long t0, unsigned* giveups, int* gave_up) {
    constexpr int PB = PA == 1 ? 9 : 1, PC = 81;
    const int lane = threadIdx.x % 32, set = threadIdx.x / 32;
    const long long lo = a.lo[c], hi = a.hi[c];
    const long long e = t0 + lane;
    T* const mine = slab + lane;
    auto sl = [&](int r) -> T& { return mine[r * 32]; };
    {   // ---- group 1: (A,1) (B,1) on the plane C = set, as soon as it has arrived
        unsigned done = 0;
        const unsigned bar_s = smem_u32(bars + set);
        for (unsigned spins = 0; spins < kTmaWaitLimit; ++spins) {
            asm volatile(
                "{\n\t.reg .pred p;\n\tmbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\tselp.u32 %0, 1, 0, p;\n\t}"
                : "=r"(done)
                : "r"(bar_s), "r"(0)
                : "memory");
            if (done) break;
        }
        if (!done) *gave_up = 1;
        const int r0 = set * PC;
        auto load_row = [&](int j, T (&row)[9]) {
#pragma unroll
            for (int i = 0; i < 9; ++i) row[i] = sl(r0 + i * PA + j * PB);
            reg_step<9, 1, 9, 1>(row);                                      // (A,1)
        };
        auto emit = [&](int j, const T (&p)[9], const T (&q)[9], const T (&r)[9]) {     // (B,1) for row j
#pragma unroll
            for (int i = 0; i < 9; ++i) sl(r0 + i * PA + j * PB) = add3(p[i], q[i], r[i]);
        };
        T first[9], second[9], prev[9], cur[9], next[9];
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
    if (*gave_up) {                     // a wait ran out: counted once, nothing is stored
        if (threadIdx.x == 0) atomicAdd(giveups, 1u);
        return;
    }
    // ---- group 2: (C,1) (A,3) on the sets {A in a0 + 3 i, B = j, all C}; flat index k + 9 i
#pragma unroll 1
    for (int m = 0; m < 3; ++m) {
        const int q = set + 9 * m, r0 = (q % 3) * PA + (q / 3) * PB;
        T v[27];
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
#pragma unroll 1
    for (int c0 = 0; c0 < 3; ++c0) {
#pragma unroll
        for (int m = 0; m < 3; ++m) {       // unrolled: the three sets of a thread overlap their shared-memory round trips
            const int q = set + 9 * m, i = q % 9, b0 = q / 9;      // 27 sets of this phase: A = i, B in b0 + 3 jj
            const int r0 = i * PA + b0 * PB + c0 * PC;
            T v[9];
#pragma unroll
            for (int idx = 0; idx < 9; ++idx) v[idx] = sl(r0 + 3 * (idx % 3) * PB + 3 * (idx / 3) * PC);
            reg_step<9, 1, 3, 1>(v);        // (B,3)
            reg_step<9, 3, 3, 1>(v);        // (C,3)
            if constexpr (FULL) {
#pragma unroll
                for (int idx = 0; idx < 9; ++idx) sl(r0 + 3 * (idx % 3) * PB + 3 * (idx / 3) * PC) = v[idx];
            } else if (e >= lo && e < hi) {
                const int g0 = i * sA + b0 * sB + c0 * sC;
#pragma unroll
                for (int idx = 0; idx < 9; ++idx)
                    reinterpret_cast<T*>(out.ptr(g0 + 3 * (idx % 3) * sB + 3 * (idx / 3) * sC))[e] = v[idx];
            }
        }
        if constexpr (FULL) {
            __syncthreads();                // the three planes of this phase are complete in the slab
            if (threadIdx.x == 0) {
                asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
                for (int kk = 0; kk < 3; ++kk) {
                    const int k = c0 + 3 * kk;
                    asm volatile("cp.async.bulk.tensor.4d.global.shared::cta.bulk_group [%0, {%1, %2, %3, %4}], [%5];" ::"l"(omap),
                                 "r"((int)t0), "r"(cpos == 1 ? k : 0), "r"(cpos == 2 ? k : 0), "r"(cpos == 3 ? k : 0),
                                 "r"(smem_u32(slab) + k * PC * 128)
                                 : "memory");
                }
                asm volatile("cp.async.bulk.commit_group;" ::: "memory");
            }
        }
    }
    if constexpr (FULL) {
        if (threadIdx.x == 0) asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory");    // the slab may go once the engine has read it
    }
}

template <typename T>
__global__ void __launch_bounds__(288, 2) k_lat_t999_planes(const __grid_constant__ PlaneMaps maps, StrideAddr out, LatArgs a,
                                                            unsigned* giveups) {
    extern __shared__ __align__(128) unsigned char smem_raw[];
    T* slab = reinterpret_cast<T*>(smem_raw);                           // [9 planes][81][32]
    unsigned long long* bars = reinterpret_cast<unsigned long long*>(smem_raw + kTmaTileBytes);
    int* gave_up = reinterpret_cast<int*>(bars + 9);
    const int c = blockIdx.y;                                           // everything below is CTA-uniform
    const long long t0 = (a.lo[c] & ~31LL) + (long long)blockIdx.x * 32;
    if (t0 >= a.hi[c]) return;
    const int cpos = c == 0 ? 3 : (c == 1 ? 1 : 2);                     // where the C coordinate sits in the slice's tensor maps
    if (threadIdx.x == 0) {
        *gave_up = 0;
        for (int k = 0; k < 9; ++k) asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(bars + k)), "r"(1) : "memory");
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
        for (int k = 0; k < 9; ++k) {
            const unsigned bar_s = smem_u32(bars + k);
            asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar_s), "r"(81 * 128) : "memory");
            asm volatile(
                "cp.async.bulk.tensor.4d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3, %4, %5}], [%6];" ::"r"(
                    smem_u32(slab) + k * 81 * 128),
                "l"(&maps.in[c]), "r"((int)t0), "r"(cpos == 1 ? k : 0), "r"(cpos == 2 ? k : 0), "r"(cpos == 3 ? k : 0), "r"(bar_s)
                : "memory");
        }
    }
    __syncthreads();                    // the barriers are initialised before anybody polls them
    const bool full = t0 >= a.lo[c] && t0 + 32 <= a.hi[c];
    if (c == 2) {
        if (full) t999_planes_body<T, 9, true>(&maps.out[c], out, a, c, cpos, slab, bars, t0, giveups, gave_up);
        else t999_planes_body<T, 9, false>(&maps.out[c], out, a, c, cpos, slab, bars, t0, giveups, gave_up);
    } else {
        if (full) t999_planes_body<T, 1, true>(&maps.out[c], out, a, c, cpos, slab, bars, t0, giveups, gave_up);
        else t999_planes_body<T, 1, false>(&maps.out[c], out, a, c, cpos, slab, bars, t0, giveups, gave_up);
    }
}

// ------------------------------------------------------------------ host side

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*, const cuuint64_t*,
                                  const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                                  CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

static EncodeTiledFn encode_tiled_fn() {
    static EncodeTiledFn fn = []() -> EncodeTiledFn {
        void* p = nullptr;
        cudaDriverEntryPointQueryResult q;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) != cudaSuccess || q != cudaDriverEntryPointSuccess) {
            (void)cudaGetLastError();
            return nullptr;
        }
        return (EncodeTiledFn)p;
    }();
    return fn;
}

// A tiled map of 4-byte words, no swizzle, 256-byte L2 promotion; gstride has rank - 1 entries (bytes).
bool tma_encode_raw(CUtensorMap* out, int rank, void* base, const cuuint64_t* gdim, const cuuint64_t* gstride, const cuuint32_t* box) {
    EncodeTiledFn enc = encode_tiled_fn();
    if (!enc) return false;
    const cuuint32_t estride[5] = {1, 1, 1, 1, 1};
    return enc(out, CU_TENSOR_MAP_DATA_TYPE_UINT32, (cuuint32_t)rank, base, gdim, gstride, box, estride, CU_TENSOR_MAP_INTERLEAVE_NONE,
               CU_TENSOR_MAP_SWIZZLE_NONE, CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

bool tma_encode_ranks(const StrideAddr& in, int n, size_t count, int box_rows, CUtensorMap* out) {
    if ((in.stride & 15) || ((uintptr_t)in.base & 15) || count == 0 || count >= ((size_t)1 << 31)) return false;
    if (n > 1 && (size_t)in.stride < count * 4) return false;
    if (box_rows < 1 || box_rows > 256 || n % box_rows) return false;
    EncodeTiledFn enc = encode_tiled_fn();
    if (!enc) return false;
    const cuuint64_t gdim[2] = {(cuuint64_t)count, (cuuint64_t)n};
    const cuuint64_t gstride[1] = {(cuuint64_t)(n > 1 ? in.stride : ((count * 4 + 15) & ~(size_t)15))};
    const cuuint32_t box[2] = {32, (cuuint32_t)box_rows};
    const cuuint32_t estride[2] = {1, 1};
    return enc(out, CU_TENSOR_MAP_DATA_TYPE_UINT32, 2, in.base, gdim, gstride, box, estride, CU_TENSOR_MAP_INTERLEAVE_NONE,
               CU_TENSOR_MAP_SWIZZLE_NONE, CU_TENSOR_MAP_L2_PROMOTION_L2_128B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// Tensor map of one slice of the 9 x 9 x 9 torus over equally spaced rank buffers: dimensions (column, then the three
// torus dimensions ordered by increasing rank stride), boxes of box_cols columns x one C-plane.  strides[k] = rank
// stride of the slice's k-th dimension (A, B, C).
bool encode_planes(const StrideAddr& base, size_t count, const int strides[3], int box_cols, CUtensorMap* out) {
    if ((base.stride & 15) || ((uintptr_t)base.base & 15) || count == 0 || count >= ((size_t)1 << 31)) return false;
    if ((size_t)base.stride < count * 4) return false;
    EncodeTiledFn enc = encode_tiled_fn();
    if (!enc) return false;
    int order[3] = {0, 1, 2};
    for (int i = 0; i < 3; ++i)
        for (int j = i + 1; j < 3; ++j)
            if (strides[order[j]] < strides[order[i]]) { const int t = order[i]; order[i] = order[j]; order[j] = t; }
    cuuint64_t gdim[4] = {(cuuint64_t)count, 9, 9, 9};
    cuuint64_t gstride[3];
    cuuint32_t box[4] = {(cuuint32_t)box_cols, 9, 9, 9};
    const cuuint32_t estride[4] = {1, 1, 1, 1};
    for (int i = 0; i < 3; ++i) {
        gstride[i] = (cuuint64_t)strides[order[i]] * base.stride;
        if (order[i] == 2) box[1 + i] = 1;          // one C-plane per box
    }
    return enc(out, CU_TENSOR_MAP_DATA_TYPE_UINT32, 4, base.base, gdim, gstride, box, estride, CU_TENSOR_MAP_INTERLEAVE_NONE,
               CU_TENSOR_MAP_SWIZZLE_NONE, box_cols >= 64 ? CU_TENSOR_MAP_L2_PROMOTION_L2_256B : CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
               CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// false: this call cannot use the TMA kernels (the caller falls back to k_lat_t999)
bool run_fused_t999_tma(const Call& c, const LatArgs& a, trv_status_t* status) {
    StrideAddr sin, sout;
    if (!uniform_stride(c.in, 729, &sin) || !uniform_stride((const void* const*)c.out, 729, &sout)) return false;
    unsigned* giveups = tma_giveup_counter();
    if (!giveups) return false;
    long long tiles_x = 0;
    for (int sl = 0; sl < 3; ++sl)
        if (a.hi[sl] > a.lo[sl]) {
            const long long t = (a.hi[sl] - (a.lo[sl] & ~31LL) + 31) / 32;
            if (t > tiles_x) tiles_x = t;
        }
    if (tiles_x > (1LL << 30)) return false;
    PlaneMaps maps;
    bool planes = true;             // needs six four-dimensional tensor maps; else the whole-tile kernel below
    for (int sl = 0; sl < 3 && planes; ++sl)
        planes = encode_planes(sin, c.count, a.rs[sl], 32, &maps.in[sl]) && encode_planes(sout, c.count, a.rs[sl], 32, &maps.out[sl]);
    if (planes) {
        *status = TRV_OK;
        if (tiles_x == 0) return true;
        constexpr int psmem = (int)kTmaTileBytes + 9 * 8 + 16;
        g_last_kernel = "lat_t999_planes";
        if (c.dtype == TRV_FLOAT32) {
            if (!allow_big_smem(k_lat_t999_planes<float>, psmem)) { *status = TRV_ERR_CUDA; return true; }
            TRV_LAUNCH((k_lat_t999_planes<float>), dim3((unsigned)tiles_x, 3, 1), 288, psmem, c.st, maps, sout, a, giveups);
        } else {
            if (!allow_big_smem(k_lat_t999_planes<uint32_t>, psmem)) { *status = TRV_ERR_CUDA; return true; }
            TRV_LAUNCH((k_lat_t999_planes<uint32_t>), dim3((unsigned)tiles_x, 3, 1), 288, psmem, c.st, maps, sout, a, giveups);
        }
        if (cudaGetLastError() != cudaSuccess) *status = TRV_ERR_CUDA;
        return true;
    }
    CUtensorMap tmap;
    if (!tma_encode_ranks(sin, 729, c.count, 243, &tmap)) return false;
    *status = TRV_OK;
    if (tiles_x == 0) return true;
    constexpr int smem = (int)kTmaTileBytes + 16;
    g_last_kernel = "lat_t999_tma";
    if (c.dtype == TRV_FLOAT32) {
        if (!allow_big_smem(k_lat_t999_tma<float>, smem)) { *status = TRV_ERR_CUDA; return true; }
        TRV_LAUNCH((k_lat_t999_tma<float>), dim3((unsigned)tiles_x, 3, 1), 288, smem, c.st, tmap, sout, a, giveups);
    } else {
        if (!allow_big_smem(k_lat_t999_tma<uint32_t>, smem)) { *status = TRV_ERR_CUDA; return true; }
        TRV_LAUNCH((k_lat_t999_tma<uint32_t>), dim3((unsigned)tiles_x, 3, 1), 288, smem, c.st, tmap, sout, a, giveups);
    }
    if (cudaGetLastError() != cudaSuccess) *status = TRV_ERR_CUDA;
    return true;
}

unsigned* tma_giveup_counter() {
    void* p = nullptr;
    if (cudaGetSymbolAddress(&p, g_tma_giveups) != cudaSuccess) { (void)cudaGetLastError(); return nullptr; }
    return (unsigned*)p;
}

unsigned tma_giveups() {
    unsigned v = 0;
    if (cudaMemcpyFromSymbol(&v, g_tma_giveups, sizeof(v)) != cudaSuccess) return ~0u;
    return v;
}

}  // namespace trv
