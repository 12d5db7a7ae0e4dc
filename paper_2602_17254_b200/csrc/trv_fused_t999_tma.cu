// FUSED latency-optimal kernel for the 9 x 9 x 9 torus (Sec. 4.2, Sec. 5): the tile arrives by TMA.
//
// Same three closed groups as k_lat_t999 (trv_fused_t999.cu), but the 32-column x 729-rank tile is
// fetched by three bulk tensor copies (cp.async.bulk.tensor, boxes of 32 columns x 243 ranks) that one
// thread issues; the whole 93 KB of a tile are then in flight at once instead of nine loads per thread
// at a time, and group 1 runs on shared memory like the other two.  Needs equally spaced rank buffers
// (one tensor map describes them as a [729][count] matrix); other callers keep k_lat_t999.
// The wait on the copy's mbarrier is bounded; a waiter that gives up counts it in a device-side
// counter (trv_tma.cuh) and the CTA leaves without storing.
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

// false: this call cannot use the TMA kernel (the caller falls back to k_lat_t999)
bool run_fused_t999_tma(const Call& c, const LatArgs& a, trv_status_t* status) {
    StrideAddr sin, sout;
    if (!uniform_stride(c.in, 729, &sin) || !uniform_stride((const void* const*)c.out, 729, &sout)) return false;
    CUtensorMap tmap;
    if (!tma_encode_ranks(sin, 729, c.count, 243, &tmap)) return false;
    unsigned* giveups = tma_giveup_counter();
    if (!giveups) return false;
    long long tiles_x = 0;
    for (int sl = 0; sl < 3; ++sl)
        if (a.hi[sl] > a.lo[sl]) {
            const long long t = (a.hi[sl] - (a.lo[sl] & ~31LL) + 31) / 32;
            if (t > tiles_x) tiles_x = t;
        }
    *status = TRV_OK;
    if (tiles_x == 0) return true;
    if (tiles_x > (1LL << 30)) return false;
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
