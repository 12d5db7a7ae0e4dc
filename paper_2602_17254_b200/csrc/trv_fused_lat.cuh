// Pieces shared by the fused latency-form kernels: register-resident joint-reduction steps,
// tile loads/stores, launch arguments.
#pragma once
#include "trv_dev.cuh"

namespace trv {

constexpr int ipow3(int e) { return e <= 0 ? 1 : 3 * ipow3(e - 1); }
constexpr int ipow(int b, int e) { return e <= 0 ? 1 : b * ipow(b, e - 1); }
constexpr int ilog3(int n) { return n <= 1 ? 0 : 1 + ilog3(n / 3); }

// FULL is a compile-time property of the whole tile (every column of the CTA lies inside the
// slice): the common case is then straight-line code whose loads the compiler can batch; only the
// one or two edge tiles of a slice take the masked, element-by-element form.
template <typename T, int V, bool FULL>
__device__ __forceinline__ Elem<T, V> load_elem(const char* row, long long e, long long lo, long long hi) {
    const T* p = reinterpret_cast<const T*>(row);
    Elem<T, V> r;
    if constexpr (FULL) {
        r = *reinterpret_cast<const Elem<T, V>*>(p + e);
    } else {
#pragma unroll
        for (int k = 0; k < V; ++k) r.x[k] = (e + k >= lo && e + k < hi) ? p[e + k] : T(0);
    }
    return r;
}
template <typename T, int V, bool FULL>
__device__ __forceinline__ void store_elem(char* row, long long e, long long lo, long long hi, const Elem<T, V>& v) {
    T* p = reinterpret_cast<T*>(row);
    if constexpr (FULL) {
        *reinterpret_cast<Elem<T, V>*>(p + e) = v;
    } else {
#pragma unroll
        for (int k = 0; k < V; ++k)
            if (e + k >= lo && e + k < hi) p[e + k] = v.x[k];
    }
}

// One joint-reduction step on a register array: along the axis with flat stride STRIDE and ring
// length L, new[i] = (old[i - DIST] + old[i]) + old[i + DIST], indices modulo L.
template <int N, int STRIDE, int L, int DIST, typename E>
__device__ __forceinline__ void reg_step(E (&v)[N]) {
#pragma unroll
    for (int base = 0; base < N; ++base) {
        if ((base / STRIDE) % L != 0) continue;
        E line[L];
#pragma unroll
        for (int i = 0; i < L; ++i) line[i] = v[base + i * STRIDE];
#pragma unroll
        for (int i = 0; i < L; ++i) v[base + i * STRIDE] = add3(line[(i - DIST + L) % L], line[i], line[(i + DIST) % L]);
    }
}

struct LatArgs {
    int nslices;
    long long lo[TRV_MAX_DIMS], hi[TRV_MAX_DIMS];   // local element range of each slice
    int rs[TRV_MAX_DIMS][4];                        // rank stride of the slice's k-th dimension in its own order
};

trv_status_t run_fused_t999(const Call& c, const LatArgs& a);
bool run_fused_t999_tma(const Call& c, const LatArgs& a, trv_status_t* status);
bool run_fused_t999_wide(const Call& c, const LatArgs& a, trv_status_t* status);
bool run_fused_t2727_wide(const Call& c, const LatArgs& a, trv_status_t* status);
bool run_fused_t981_wide(const Call& c, const LatArgs& a, trv_status_t* status);
bool run_fused_r729_wide(const Call& c, const LatArgs& a, trv_status_t* status);
bool fused_lines_supported(const Plan& p);
void lines_prepare(Plan& p);
void latency_prepare(Plan& p);
trv_status_t run_fused_lines(const Call& c, const LatArgs& a);

}  // namespace trv
