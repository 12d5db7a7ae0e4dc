// Per-step, per-directed-link load tally (Sec. 2.1: c_k; Fig. 1; App. E routing).
//
// In one schedule row every message of a collective travels inside ONE ring of one torus
// dimension, hop by hop in a fixed direction.  A message from ring position s that travels
// H hops in the + direction crosses the + links leaving s, s+1, ..., s+H-1; so the load of
// the + link leaving position i is a circular WINDOW SUM of the per-source weights over
// s = i-H+1 .. i (and over s = i .. i+H-1 for the - direction).  One warp owns one ring:
// it builds the circular prefix sums of the weights with shuffle scans and takes window
// sums as prefix differences.  A second kernel reduces the per-row maxima with warp
// reductions.  All integer work.
#include <vector>

#include "trv_dev.cuh"

namespace trv {

struct MsgClass {
    int dir;        // +1 / -1
    int hops;       // links crossed
    int delta;      // destination = source + delta (ring positions, wraps)
    int filter;     // 0: every source sends; 1: sources with (q & bit) == 0; 2: (q & bit) != 0, where q = pos,
    int bit;        //    or q = (size - pos) % size when `backwards` is set (a mirrored Recursive Doubling)
    int backwards;
    int plane;      // which of the two per-source weight arrays: bytes sent to the first / second peer
};
struct RowSlice {
    int dim, stride, size;      // the ring's dimension
    int nclass;
    MsgClass cls[2];
};

constexpr int kMaxRing = 1024;

__device__ __forceinline__ long long warp_scan_incl(long long v, int lane) {
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        long long u = __shfl_up_sync(0xffffffffu, v, o);
        if (lane >= o) v += u;
    }
    return v;
}

// grid: (rings of the row's dimension, slices, rows); block: one warp
__global__ void __launch_bounds__(32) k_link_tally(const RowSlice* __restrict__ desc, const long long* __restrict__ mbytes,
                                                   int n, int D, int NS, int* __restrict__ msgs, long long* __restrict__ bytes) {
    __shared__ long long P[kMaxRing];   // inclusive prefix of bytes by source position
    __shared__ int C[kMaxRing];         // inclusive prefix of message counts
    const int lane = threadIdx.x, c = blockIdx.y, row = blockIdx.z;
    const RowSlice rs = desc[row * NS + c];
    const int a = rs.size;
    if ((int)blockIdx.x >= n / a) return;
    // ring number -> rank of its position 0
    const int q = blockIdx.x;
    const int base = (q % rs.stride) + (q / rs.stride) * rs.stride * a;
    const long long* w0 = mbytes + ((size_t)row * NS + c) * 2 * n;

    for (int k = 0; k < rs.nclass; ++k) {
        const MsgClass mc = rs.cls[k];
        const long long* w = w0 + (size_t)mc.plane * n;
        long long carry = 0;
        int ccarry = 0;
        for (int s0 = 0; s0 < a; s0 += 32) {
            const int s = s0 + lane;
            long long wt = 0;
            int cnt = 0;
            if (s < a) {
                const int q = mc.backwards ? (a - s) % a : s;
                const bool sends = mc.filter == 0 || (mc.filter == 1 ? (q & mc.bit) == 0 : (q & mc.bit) != 0);
                if (sends) {
                    wt = w[base + s * rs.stride];
                    cnt = 1;
                }
            }
            const long long ps = warp_scan_incl(wt, lane) + carry;
            const int pc = (int)warp_scan_incl((long long)cnt, lane) + ccarry;
            if (s < a) { P[s] = ps; C[s] = pc; }
            carry = __shfl_sync(0xffffffffu, ps, 31);
            ccarry = __shfl_sync(0xffffffffu, pc, 31);
        }
        __syncwarp();
        const long long tot = carry;
        const int ctot = ccarry;
        for (int i = lane; i < a; i += 32) {
            long long lb;
            int lm;
            if (mc.dir > 0) {
                const int lo = i - mc.hops;     // window s = lo+1 .. i
                if (lo >= 0) { lb = P[i] - P[lo]; lm = C[i] - C[lo]; }
                else if (lo == -1) { lb = P[i]; lm = C[i]; }
                else { lb = P[i] + tot - P[lo + a]; lm = C[i] + ctot - C[lo + a]; }
            } else {
                const int hi = i + mc.hops - 1;  // window s = i .. hi
                const long long pb = i > 0 ? P[i - 1] : 0;
                const int pm = i > 0 ? C[i - 1] : 0;
                if (hi < a) { lb = P[hi] - pb; lm = C[hi] - pm; }
                else { lb = tot - pb + P[hi - a]; lm = ctot - pm + C[hi - a]; }
            }
            const size_t li = (((size_t)row * n + (base + i * rs.stride)) * D + rs.dim) * 2 + (mc.dir > 0 ? 0 : 1);
            if (lm) atomicAdd(&msgs[li], lm);
            if (lb) atomicAdd((unsigned long long*)&bytes[li], (unsigned long long)lb);
        }
        __syncwarp();
    }
}

// grid: rows; block: 256.  Max over the links of a row.
__global__ void __launch_bounds__(256) k_link_max(const int* __restrict__ msgs, const long long* __restrict__ bytes,
                                                  int links, int* __restrict__ max_msgs, long long* __restrict__ max_bytes) {
    __shared__ int sm[8];
    __shared__ long long sb[8];
    const int row = blockIdx.x;
    int m = 0;
    long long b = 0;
    for (int l = threadIdx.x; l < links; l += blockDim.x) {
        m = max(m, msgs[(size_t)row * links + l]);
        b = max(b, bytes[(size_t)row * links + l]);
    }
    m = __reduce_max_sync(0xffffffffu, m);
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) b = max(b, __shfl_xor_sync(0xffffffffu, b, o));
    if ((threadIdx.x & 31) == 0) { sm[threadIdx.x >> 5] = m; sb[threadIdx.x >> 5] = b; }
    __syncthreads();
    if (threadIdx.x < 32) {
        m = threadIdx.x < 8 ? sm[threadIdx.x] : 0;
        b = threadIdx.x < 8 ? sb[threadIdx.x] : 0;
        m = __reduce_max_sync(0xffffffffu, m);
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) b = max(b, __shfl_xor_sync(0xffffffffu, b, o));
        if (threadIdx.x == 0) { max_msgs[row] = m; max_bytes[row] = b; }
    }
}

trv_status_t run_link_loads(const Plan& p, size_t count, size_t elem_size, int32_t* msgs, int64_t* bytes,
                            int32_t* max_msgs, int64_t* max_bytes) {
    const int n = p.n, D = p.ndims, NS = p.nslices, T = p.rows();
    const size_t links = (size_t)n * D * 2;
    std::vector<RowSlice> desc((size_t)T * NS);
    std::vector<long long> mb((size_t)T * NS * 2 * n);  // [row][slice][peer number][source rank]
    int max_rings = 1;
    for (int row = 0; row < T; ++row) {
        for (int c = 0; c < NS; ++c) {
            const Step& st = p.steps[c][p.row_step(c, row)];
            RowSlice& rs = desc[(size_t)row * NS + c];
            rs.dim = st.dim; rs.stride = p.stride[st.dim]; rs.size = p.dims[st.dim];
            if (rs.size > kMaxRing) return TRV_ERR_UNSUPPORTED;
            if (n / rs.size > max_rings) max_rings = n / rs.size;
            const int d = st.dist;
            const int sg = d < 0 ? -1 : 1, ad = d < 0 ? -d : d;       // comparators: negative = mirrored collective
            if (p.general) {
                // a direction in which no block travels in this step carries no message at all
                const int t = p.step_of_row(row);
                bool any[2] = {false, false};
                for (int o = 1; o < n; ++o)
                    if (p.gstep[c][o] == t) any[(row < p.S) == (p.gsgn[c][o] > 0) ? 1 : 0] = true;
                rs.nclass = 0;
                if (any[0]) rs.cls[rs.nclass++] = MsgClass{-1, d, -d, 0, 0, 0, 0};
                if (any[1]) rs.cls[rs.nclass++] = MsgClass{+1, d, +d, 0, 0, 0, 1};
            } else if (p.algo == TRV_ALGO_TRIVANCE) {
                rs.nclass = 2;
                rs.cls[0] = MsgClass{-1, d, -d, 0, 0, 0, 0};
                rs.cls[1] = MsgClass{+1, d, +d, 0, 0, 0, 1};
            } else if (p.algo == TRV_ALGO_BRUCK) {
                rs.nclass = 2;
                rs.cls[0] = MsgClass{sg, ad, d, 0, 0, 0, 0};
                rs.cls[1] = MsgClass{sg, 2 * ad, 2 * d, 0, 0, 0, 1};
            } else if (p.algo == TRV_ALGO_SWING) {
                // even positions send to pos + d, odd ones to pos - d, each the short way round
                rs.nclass = 2;
                rs.cls[0] = MsgClass{sg, ad, d, 1, 1, 0, 0};
                rs.cls[1] = MsgClass{-sg, ad, -d, 2, 1, 0, 0};
            } else if (p.algo == TRV_ALGO_BUCKET) {
                rs.nclass = 1;
                rs.cls[0] = MsgClass{sg, 1, sg, 0, 0, 0, 0};
            } else {
                rs.nclass = 2;
                rs.cls[0] = MsgClass{sg, ad, d, 1, ad, sg < 0 ? 1 : 0, 0};
                rs.cls[1] = MsgClass{-sg, ad, -d, 2, ad, sg < 0 ? 1 : 0, 0};
            }
            static_assert(sizeof(long long) == sizeof(int64_t), "int64");
            for (int side = 0; side < 2; ++side)
                message_bytes_side(p, (int64_t)count, (int64_t)elem_size, c, row, side,
                                   (int64_t*)&mb[(((size_t)row * NS + c) * 2 + side) * n]);
        }
    }

    RowSlice* d_desc = nullptr;
    long long *d_mb = nullptr, *d_bytes = nullptr, *d_maxb = nullptr;
    int *d_msgs = nullptr, *d_maxm = nullptr;
    trv_status_t st = TRV_OK;
    auto ok = [&](cudaError_t e) { if (e != cudaSuccess && st == TRV_OK) st = TRV_ERR_CUDA; return e == cudaSuccess; };
    if (cudaMalloc(&d_desc, desc.size() * sizeof(RowSlice)) != cudaSuccess ||
        cudaMalloc(&d_mb, mb.size() * sizeof(long long)) != cudaSuccess ||
        cudaMalloc(&d_msgs, (size_t)T * links * sizeof(int)) != cudaSuccess ||
        cudaMalloc(&d_bytes, (size_t)T * links * sizeof(long long)) != cudaSuccess ||
        cudaMalloc(&d_maxm, (size_t)T * sizeof(int)) != cudaSuccess ||
        cudaMalloc(&d_maxb, (size_t)T * sizeof(long long)) != cudaSuccess) {
        (void)cudaGetLastError();
        st = TRV_ERR_ALLOC;
    }
    if (st == TRV_OK) {
        ok(cudaMemcpy(d_desc, desc.data(), desc.size() * sizeof(RowSlice), cudaMemcpyHostToDevice));
        ok(cudaMemcpy(d_mb, mb.data(), mb.size() * sizeof(long long), cudaMemcpyHostToDevice));
        ok(cudaMemset(d_msgs, 0, (size_t)T * links * sizeof(int)));
        ok(cudaMemset(d_bytes, 0, (size_t)T * links * sizeof(long long)));
    }
    if (st == TRV_OK) {
        dim3 grid(max_rings, NS, T);
        TRV_LAUNCH(k_link_tally, grid, 32, 0, 0, d_desc, d_mb, n, D, NS, d_msgs, d_bytes);
        TRV_LAUNCH(k_link_max, T, 256, 0, 0, d_msgs, d_bytes, (int)links, d_maxm, d_maxb);
        ok(cudaGetLastError());
        if (msgs) ok(cudaMemcpy(msgs, d_msgs, (size_t)T * links * sizeof(int), cudaMemcpyDeviceToHost));
        if (bytes) ok(cudaMemcpy(bytes, d_bytes, (size_t)T * links * sizeof(long long), cudaMemcpyDeviceToHost));
        if (max_msgs) ok(cudaMemcpy(max_msgs, d_maxm, (size_t)T * sizeof(int), cudaMemcpyDeviceToHost));
        if (max_bytes) ok(cudaMemcpy(max_bytes, d_maxb, (size_t)T * sizeof(long long), cudaMemcpyDeviceToHost));
        ok(cudaDeviceSynchronize());
    }
    cudaFree(d_desc); cudaFree(d_mb); cudaFree(d_msgs); cudaFree(d_bytes); cudaFree(d_maxm); cudaFree(d_maxb);
    g_last_kernel = "link_tally";
    return st;
}

}  // namespace trv
