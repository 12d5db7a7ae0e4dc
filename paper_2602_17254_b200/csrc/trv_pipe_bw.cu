// PIPELINED kernel family, bandwidth-optimal form: Reduce-Scatter and AllGather run by the chunk-level
// readiness engine of App. D ("one work descriptor per rank, step and chunk, containing both peer connections,
// buffer offsets, the active block range and the element count"), emulated inside one GPU.
//
// A chunk is a piece of ONE block of one collective (at most chunk_elems elements), so a chunk's active block
// range is that block.  A work item is (row, rank, chunk):
//   Reduce-Scatter row t : rank p, for a chunk of a block j it still answers for (j = p modulo 3^(visits so far) in
//                          every dimension, Sec. 4.3), adds (from_left + own) + from_right.  All ranks share one
//                          address space, so the peers' partials ARE the receive slots: the item reads them where
//                          they lie.  It is executable when the chunk's readiness entries of the left peer, the right
//                          peer and the rank itself all show t finished steps: the two-receive condition.
//   AllGather row        : rank p copies the finished chunk from the peer that holds it; executable when that peer's
//                          entry shows the final value (S).
// Everything runs in place in the output buffers (step 0 reads the inputs): the blocks a rank writes in a step are
// never the blocks its peers read from it in that step (Sec. 4.1: they lie in different residue classes), and a rank
// overwrites a stale partial in the AllGather only after the owner's final value exists, which needed that partial.
//
// Scheduling, generation and bounded waits are those of the latency-form engine (trv_pipe.cu): one persistent kernel,
// every warp a worker drawing tickets in an order in which an item follows the items it waits for (groups of chunks;
// inside a group row by row); a memset node zeroes ticket, error flag and entries; every wait gives up after
// kSpinLimit polls with TRV_ERR_TIMEOUT in the scratch header.
#include "trv_dev.cuh"
#include "trv_wait.cuh"

namespace trv {

constexpr int kPbThreads = 256;
constexpr int kPbMaxS = 8;
constexpr int kPbMaxD = 4;

struct PipeBwArgs {
    int n, S, D, nsub, group;               // sub-chunks per block; chunks per group
    int chunk_elems;
    unsigned spin_limit;
    long long nchunks;                      // D * n * nsub
    long long w0, w1;                       // the buffers hold global elements [w0, w1)
    long long slo[kPbMaxD], shi[kPbMaxD];   // the collectives' slices (global)
    int dims[kPbMaxD], stride[kPbMaxD];
    int sdim[kPbMaxD][kPbMaxS], sdist[kPbMaxD][kPbMaxS];
    int mod[kPbMaxD][kPbMaxS][kPbMaxD];     // 3^(visits of dimension d up to and including step t)
    int cnt[2 * kPbMaxS];                   // items per chunk in a row
    int* done;                              // readiness entries [chunk][rank]
    PipeHeader* hdr;
};

// the i-th rank (i < n / 3^(t+1)) that still answers for block j after Reduce-Scatter step t of collective c
__device__ __forceinline__ int pb_active_rank(const PipeBwArgs& a, int c, int t, int j, int i) {
    int p = 0;
#pragma unroll
    for (int d = 0; d < kPbMaxD; ++d)
        if (d < a.D) {
            const int m = a.mod[c][t][d], per = a.dims[d] / m;
            const int jd = (j / a.stride[d]) % a.dims[d];
            p += ((jd % m) + m * (i % per)) * a.stride[d];
            i /= per;
        }
    return p;
}
__device__ __forceinline__ int pb_shift(const PipeBwArgs& a, int p, int d, int delta) {
    const int size = a.dims[d], st = a.stride[d], x = (p / st) % size;
    int y = x + delta;
    if (y < 0) y += size;
    if (y >= size) y -= size;
    return p + (y - x) * st;
}

template <typename T, int CAP>
__global__ void __launch_bounds__(kPbThreads) k_bw_pipe(PtrTab<CAP> in, PtrTab<CAP> out, PipeBwArgs a) {
    using V = typename Vec4<T>::type;
    constexpr unsigned kFull = 0xffffffffu;
    const int lane = threadIdx.x & 31;
    int per_chunk = 0;
    for (int r = 0; r < 2 * a.S; ++r) per_chunk += a.cnt[r];
    const long long total = a.nchunks * per_chunk;
    for (;;) {
        long long item = 0;
        if (lane == 0) item = (long long)atomicAdd(&a.hdr->ticket, 1ULL);
        item = __shfl_sync(kFull, item, 0);
        if (item >= total) break;
        // item -> (group, row, chunk, index among the row's ranks for that chunk)
        const long long gsz = (long long)a.group * per_chunk;
        const long long g = item / gsz;
        const long long kg = min((long long)a.group, a.nchunks - g * a.group);     // chunks in this group
        long long local = item - g * gsz;
        int row = 0;
        while (local >= kg * a.cnt[row]) { local -= kg * a.cnt[row]; ++row; }
        const long long chunk = g * a.group + local / a.cnt[row];
        const int i = (int)(local % a.cnt[row]);
        const int c = (int)(chunk / ((long long)a.n * a.nsub));
        const int j = (int)((chunk / a.nsub) % a.n), s = (int)(chunk % a.nsub);
        // the chunk's elements: piece s of block j of collective c, cut to the window the buffers hold
        const unsigned long long len = (unsigned long long)(a.shi[c] - a.slo[c]);
        long long e0 = a.slo[c] + (long long)(((unsigned long long)j * len) / (unsigned)a.n);
        long long e1 = a.slo[c] + (long long)(((unsigned long long)(j + 1) * len) / (unsigned)a.n);
        e0 += (long long)s * a.chunk_elems;
        if (e1 > e0 + a.chunk_elems) e1 = e0 + a.chunk_elems;
        e0 = max(e0, a.w0) - a.w0;
        e1 = min(e1, a.w1) - a.w0;

        const bool rs = row < a.S;
        const int t = rs ? row : 2 * a.S - 1 - row;
        const int d = a.sdim[c][t], dist = a.sdist[c][t];
        int p, pl = 0, pr = 0, q = 0;
        if (rs) {
            p = pb_active_rank(a, c, t, j, i);
            pl = pb_shift(a, p, d, -dist);
            pr = pb_shift(a, p, d, dist);
        } else {        // the holders before this row answer for j after step t; each hands it to both peers
            const int holders = a.cnt[row] / 2;
            q = pb_active_rank(a, c, t, j, i % holders);
            p = pb_shift(a, q, d, i < holders ? -dist : dist);
        }
        int* const entries = a.done + (size_t)chunk * a.n;

        // ---- readiness
        int ok = 1;
        if (rs) {
            if (t > 0 && lane < 3) ok = wait_entry(entries + (lane == 0 ? pl : (lane == 1 ? pr : p)), t, a.hdr, a.spin_limit, item) ? 1 : 0;
        } else if (lane == 0) {
            ok = wait_entry(entries + q, a.S, a.hdr, a.spin_limit, item) ? 1 : 0;
        }
        ok = __all_sync(kFull, ok);
        if (!ok) break;

        if (e1 > e0) {
            long long alo = (e0 + 3) & ~3LL;
            if (alo > e1) alo = e1;
            long long ahi = e1 & ~3LL;
            if (ahi < alo) ahi = alo;
            const long long head = alo - e0, tail = e1 - ahi;
            T* O = (T*)out.p[p];
            if (rs) {       // the joint reduction of this chunk: (from_left + own) + from_right
                const T* L = (const T*)(t == 0 ? in.p[pl] : out.p[pl]);
                const T* M = (const T*)(t == 0 ? in.p[p] : out.p[p]);
                const T* R = (const T*)(t == 0 ? in.p[pr] : out.p[pr]);
                if (lane < head) { const long long e = e0 + lane; O[e] = add3(__ldcg(L + e), __ldcg(M + e), __ldcg(R + e)); }
                else if (lane < head + tail) { const long long e = ahi + (lane - head); O[e] = add3(__ldcg(L + e), __ldcg(M + e), __ldcg(R + e)); }
#pragma unroll 4
                for (long long e = alo + 4LL * lane; e < ahi; e += 128) {
                    const V l = __ldcg((const V*)(L + e)), m = __ldcg((const V*)(M + e)), r = __ldcg((const V*)(R + e));
                    *(V*)(O + e) = add3v(l, m, r);
                }
            } else {
                const T* Q = (const T*)out.p[q];
                if (lane < head) { const long long e = e0 + lane; O[e] = __ldcg(Q + e); }
                else if (lane < head + tail) { const long long e = ahi + (lane - head); O[e] = __ldcg(Q + e); }
#pragma unroll 4
                for (long long e = alo + 4LL * lane; e < ahi; e += 128) *(V*)(O + e) = __ldcg((const V*)(Q + e));
            }
        }
        // ---- publish: rank p has finished this row for this chunk
        __threadfence();
        __syncwarp();
        if (lane == 0) st_release(entries + p, rs ? t + 1 : a.S);
    }
}

// ------------------------------------------------------------------ host side

static int pb_chunk_elems(size_t count) { return count >= ((size_t)1 << 16) ? 2048 : 1024; }

// sub-chunks per block: enough for the longest block of any collective
static int pb_nsub(const Plan& p, size_t gcount, int chunk_elems) {
    const size_t longest = gcount / (size_t)p.ndims / (size_t)p.n + 2;
    return (int)((longest + chunk_elems - 1) / chunk_elems);
}

bool pipeline_bw_supported(const Plan& p) {
    return !p.general && p.algo == TRV_ALGO_TRIVANCE && p.variant == TRV_BANDWIDTH_OPTIMAL && p.S <= kPbMaxS && p.ndims <= kPbMaxD;
}

size_t pipeline_bw_scratch_bytes(const Plan& p, size_t gcount) {
    const int ce = pb_chunk_elems(gcount);
    const size_t chunks = (size_t)p.ndims * p.n * pb_nsub(p, gcount, ce);
    return kPipeHeaderBytes + ((chunks * p.n * sizeof(int) + 255) & ~(size_t)255);
}

template <int CAP>
static trv_status_t pb_impl(const Call& c, PipeBwArgs& a) {
    const Plan& p = *c.plan;
    PtrTab<CAP> in, out;
    for (int r = 0; r < p.n; ++r) { in.p[r] = const_cast<void*>(c.in[r]); out.p[r] = c.out[r]; }
    int dev = 0, sms = 0, per_sm = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess)
        return TRV_ERR_CUDA;
    const bool f32 = c.dtype == TRV_FLOAT32;
    if ((f32 ? cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, k_bw_pipe<float, CAP>, kPbThreads, 0)
             : cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, k_bw_pipe<uint32_t, CAP>, kPbThreads, 0)) != cudaSuccess || per_sm < 1)
        return TRV_ERR_CUDA;
    int per_chunk = 0;
    for (int r = 0; r < 2 * a.S; ++r) per_chunk += a.cnt[r];
    const long long total = a.nchunks * per_chunk;
    long long grid = (long long)sms * per_sm;
    if (grid > (total + 7) / 8) grid = (total + 7) / 8;
    const long long workers = grid * (kPbThreads / 32);
    // a group's first row (n / 3 items per chunk) is about two grids' worth of items
    a.group = (int)((2 * workers + a.cnt[0] - 1) / a.cnt[0]);
    if (a.group < 1) a.group = 1;
    const size_t entries = (size_t)a.nchunks * a.n * sizeof(int);
    if (cudaMemsetAsync(c.scratch, 0, kPipeHeaderBytes + entries, c.st) != cudaSuccess) return TRV_ERR_CUDA;
    if (f32) TRV_LAUNCH((k_bw_pipe<float, CAP>), (unsigned)grid, kPbThreads, 0, c.st, in, out, a);
    else TRV_LAUNCH((k_bw_pipe<uint32_t, CAP>), (unsigned)grid, kPbThreads, 0, c.st, in, out, a);
    return cudaGetLastError() == cudaSuccess ? TRV_OK : TRV_ERR_CUDA;
}

trv_status_t run_pipeline_bandwidth(const Call& c) {
    const Plan& p = *c.plan;
    if (!pipeline_bw_supported(p)) return TRV_ERR_UNSUPPORTED;
    if (c.scratch_bytes < pipeline_bw_scratch_bytes(p, c.gcount) || !c.scratch) return TRV_ERR_SCRATCH;
    g_last_kernel = "bw_pipe";
    PipeBwArgs a;
    a.n = p.n; a.S = p.S; a.D = p.ndims;
    a.chunk_elems = pb_chunk_elems(c.gcount);
    a.nsub = pb_nsub(p, c.gcount, a.chunk_elems);
    a.nchunks = (long long)p.ndims * p.n * a.nsub;
    a.spin_limit = kSpinLimit;
    a.w0 = (long long)c.goff; a.w1 = (long long)(c.goff + c.count);
    for (int d = 0; d < kPbMaxD; ++d) { a.dims[d] = d < p.ndims ? p.dims[d] : 1; a.stride[d] = d < p.ndims ? p.stride[d] : p.n; }
    int pw = 1;
    for (int t = 0; t < p.S; ++t) {
        pw *= 3;
        a.cnt[t] = p.n / pw;                    // ranks that still answer for a block after step t
        a.cnt[2 * p.S - 1 - t] = 2 * (p.n / pw);  // AllGather row of step t: every holder serves both peers
    }
    for (int sl = 0; sl < p.ndims; ++sl) {
        a.slo[sl] = slice_lo((int64_t)c.gcount, p.ndims, sl);
        a.shi[sl] = slice_lo((int64_t)c.gcount, p.ndims, sl + 1);
        for (int t = 0; t < p.S; ++t) {
            a.sdim[sl][t] = p.steps[sl][t].dim; a.sdist[sl][t] = p.steps[sl][t].dist;
            for (int d = 0; d < kPbMaxD; ++d) a.mod[sl][t][d] = d < p.ndims ? p.mod[sl][t][d] : 1;
        }
    }
    char* base = (char*)c.scratch;
    a.hdr = (PipeHeader*)base;
    a.done = (int*)(base + kPipeHeaderBytes);
    if (p.n <= 32) return pb_impl<32>(c, a);
    if (p.n <= 256) return pb_impl<256>(c, a);
    return pb_impl<TRV_MAX_RANKS>(c, a);
}

}  // namespace trv
