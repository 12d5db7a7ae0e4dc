// PIPELINED kernel family: the latency-optimal form run by a chunk-level readiness engine
// (App. D; Discussion, "Joint Reduction Overheads"), emulated inside one GPU.
//
// The paper's sketch: one work descriptor per (rank, step, chunk) naming both peers, the buffer
// offsets and the element count; a per-chunk readiness entry that the arrival of the left and of
// the right chunk each mark; the reduction of a chunk runs as soon as both are marked and the entry
// belongs to the current generation, reads the two incoming chunks where they were received, and
// adds them to the local partial; chunks are taken in the same order on both sides.
//
// Here: ONE persistent kernel whose warps are the workers.  A work item is (chunk, step, rank).  All ranks share one address
// space, so the peer's partial of the previous step IS the receive slot: nothing is copied, and
// "the left chunk has arrived" means "the left peer has finished this chunk's previous step".
// The readiness entry of (chunk, rank) is a counter of finished steps, written with release
// semantics after the item's stores; an item of step t waits until the entries of its left peer,
// its right peer and itself have reached t (read-after-write), and until the two ranks that read
// the buffer it is about to overwrite have finished reading it (write-after-read: the ranks at the
// PREVIOUS step's distance; for an in-place call's last step the ranks at the first step's
// distance).  A memset node in front of the kernel zeroes the entries: that is the generation.
//
// Items are handed out by a ticket counter in a fixed total order in which every item comes after
// the items it waits for (groups of K chunks; inside a group step by step, inside a step chunk by
// chunk, rank by rank).  A warp therefore only ever waits for items that were taken earlier, by warps
// that are already running: no deadlock whatever the grid size, no cooperative launch needed.  K is
// chosen so that one step of a group is about two grids' worth of items: when a warp reaches step
// t + 1 of a group, step t is almost always done and nobody spins.  What bounds the engine is the
// latency of an item (ticket, readiness loads, data round trip, fence, publish) times the items
// per worker, so it runs with as many resident warps as fit; a group is then too large to stay in
// L2 (2 x 5920 workers x 8 KB = 97 MB per buffer) and the DRAM traffic is 4.8x the one-read-one-
// write minimum (ring 243: the STEP family moves 7x).  Smaller grids or chunks, which would keep a
// group in L2, were 1.5 to 5x slower.
//
// Every wait is bounded: after kSpinLimit polls a waiter records TRV_ERR_TIMEOUT and the item in
// the header, every other waiter sees that and leaves, and the kernel ends; trv_pipeline_status
// reports it.  Data written by other SMs is read with L1-bypassing loads.
#include "trv_dev.cuh"
#include "trv_wait.cuh"

namespace trv {

constexpr int kPipeThreads = 256;
constexpr int kPipeMaxS = 8;
struct PipeArgs {
    int n, S, nslices, in_place;
    int chunk_elems, nchunks, group;        // elements per chunk; chunks in all slices; chunks per group (K)
    unsigned spin_limit;
    long long lo[TRV_MAX_DIMS], hi[TRV_MAX_DIMS];   // local element range of each slice
    int cbase[TRV_MAX_DIMS + 1];                    // first chunk of each slice
    int stride[TRV_MAX_DIMS][kPipeMaxS], size[TRV_MAX_DIMS][kPipeMaxS], dist[TRV_MAX_DIMS][kPipeMaxS];
    char* buf[2];               // scratch partials: rank r's row at buf[i] + r * row_bytes
    size_t row_bytes;
    int* done;                  // readiness entries [chunk][rank]
    PipeHeader* hdr;
};

__device__ __forceinline__ int peer_of(int p, int stride, int size, int delta) {
    const int x = (p / stride) % size;
    int y = x + delta;
    if (y < 0) y += size;
    if (y >= size) y -= size;
    return p + (y - x) * stride;
}

template <typename T>
__device__ __forceinline__ T ld_cg(const T* p) { return __ldcg(p); }

// Every WARP is a worker of its own: it draws tickets, waits and publishes without involving the
// rest of its CTA, so a CTA keeps eight items in flight.
template <typename T, int CAP>
__global__ void __launch_bounds__(kPipeThreads) k_lat_pipe(PtrTab<CAP> in, PtrTab<CAP> out, PipeArgs a) {
    using V = typename Vec4<T>::type;
    constexpr unsigned kFull = 0xffffffffu;
    const int lane = threadIdx.x & 31;
    const long long per_chunk = (long long)a.S * a.n;
    const long long total = (long long)a.nchunks * per_chunk;
    for (;;) {
        long long item = 0;
        if (lane == 0) item = (long long)atomicAdd(&a.hdr->ticket, 1ULL);
        item = __shfl_sync(kFull, item, 0);
        if (item >= total) break;
        // item -> (chunk c, step t, rank p): groups of K chunks, step-major inside a group
        const long long gsz = (long long)a.group * per_chunk;
        const int g = (int)(item / gsz);
        const int kg = min(a.group, a.nchunks - g * a.group);      // chunks in this group
        const long long local = item - (long long)g * gsz;
        const int t = (int)(local / ((long long)kg * a.n));
        const int rem = (int)(local % ((long long)kg * a.n));
        const int c = g * a.group + rem / a.n, p = rem % a.n;
        int sl = 0;
        while (sl + 1 < a.nslices && c >= a.cbase[sl + 1]) ++sl;
        const long long e0 = a.lo[sl] + (long long)(c - a.cbase[sl]) * a.chunk_elems;
        const long long e1 = min(a.hi[sl], e0 + a.chunk_elems);
        const int pl = peer_of(p, a.stride[sl][t], a.size[sl][t], -a.dist[sl][t]);
        const int pr = peer_of(p, a.stride[sl][t], a.size[sl][t], +a.dist[sl][t]);

        // ---- readiness: both incoming chunks and the local partial; then the buffer to overwrite
        int ok = 1;
        if (t > 0 && lane < 7) {
            int q = -1, need = t;
            if (lane == 0) q = pl;
            else if (lane == 1) q = pr;
            else if (lane == 2) q = p;
            else if (lane == 3) q = peer_of(p, a.stride[sl][t - 1], a.size[sl][t - 1], -a.dist[sl][t - 1]);
            else if (lane == 4) q = peer_of(p, a.stride[sl][t - 1], a.size[sl][t - 1], +a.dist[sl][t - 1]);
            else if (a.in_place && t == a.S - 1) {
                q = peer_of(p, a.stride[sl][0], a.size[sl][0], lane == 5 ? -a.dist[sl][0] : +a.dist[sl][0]);
                need = 1;
            }
            if (q >= 0) ok = wait_entry(a.done + (size_t)c * a.n + q, need, a.hdr, a.spin_limit, item) ? 1 : 0;
        }
        ok = __all_sync(kFull, ok);
        if (!ok) break;

        // ---- the joint reduction of this chunk: (from_left + own) + from_right
        const T *L, *M, *R;
        if (t == 0) {
            L = (const T*)in.p[pl]; M = (const T*)in.p[p]; R = (const T*)in.p[pr];
        } else {
            const char* b = a.buf[(t - 1) & 1];
            L = (const T*)(b + (size_t)pl * a.row_bytes); M = (const T*)(b + (size_t)p * a.row_bytes);
            R = (const T*)(b + (size_t)pr * a.row_bytes);
        }
        T* O = (t == a.S - 1) ? (T*)out.p[p] : (T*)(a.buf[t & 1] + (size_t)p * a.row_bytes);
        long long alo = (e0 + 3) & ~3LL;
        if (alo > e1) alo = e1;
        long long ahi = e1 & ~3LL;
        if (ahi < alo) ahi = alo;
        const long long head = alo - e0, tail = e1 - ahi;
        if (lane < head) { const long long e = e0 + lane; O[e] = add3(ld_cg(L + e), ld_cg(M + e), ld_cg(R + e)); }
        else if (lane < head + tail) { const long long e = ahi + (lane - head); O[e] = add3(ld_cg(L + e), ld_cg(M + e), ld_cg(R + e)); }
#pragma unroll 4
        for (long long e = alo + 4LL * lane; e < ahi; e += 128) {
            const V l = ld_cg((const V*)(L + e)), m = ld_cg((const V*)(M + e)), r = ld_cg((const V*)(R + e));
            *(V*)(O + e) = add3v(l, m, r);
        }
        // ---- publish: this chunk of rank p has finished step t
        __threadfence();
        __syncwarp();
        if (lane == 0) st_release(a.done + (size_t)c * a.n + p, t + 1);
    }
}

// One CTA waits, with a short limit, for a readiness entry that nothing sets: exercises the give-up path.
__global__ void k_pipe_wait_never(PipeHeader* hdr, const int* entry, unsigned limit) {
    if (threadIdx.x == 0) wait_entry(entry, 1, hdr, limit, -1);
}

// ------------------------------------------------------------------ host side

static size_t pipe_padded(size_t count) { return (count + 63) & ~(size_t)63; }
static int pipe_buffers(const Plan& p) { return p.S >= 3 ? 2 : (p.S == 2 ? 1 : 0); }
// Measured on B200 (ring 27 x 2 MiB / ring 243 x 8 MiB, us per call): 512 elements 135 / 5854, 1024: 112 / 4455,
// 2048: 81 / 4126, 4096: 116 / 3961 (with groups of two grids' worth of items; one grid's worth: 104 / 4336).
static int pipe_chunk_elems(size_t count) { return count >= ((size_t)1 << 16) ? 2048 : 1024; }

static int pipe_chunks(const Call& c, int chunk_elems, int* cbase) {
    int total = 0;
    for (int sl = 0; sl < c.plan->ndims; ++sl) {
        long long lo, hi;
        local_slice(c, sl, &lo, &hi);
        if (cbase) cbase[sl] = total;
        total += (int)((hi - lo + chunk_elems - 1) / chunk_elems);
    }
    if (cbase) cbase[c.plan->ndims] = total;
    return total;
}

bool pipeline_supported(const Plan& p, bool in_place) {
    if (p.general || p.algo != TRV_ALGO_TRIVANCE || p.variant != TRV_LATENCY_OPTIMAL || p.S > kPipeMaxS) return false;
    return !(in_place && p.S == 1);     // a single step in place would read what its neighbours overwrite
}

// room for the readiness entries: an upper bound on the chunks of any window of `count` elements
static size_t pipe_entry_bytes(const Plan& p, size_t count) {
    const size_t chunks = count / (size_t)pipe_chunk_elems(count) + (size_t)p.ndims + 1;
    return (chunks * p.n * sizeof(int) + 255) & ~(size_t)255;
}

size_t pipeline_scratch_bytes(const Plan& p, size_t count) {
    return kPipeHeaderBytes + pipe_entry_bytes(p, count) + (size_t)pipe_buffers(p) * p.n * pipe_padded(count) * 4;
}

template <int CAP>
static trv_status_t pipe_impl(const Call& c, PipeArgs& a) {
    const Plan& p = *c.plan;
    PtrTab<CAP> in, out;
    for (int r = 0; r < p.n; ++r) { in.p[r] = const_cast<void*>(c.in[r]); out.p[r] = c.out[r]; }
    int dev = 0, sms = 0, per_sm = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess)
        return TRV_ERR_CUDA;
    const bool f32 = c.dtype == TRV_FLOAT32;
    if ((f32 ? cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, k_lat_pipe<float, CAP>, kPipeThreads, 0)
             : cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, k_lat_pipe<uint32_t, CAP>, kPipeThreads, 0)) != cudaSuccess || per_sm < 1)
        return TRV_ERR_CUDA;
    const long long total = (long long)a.nchunks * a.S * a.n;
    long long grid = (long long)sms * per_sm;
    if (grid > (total + 7) / 8) grid = (total + 7) / 8;
    const long long workers = grid * (kPipeThreads / 32);
    a.group = (int)((2 * workers + a.n - 1) / a.n);
    if (a.group < 1) a.group = 1;
    // the generation: ticket, error and all readiness entries start at zero
    const size_t entries = (size_t)a.nchunks * a.n * sizeof(int);
    if (cudaMemsetAsync(c.scratch, 0, kPipeHeaderBytes + entries, c.st) != cudaSuccess) return TRV_ERR_CUDA;
    if (f32) TRV_LAUNCH((k_lat_pipe<float, CAP>), (unsigned)grid, kPipeThreads, 0, c.st, in, out, a);
    else TRV_LAUNCH((k_lat_pipe<uint32_t, CAP>), (unsigned)grid, kPipeThreads, 0, c.st, in, out, a);
    return cudaGetLastError() == cudaSuccess ? TRV_OK : TRV_ERR_CUDA;
}

trv_status_t run_pipeline_latency(const Call& c) {
    const Plan& p = *c.plan;
    if (!pipeline_supported(p, c.in_place)) return TRV_ERR_UNSUPPORTED;
    if (c.scratch_bytes < pipeline_scratch_bytes(p, c.count) || !c.scratch) return TRV_ERR_SCRATCH;
    if (c.count >= ((size_t)1 << 31)) return TRV_ERR_UNSUPPORTED;
    g_last_kernel = "lat_pipe";
    PipeArgs a;
    a.n = p.n; a.S = p.S; a.nslices = p.ndims; a.in_place = c.in_place ? 1 : 0;
    a.chunk_elems = pipe_chunk_elems(c.count);
    a.nchunks = pipe_chunks(c, a.chunk_elems, a.cbase);
    a.spin_limit = kSpinLimit;
    if (a.nchunks == 0) return TRV_OK;
    for (int sl = 0; sl < p.ndims; ++sl) {
        local_slice(c, sl, &a.lo[sl], &a.hi[sl]);
        for (int t = 0; t < p.S; ++t) {
            const Step& st = p.steps[sl][t];
            a.stride[sl][t] = p.stride[st.dim]; a.size[sl][t] = p.dims[st.dim]; a.dist[sl][t] = st.dist;
        }
    }
    char* base = (char*)c.scratch;
    a.hdr = (PipeHeader*)base;
    a.done = (int*)(base + kPipeHeaderBytes);
    a.row_bytes = pipe_padded(c.count) * 4;
    a.buf[0] = base + kPipeHeaderBytes + pipe_entry_bytes(p, c.count);
    a.buf[1] = a.buf[0] + (size_t)p.n * a.row_bytes;
    if (p.n <= 32) return pipe_impl<32>(c, a);
    if (p.n <= 256) return pipe_impl<256>(c, a);
    return pipe_impl<TRV_MAX_RANKS>(c, a);
}

trv_status_t pipeline_status(const void* scratch, cudaStream_t st) {
    PipeHeader h;
    if (cudaStreamSynchronize(st) != cudaSuccess) return TRV_ERR_CUDA;
    if (cudaMemcpy(&h, scratch, sizeof(h), cudaMemcpyDeviceToHost) != cudaSuccess) return TRV_ERR_CUDA;
    return h.error == 0 ? TRV_OK : (trv_status_t)h.error;
}

trv_status_t pipeline_selftest_timeout(void* scratch, size_t scratch_bytes, cudaStream_t st) {
    if (!scratch || scratch_bytes < 2 * kPipeHeaderBytes) return TRV_ERR_SCRATCH;
    if (cudaMemsetAsync(scratch, 0, 2 * kPipeHeaderBytes, st) != cudaSuccess) return TRV_ERR_CUDA;
    TRV_LAUNCH(k_pipe_wait_never, 1, 32, 0, st, (PipeHeader*)scratch, (const int*)((char*)scratch + kPipeHeaderBytes), 1000u);
    return cudaGetLastError() == cudaSuccess ? TRV_OK : TRV_ERR_CUDA;
}

}  // namespace trv
