// The comparison algorithms as executable data paths (Sec. 2.4, Sec. 3.1): Bruck with joint reductions (peers
// r + 3^k and r + 2 3^k), Recursive Doubling (r XOR 2^k), Swing (r +- rho(k)), the ring (Bucket) algorithm, each
// optionally with its mirrored sub-collective on the other half of the vector.  They are baselines, so they run
// step by step, literally: at the start of a step every rank's current vector is copied to a "wire" buffer (what it
// would put on the network), then every rank reduces what its senders put there into its own buffer.
//   latency form   : the whole slice of the collective
//   bandwidth form : Reduce-Scatter: the blocks the receiver still answers for after the step (the plan's send
//                    sets); AllGather: the steps in reverse order, a rank passes on every finished block it holds
// The arithmetic is the joint-reduction kernel of trv_joint.cu on segment lists built here from the plan's tables.
// Association (the paper states none): a rank that gets m0 from the sender whose first peer it is and m1 from the
// sender whose second peer it is forms (m1 + own) + m0; with a single message own + m0.
#include <vector>

#include "trv_dev.cuh"

namespace trv {

static size_t cmp_padded(size_t count) { return (count + 63) & ~(size_t)63; }

size_t comparator_scratch_bytes(const Plan& p, size_t count) { return (size_t)p.n * cmp_padded(count) * 4; }

namespace {
struct Segs {
    std::vector<const void*> l, m, r;
    std::vector<void*> o;
    std::vector<size_t> cnt;
    void add(const void* left, const void* own, const void* right, void* out, size_t count) {
        if (!count) return;
        l.push_back(left); m.push_back(own); r.push_back(right); o.push_back(out); cnt.push_back(count);
    }
    trv_status_t run(int dtype, cudaStream_t st) {
        const trv_status_t s = joint_run(l.data(), m.data(), r.data(), o.data(), cnt.data(), cnt.size(), dtype, st);
        l.clear(); m.clear(); r.clear(); o.clear(); cnt.clear();
        return s;
    }
};
}  // namespace

trv_status_t run_comparator(const Call& c) {
    const Plan& p = *c.plan;
    const int n = p.n, S = p.S, NS = p.nslices;
    if (p.algo == TRV_ALGO_TRIVANCE) return TRV_ERR_UNSUPPORTED;
    if (p.algo == TRV_ALGO_BUCKET && p.variant != TRV_BANDWIDTH_OPTIMAL) return TRV_ERR_UNSUPPORTED;
    const size_t row = cmp_padded(c.count);
    if (!c.scratch || c.scratch_bytes < comparator_scratch_bytes(p, c.count)) return TRV_ERR_SCRATCH;
    g_last_kernel = "comparator_steps";
    char* const wire = (char*)c.scratch;
    auto wire_of = [&](int r, long long e) { return (const void*)(wire + ((size_t)r * row + (size_t)e) * 4); };
    auto out_of = [&](int r, long long e) { return (void*)((char*)c.out[r] + (size_t)e * 4); };
    Segs segs;
    trv_status_t st;
    if (!c.in_place) {
        for (int r = 0; r < n; ++r) segs.add(nullptr, c.in[r], nullptr, c.out[r], c.count);
        if ((st = segs.run(c.dtype, c.st)) != TRV_OK) return st;
    }
    const long long w0 = (long long)c.goff, w1 = (long long)(c.goff + c.count);
    auto clip = [&](long long g) { return (g < w0 ? w0 : (g > w1 ? w1 : g)) - w0; };    // global index -> local, cut to the window
    auto snapshot = [&](long long lo, long long hi) {     // every rank puts its current slice on the wire
        for (int r = 0; r < n; ++r) segs.add(nullptr, out_of(r, lo), nullptr, (void*)wire_of(r, lo), (size_t)(hi - lo));
        return segs.run(c.dtype, c.st);
    };
    std::vector<int> from((size_t)2 * n);
    std::vector<char> have, snap;
    for (int sl = 0; sl < NS; ++sl) {
        const long long slo = slice_lo((int64_t)c.gcount, NS, sl), shi = slice_lo((int64_t)c.gcount, NS, sl + 1);
        const long long llo = clip(slo), lhi = clip(shi);
        if (lhi <= llo) continue;
        std::vector<long long> bs((size_t)n + 1);
        for (int j = 0; j <= n; ++j) bs[j] = clip(block_lo(slo, shi, n, j));
        for (int t = 0; t < S; ++t) {                           // ---- latency form, or Reduce-Scatter
            if ((st = snapshot(llo, lhi)) != TRV_OK) return st;
            const Step& step = p.steps[sl][t];
            std::fill(from.begin(), from.end(), -1);
            for (int r = 0; r < n; ++r) {
                int peer[2], dir[2], hops[2];
                const int np = send_peers(p, r, step.dim, step.dist, peer, dir, hops);
                for (int k = 0; k < np; ++k) from[(size_t)2 * peer[k] + k] = r;
            }
            for (int q = 0; q < n; ++q) {
                const int r0 = from[(size_t)2 * q], r1 = from[(size_t)2 * q + 1];
                if (r0 < 0 && r1 < 0) continue;
                auto reduce = [&](long long lo, long long hi) {
                    segs.add(r1 >= 0 ? wire_of(r1, lo) : nullptr, out_of(q, lo), r0 >= 0 ? wire_of(r0, lo) : nullptr, out_of(q, lo),
                             (size_t)(hi - lo));
                };
                if (p.variant == TRV_LATENCY_OPTIMAL) { reduce(llo, lhi); continue; }
                // the blocks q still answers for after this step; neighbouring blocks travel as one range
                long long run_lo = -1, run_hi = -1;
                for (int j = 0; j < n; ++j) {
                    if (!in_send_set(p, sl, t, q, j) || bs[j + 1] <= bs[j]) continue;
                    if (bs[j] == run_hi) { run_hi = bs[j + 1]; continue; }
                    if (run_hi > run_lo) reduce(run_lo, run_hi);
                    run_lo = bs[j]; run_hi = bs[j + 1];
                }
                if (run_hi > run_lo) reduce(run_lo, run_hi);
            }
            if ((st = segs.run(c.dtype, c.st)) != TRV_OK) return st;
        }
        if (p.variant != TRV_BANDWIDTH_OPTIMAL) continue;
        // ---- AllGather: a rank passes on every finished block it holds (Bucket: the one block of the row)
        have.assign((size_t)n * n, 0);
        for (int r = 0; r < n; ++r) have[(size_t)r * n + r] = 1;
        for (int rw = 0; rw < S; ++rw) {
            const int t = S - 1 - rw;
            if ((st = snapshot(llo, lhi)) != TRV_OK) return st;
            snap = have;
            const Step& step = p.steps[sl][p.algo == TRV_ALGO_BUCKET ? p.bucket_step(sl, S + rw) : t];
            for (int r = 0; r < n; ++r) {
                int peer[2], dir[2], hops[2];
                const int np = send_peers(p, r, step.dim, step.dist, peer, dir, hops);
                for (int k = 0; k < np; ++k)
                    for (int j = 0; j < n; ++j) {
                        const bool sends = p.algo == TRV_ALGO_BUCKET ? bucket_sends(p, sl, S + rw, r, j) : snap[(size_t)r * n + j] != 0;
                        if (!sends) continue;
                        have[(size_t)peer[k] * n + j] = 1;
                        segs.add(nullptr, wire_of(r, bs[j]), nullptr, out_of(peer[k], bs[j]), (size_t)(bs[j + 1] - bs[j]));
                    }
            }
            if ((st = segs.run(c.dtype, c.st)) != TRV_OK) return st;
        }
    }
    return TRV_OK;
}

}  // namespace trv
