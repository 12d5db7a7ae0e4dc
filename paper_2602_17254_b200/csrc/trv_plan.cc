// Schedule builder: per-step (dimension, distance) lists, peers, closed-form block sets and
// per-message byte counts.  Host-only integer work; no CUDA call in this file.
#include "trv_plan.h"

#include <new>

namespace trv {

static int exact_log(int a, int base) {
    int s = 0;
    if (a < 1) return -1;
    while (a > 1) {
        if (a % base) return -1;
        a /= base;
        ++s;
    }
    return s;
}

// Sec. 4.4 with the reading stated in the header of the C interface: the AllGather of a block runs
// the steps in reverse order (the extra distance first); holders are kept in the order they got
// the block; in a step each holder, in that order, offers it to its left peer, then to its right
// peer, and a node that holds it already is skipped.  Written in offsets from the block's owner:
// kstep[o] = the ring's step in which the node at offset o sends its partial on, ksgn[o] = +1 / -1 towards
// the node after / before it.  Returns the ring's distances.
static std::vector<int> ring_tree(int n, std::vector<int8_t>& kstep, std::vector<int8_t>& ksgn) {
    int pw = 1;
    std::vector<int> dist;
    while ((long long)pw * 3 <= n) { dist.push_back(pw); pw *= 3; }
    if (pw != n) dist.push_back((n - pw + 1) / 2);
    const int S = (int)dist.size();
    kstep.assign(n, -1);
    ksgn.assign(n, 0);
    std::vector<int> order(1, 0);
    std::vector<char> held(n, 0);
    held[0] = 1;
    for (int t = S - 1; t >= 0; --t) {
        const size_t cnt = order.size();
        for (size_t i = 0; i < cnt; ++i)
            for (int side = 0; side < 2; ++side) {
                const int delta = side ? dist[t] : -dist[t];
                const int v = ((order[i] + delta) % n + n) % n;
                if (held[v]) continue;
                held[v] = 1;
                kstep[v] = (int8_t)t;
                ksgn[v] = (int8_t)(side ? -1 : +1);      // the child sends back the way the block came
                order.push_back(v);
            }
    }
    return dist;
}

// Sides of any size, one collective per dimension (Sec. 5): collective c visits the dimensions in round-robin
// order from c, a dimension that has used up its ring's steps being skipped; the k-th visit of a dimension uses
// its ring's k-th distance.  Along every dimension a block travels by that ring's tree, so the tree on the torus
// is the product of the ring trees: the node at offset o gets the block once ALL its coordinates have been
// reached, i.e. in the AllGather step that reaches the last of them; as the AllGather runs the step list
// backwards that is the SMALLEST of the steps t_d in which its non-zero coordinates o_d are reached, and it
// gets the block along that dimension.  In the Reduce-Scatter it sends its partial on in that same step.
static bool build_general(Plan& p) {
    const int D = p.ndims, n = p.n;
    std::vector<std::vector<int8_t>> kstep(D), ksgn(D);
    std::vector<std::vector<int>> dist(D);
    p.S = 0;
    for (int d = 0; d < D; ++d) {
        dist[d] = ring_tree(p.dims[d], kstep[d], ksgn[d]);
        p.sdim[d] = (int)dist[d].size();
        p.S += p.sdim[d];
    }
    if (p.S > 120) return false;
    p.general = true;
    p.nslices = D;
    p.steps.assign(D, {});
    p.gstep.assign(D, std::vector<int8_t>(n, -1));
    p.gsgn.assign(D, std::vector<int8_t>(n, 0));
    for (int c = 0; c < D; ++c) {
        std::vector<std::vector<int>> where(D);         // where[d][k] = position of the k-th visit of dimension d
        int visits[TRV_MAX_DIMS] = {0};
        int cur = c;
        for (int t = 0; t < p.S; ++t) {
            int d = cur;
            while (visits[d] >= p.sdim[d]) d = (d + 1) % D;
            p.steps[c].push_back(Step{d, dist[d][visits[d]]});
            where[d].push_back(t);
            visits[d]++;
            cur = (d + 1) % D;
        }
        for (int o = 1; o < n; ++o) {
            int best = -1, best_d = -1;
            for (int d = 0; d < D; ++d) {
                const int od = p.coord(o, d);
                if (od == 0) continue;
                const int t = where[d][kstep[d][od]];
                if (best < 0 || t < best) { best = t; best_d = d; }
            }
            p.gstep[c][o] = (int8_t)best;
            p.gsgn[c][o] = ksgn[best_d][p.coord(o, best_d)];
        }
    }
    return true;
}

static int swing_rho(int k) {      // sum_{i<=k} (-2)^i = 1, -1, 3, -5, 11, ...  (Sec. 2.4)
    int r = 0, p = 1;
    for (int i = 0; i <= k; ++i) { r += p; p *= -2; }
    return r;
}

// Swing: what a rank still answers for after step t - 1, by the recurrence
//   reach[S][p] = {p};  reach[t][p] = reach[t+1][p] | union over the peers q of p in step t of reach[t+1][q]
// (the same sets Algorithm 1 enumerates recursively).
static void build_reach(Plan& p) {
    const int n = p.n, S = p.S;
    p.words = (n + 63) / 64;
    p.reach.assign(p.nslices, {});
    for (int c = 0; c < p.nslices; ++c) {
        auto& R = p.reach[c];
        R.assign(S + 1, std::vector<uint64_t>((size_t)n * p.words, 0));
        for (int r = 0; r < n; ++r) R[S][(size_t)r * p.words + r / 64] |= 1ULL << (r % 64);
        for (int t = S - 1; t >= 0; --t)
            for (int r = 0; r < n; ++r) {
                int peer[2], dir[2], hops[2];
                const int np = send_peers(p, r, p.steps[c][t].dim, p.steps[c][t].dist, peer, dir, hops);
                for (int w = 0; w < p.words; ++w) {
                    uint64_t v = R[t + 1][(size_t)r * p.words + w];
                    for (int i = 0; i < np; ++i) v |= R[t + 1][(size_t)peer[i] * p.words + w];
                    R[t][(size_t)r * p.words + w] = v;
                }
            }
    }
}

trv_status_t build_plan(const int32_t* dims, int32_t ndims, int variant, int algo_flags, trv_plan_s** out) {
    if (!dims || !out || ndims < 1 || ndims > TRV_MAX_DIMS) return TRV_ERR_INVALID_ARG;
    if (variant != TRV_LATENCY_OPTIMAL && variant != TRV_BANDWIDTH_OPTIMAL) return TRV_ERR_INVALID_ARG;
    const bool mirror = (algo_flags & TRV_ALGO_MIRRORED) != 0, single = (algo_flags & TRV_ALGO_SINGLE) != 0;
    const int algo = algo_flags & ~(TRV_ALGO_MIRRORED | TRV_ALGO_SINGLE);
    if (algo < TRV_ALGO_TRIVANCE || algo > TRV_ALGO_BUCKET) return TRV_ERR_INVALID_ARG;
    const bool binary = algo == TRV_ALGO_RECDOUB || algo == TRV_ALGO_SWING;
    if (mirror && (algo == TRV_ALGO_TRIVANCE || (ndims != 1 && !binary && algo != TRV_ALGO_BUCKET))) return TRV_ERR_INVALID_ARG;
    if (single && (mirror || !binary)) return TRV_ERR_INVALID_ARG;
    for (int d = 0; d < ndims; ++d)
        if (dims[d] < 2) return TRV_ERR_INVALID_ARG;
    const int base = binary ? 2 : 3;
    if (algo == TRV_ALGO_BUCKET) {
        long long nn = 1;
        for (int d = 0; d < ndims; ++d) nn *= dims[d];
        if (variant != TRV_BANDWIDTH_OPTIMAL || nn > TRV_MAX_RANKS) return TRV_ERR_UNSUPPORTED;
    }

    trv_plan_s* holder = new (std::nothrow) trv_plan_s();
    if (!holder) return TRV_ERR_ALLOC;
    Plan& p = holder->plan;
    p.algo = algo; p.variant = variant; p.ndims = ndims; p.base = base;
    p.nslices = single ? 1 : ndims * (mirror ? 2 : 1);
    if (algo == TRV_ALGO_BUCKET) {
        // ring algorithm (Sec. 2.4), dimension after dimension: a_d - 1 steps per phase, every step one message to the
        // next node of the ring along the phase's dimension
        int nn = 1;
        for (int d = 0; d < ndims; ++d) {
            p.dims[d] = dims[d]; p.stride[d] = nn; nn *= dims[d]; p.S += dims[d] - 1;
            if (dims[d] != dims[0]) p.equal_dims = false;
        }
        p.n = nn;
        p.steps.assign(p.nslices, {});
        p.bk_step.assign(p.nslices, {}); p.bk_earlier.assign(p.nslices, {}); p.bk_start.assign(p.nslices, {});
        for (int c = 0; c < p.nslices; ++c) {
            int earlier = 0;
            for (int ph = 0; ph < ndims; ++ph) {
                const int d = (c + ph) % ndims;
                p.bk_start[c].push_back((int)p.steps[c].size());
                for (int s = 0; s < dims[d] - 1; ++s) {
                    p.steps[c].push_back(Step{d, c >= ndims ? -1 : 1});
                    p.bk_step[c].push_back(s);
                    p.bk_earlier[c].push_back(earlier);
                }
                earlier |= 1 << d;
            }
        }
        *out = holder;
        return TRV_OK;
    }
    bool other_side = false;
    for (int d = 0; d < ndims; ++d)
        if (exact_log(dims[d], 3) < 1) other_side = true;
    if (algo == TRV_ALGO_TRIVANCE && other_side) {
        // a side that is no power of three: only the bandwidth-optimal form is defined (Sec. 4.4)
        long long nn = 1;
        for (int d = 0; d < ndims; ++d) nn *= dims[d];
        if (variant != TRV_BANDWIDTH_OPTIMAL || nn > TRV_MAX_RANKS || ndims > 4) { delete holder; return TRV_ERR_UNSUPPORTED; }
        nn = 1;
        for (int d = 0; d < ndims; ++d) {
            p.dims[d] = dims[d]; p.stride[d] = (int)nn; nn *= dims[d];
            if (dims[d] != dims[0]) p.equal_dims = false;
        }
        p.n = (int)nn;
        if (!build_general(p)) { delete holder; return TRV_ERR_UNSUPPORTED; }
        *out = holder;
        return TRV_OK;
    }
    long long n = 1;
    for (int d = 0; d < ndims; ++d) {
        int s = exact_log(dims[d], base);
        if (s < 1) {
            delete holder;
            return binary ? TRV_ERR_UNDEFINED_SCHEDULE : TRV_ERR_UNSUPPORTED;
        }
        p.dims[d] = dims[d]; p.sdim[d] = s; p.stride[d] = (int)n;
        n *= dims[d]; p.S += s;
        if (n > TRV_MAX_RANKS) { delete holder; return TRV_ERR_UNSUPPORTED; }
        if (dims[d] != dims[0]) p.equal_dims = false;
    }
    p.n = (int)n;

    // Sec. 5: collective c starts on dimension c and moves to the next dimension every step;
    // a dimension that has used up its log_base(a_d) steps is skipped.
    p.steps.resize(p.nslices);
    p.mod.resize(p.nslices);
    for (int c = 0; c < p.nslices; ++c) {
        int visits[TRV_MAX_DIMS] = {0};
        int pw[TRV_MAX_DIMS];
        for (int d = 0; d < ndims; ++d) pw[d] = 1;
        const int sign = c >= ndims ? -1 : 1;
        int cur = c % ndims;
        for (int t = 0; t < p.S; ++t) {
            int d = cur;
            while (visits[d] >= p.sdim[d]) d = (d + 1) % ndims;
            p.steps[c].push_back(Step{d, sign * (algo == TRV_ALGO_SWING ? swing_rho(visits[d]) : pw[d])});
            visits[d]++; pw[d] *= base;
            p.mod[c].push_back(std::vector<int>(pw, pw + ndims));
            cur = (d + 1) % ndims;
        }
    }
    if (algo == TRV_ALGO_SWING) build_reach(p);
    *out = holder;
    return TRV_OK;
}

// Bucket: is block j in the message node src passes on in `row`?  Reduce-Scatter step s of a phase carries the blocks whose
// coordinate in the phase's dimension is src's minus (s + 1) (mirrored: plus), AllGather step s those with src's minus s
// -- the ring rule "block r - t - 1, then block r - t" -- among the blocks that agree with src in the earlier dimensions.
bool bucket_sends(const Plan& p, int c, int row, int src, int j) {
    const int t = p.bucket_step(c, row), d = p.steps[c][t].dim, sg = p.steps[c][t].dist, a = p.dims[d];
    const int off = p.bk_step[c][t] + (row < p.S ? 1 : 0);
    if (p.coord(j, d) != ((p.coord(src, d) - sg * off) % a + a) % a) return false;
    for (int q = 0; q < p.ndims; ++q)
        if (((p.bk_earlier[c][t] >> q) & 1) && p.coord(j, q) != p.coord(src, q)) return false;
    return true;
}

bool in_send_set(const Plan& p, int c, int t, int dst, int j) {
    if (p.algo == TRV_ALGO_SWING) return (p.reach[c][t + 1][(size_t)dst * p.words + j / 64] >> (j % 64)) & 1;
    if (p.algo == TRV_ALGO_BUCKET)      // what dst's upstream neighbour passes on in Reduce-Scatter step t
        return bucket_sends(p, c, t, p.shift(dst, p.steps[c][t].dim, -p.steps[c][t].dist), j);
    if (p.algo == TRV_ALGO_RECDOUB && c >= p.ndims) {     // the mirrored collective is the same pattern on the rings read backwards
        int nd = 0, nj = 0;                               // every coordinate x -> (side - x) mod side
        for (int d = 0; d < p.ndims; ++d) {
            nd += ((p.dims[d] - p.coord(dst, d)) % p.dims[d]) * p.stride[d];
            nj += ((p.dims[d] - p.coord(j, d)) % p.dims[d]) * p.stride[d];
        }
        return in_send_set(p, c - p.ndims, t, nd, nj);
    }
    for (int d = 0; d < p.ndims; ++d) {
        int m = p.mod[c][t][d];
        if ((p.coord(j, d) - p.coord(dst, d)) % m != 0) return false;
    }
    return true;
}

int send_peers(const Plan& p, int r, int dim, int dist, int peer[2], int dir[2], int hops[2]) {
    if (p.algo == TRV_ALGO_TRIVANCE) {
        peer[0] = p.shift(r, dim, -dist); dir[0] = -1; hops[0] = dist;
        peer[1] = p.shift(r, dim, +dist); dir[1] = +1; hops[1] = dist;
        return 2;
    }
    // comparators: a negative distance marks the mirrored collective (everything reversed)
    const int sg = dist < 0 ? -1 : 1, a = dist < 0 ? -dist : dist;
    peer[1] = -1; dir[1] = 0; hops[1] = 0;
    switch (p.algo) {
        case TRV_ALGO_BRUCK:
            peer[0] = p.shift(r, dim, sg * a);     dir[0] = sg; hops[0] = a;
            peer[1] = p.shift(r, dim, sg * 2 * a); dir[1] = sg; hops[1] = 2 * a;
            return 2;
        case TRV_ALGO_SWING: {          // r + rho for even r, r - rho for odd r; the short way round
            const int delta = (p.coord(r, dim) % 2 == 0) ? dist : -dist;
            peer[0] = p.shift(r, dim, delta); dir[0] = delta > 0 ? +1 : -1; hops[0] = delta > 0 ? delta : -delta;
            return 1;
        }
        case TRV_ALGO_BUCKET:
            peer[0] = p.shift(r, dim, sg); dir[0] = sg; hops[0] = 1;
            return 1;
        default: {                      // Recursive Doubling; mirrored: positions counted backwards
            const int size = p.dims[dim], x = p.coord(r, dim);
            const int xm = sg > 0 ? x : (size - x) % size;
            const int ym = xm ^ a;
            const int y = sg > 0 ? ym : (size - ym) % size;
            peer[0] = r + (y - x) * p.stride[dim]; dir[0] = ym > xm ? sg : -sg; hops[0] = a;
            return 1;
        }
    }
}

int general_recv_mask(const Plan& p, int c, int t, int dst, int j) {
    const int d = p.steps[c][t].dim, dist = p.steps[c][t].dist;
    const int o = p.sub(dst, j);
    const int ol = p.shift(o, d, -dist), orr = p.shift(o, d, dist);
    int mask = 0;
    if (p.gstep[c][ol] == t && p.gsgn[c][ol] > 0) mask |= 1;
    if (orr != ol && p.gstep[c][orr] == t && p.gsgn[c][orr] < 0) mask |= 2;
    return mask;
}

void message_bytes_side(const Plan& p, int64_t E, int64_t elem_size, int c, int row, int side, int64_t* out) {
    const int n = p.n;
    if (p.general) {
        // Reduce-Scatter row: the node at offset o sends block (node - o); AllGather row: the parent
        // of the node at offset o, which sits at offset o + sgn * dist along the step's dimension, sends it to that node.
        const int t = p.step_of_row(row), d = p.steps[c][t].dim, dist = p.steps[c][t].dist;
        const bool rs = row < p.S;
        const int64_t lo = slice_lo(E, p.nslices, c), hi = slice_lo(E, p.nslices, c + 1);
        for (int r = 0; r < n; ++r) out[r] = 0;
        for (int o = 1; o < n; ++o) {
            if (p.gstep[c][o] != t) continue;
            const int sends_right = rs ? (p.gsgn[c][o] > 0) : (p.gsgn[c][o] < 0);
            if (sends_right != side) continue;
            const int src_off = rs ? o : p.shift(o, d, p.gsgn[c][o] * dist);
            for (int r = 0; r < n; ++r) {
                const int j = p.sub(r, src_off);
                out[r] += (block_lo(lo, hi, n, j + 1) - block_lo(lo, hi, n, j)) * elem_size;
            }
        }
        return;
    }
    std::vector<int64_t> tmp((size_t)n);
    message_bytes(p, E, elem_size, c, row, tmp.data());
    const Step& st = p.steps[c][p.row_step(c, row)];
    const bool by_source = p.variant == TRV_BANDWIDTH_OPTIMAL && row >= p.S;
    for (int r = 0; r < n; ++r) {
        int peer[2], dir[2], hops[2];
        const int np = send_peers(p, r, st.dim, st.dist, peer, dir, hops);
        out[r] = side < np ? (by_source ? tmp[r] : tmp[peer[side]]) : 0;
    }
}

void message_bytes(const Plan& p, int64_t E, int64_t elem_size, int c, int row, int64_t* out) {
    const int n = p.n, D = p.ndims;
    const int64_t lo = slice_lo(E, p.nslices, c), hi = slice_lo(E, p.nslices, c + 1);
    if (p.variant == TRV_LATENCY_OPTIMAL) {
        for (int r = 0; r < n; ++r) out[r] = (hi - lo) * elem_size;
        return;
    }
    auto blen = [&](int j) { return (block_lo(lo, hi, n, j + 1) - block_lo(lo, hi, n, j)) * elem_size; };
    if (p.algo == TRV_ALGO_BUCKET) {
        // Reduce-Scatter rows by destination (what its upstream neighbour passes on), AllGather rows by source
        const Step& st = p.steps[c][p.bucket_step(c, row)];
        for (int r = 0; r < n; ++r) {
            const int src = row < p.S ? p.shift(r, st.dim, -st.dist) : r;
            int64_t sum = 0;
            for (int j = 0; j < n; ++j)
                if (bucket_sends(p, c, row, src, j)) sum += blen(j);
            out[r] = sum;
        }
        return;
    }
    if (p.algo == TRV_ALGO_SWING || (p.algo == TRV_ALGO_RECDOUB && c >= p.ndims)) {
        const int t = p.step_of_row(row);
        for (int r = 0; r < n; ++r) {
            int64_t sum = 0;
            for (int j = 0; j < n; ++j)
                if (in_send_set(p, c, t, r, j)) sum += blen(j);
            out[r] = sum;
        }
        return;
    }
    // The set of row `row` is the same congruence class for Reduce-Scatter (blocks destined to
    // travel on through the receiver) and for the mirrored AllGather row (finished blocks the
    // sender holds): all j that agree with the rank modulo mod[c][t][d] in every dimension.
    const int t = p.step_of_row(row);
    for (int r = 0; r < n; ++r) {
        int64_t sum = 0;
        // enumerate j_d = (r_d mod m_d) + m_d * i_d
        int idx[TRV_MAX_DIMS] = {0};
        for (;;) {
            int j = 0;
            for (int d = 0; d < D; ++d) j += ((p.coord(r, d) % p.mod[c][t][d]) + p.mod[c][t][d] * idx[d]) * p.stride[d];
            sum += block_lo(lo, hi, n, j + 1) - block_lo(lo, hi, n, j);
            int d = 0;
            for (; d < D; ++d) {
                if (++idx[d] < p.dims[d] / p.mod[c][t][d]) break;
                idx[d] = 0;
            }
            if (d == D) break;
        }
        out[r] = sum * elem_size;
    }
}

}  // namespace trv
