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
// peer, and a node that holds it already is skipped.  Written in offsets from the block's owner.
static void build_general_ring(Plan& p, int n) {
    int pw = 1;
    std::vector<Step> steps;
    while ((long long)pw * 3 <= n) { steps.push_back(Step{0, pw}); pw *= 3; }
    steps.push_back(Step{0, (n - pw + 1) / 2});
    p.general = true;
    p.nslices = 1;
    p.S = (int)steps.size();
    p.gstep.assign(n, -1);
    p.gsgn.assign(n, 0);
    std::vector<int> order(1, 0);
    std::vector<char> held(n, 0);
    held[0] = 1;
    for (int t = p.S - 1; t >= 0; --t) {
        const size_t cnt = order.size();
        for (size_t i = 0; i < cnt; ++i)
            for (int side = 0; side < 2; ++side) {
                const int delta = side ? steps[t].dist : -steps[t].dist;
                const int v = ((order[i] + delta) % n + n) % n;
                if (held[v]) continue;
                held[v] = 1;
                p.gstep[v] = (int8_t)t;
                p.gsgn[v] = (int8_t)(side ? -1 : +1);      // the child sends back the way the block came
                order.push_back(v);
            }
    }
    p.steps.assign(1, steps);
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
    const bool mirror = (algo_flags & TRV_ALGO_MIRRORED) != 0;
    const int algo = algo_flags & ~TRV_ALGO_MIRRORED;
    if (algo < TRV_ALGO_TRIVANCE || algo > TRV_ALGO_BUCKET) return TRV_ERR_INVALID_ARG;
    if (mirror && (algo == TRV_ALGO_TRIVANCE || ndims != 1)) return TRV_ERR_INVALID_ARG;
    for (int d = 0; d < ndims; ++d)
        if (dims[d] < 2) return TRV_ERR_INVALID_ARG;
    const bool binary = algo == TRV_ALGO_RECDOUB || algo == TRV_ALGO_SWING;
    const int base = binary ? 2 : 3;
    if ((binary || algo == TRV_ALGO_BUCKET) && ndims != 1) return TRV_ERR_UNSUPPORTED;
    if (algo == TRV_ALGO_BUCKET && (variant != TRV_BANDWIDTH_OPTIMAL || dims[0] > TRV_MAX_RANKS)) return TRV_ERR_UNSUPPORTED;

    trv_plan_s* holder = new (std::nothrow) trv_plan_s();
    if (!holder) return TRV_ERR_ALLOC;
    Plan& p = holder->plan;
    p.algo = algo; p.variant = variant; p.ndims = ndims; p.base = base;
    p.nslices = ndims * (mirror ? 2 : 1);
    if (algo == TRV_ALGO_BUCKET) {
        // ring algorithm (Sec. 2.4): n - 1 steps per phase, every step one block to the next node
        p.dims[0] = dims[0]; p.stride[0] = 1; p.n = dims[0]; p.S = dims[0] - 1;
        p.steps.assign(p.nslices, {});
        for (int c = 0; c < p.nslices; ++c) p.steps[c].assign(p.S, Step{0, c >= ndims ? -1 : 1});
        *out = holder;
        return TRV_OK;
    }
    if (algo == TRV_ALGO_TRIVANCE && ndims == 1 && exact_log(dims[0], 3) < 0) {
        // a ring of any other size: only the bandwidth-optimal form is defined (Sec. 4.4)
        if (variant != TRV_BANDWIDTH_OPTIMAL || dims[0] > TRV_MAX_RANKS) { delete holder; return TRV_ERR_UNSUPPORTED; }
        p.dims[0] = dims[0]; p.stride[0] = 1; p.n = dims[0];
        build_general_ring(p, dims[0]);
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

bool in_send_set(const Plan& p, int c, int t, int dst, int j) {
    if (p.algo == TRV_ALGO_SWING) return (p.reach[c][t + 1][(size_t)dst * p.words + j / 64] >> (j % 64)) & 1;
    if (p.algo == TRV_ALGO_BUCKET) {    // step t: node r sends block r - t - 1 on (mirrored: r + t + 1)
        const int sg = p.steps[c][t].dist, src = ((dst - sg) % p.n + p.n) % p.n;
        return j == ((src - sg * (t + 1)) % p.n + p.n) % p.n;
    }
    if (p.algo == TRV_ALGO_RECDOUB && c >= p.ndims) {     // the mirrored collective is the same pattern on the ring read backwards
        const int n = p.n;
        return in_send_set(p, c - p.ndims, t, (n - dst) % n, (n - j) % n);
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

int general_recv_mask(const Plan& p, int t, int dst, int j) {
    const int n = p.n, dist = p.steps[0][t].dist;
    const int o = ((dst - j) % n + n) % n;
    const int ol = ((o - dist) % n + n) % n, orr = (o + dist) % n;
    int mask = 0;
    if (p.gstep[ol] == t && p.gsgn[ol] > 0) mask |= 1;
    if (orr != ol && p.gstep[orr] == t && p.gsgn[orr] < 0) mask |= 2;
    return mask;
}

void message_bytes_side(const Plan& p, int64_t E, int64_t elem_size, int c, int row, int side, int64_t* out) {
    const int n = p.n;
    if (p.general) {
        // Reduce-Scatter row: the node at offset o sends block (node - o); AllGather row: the parent
        // of the node at offset o, which sits at offset o + sgn * dist, sends it to that node.
        const int t = p.step_of_row(row), dist = p.steps[0][t].dist;
        const bool rs = row < p.S;
        for (int r = 0; r < n; ++r) out[r] = 0;
        for (int o = 1; o < n; ++o) {
            if (p.gstep[o] != t) continue;
            const int sends_right = rs ? (p.gsgn[o] > 0) : (p.gsgn[o] < 0);
            if (sends_right != side) continue;
            const int src_off = rs ? o : ((o + p.gsgn[o] * dist) % n + n) % n;
            for (int r = 0; r < n; ++r) {
                const int j = ((r - src_off) % n + n) % n;
                out[r] += (block_lo(0, E, n, j + 1) - block_lo(0, E, n, j)) * elem_size;
            }
        }
        return;
    }
    std::vector<int64_t> tmp((size_t)n);
    message_bytes(p, E, elem_size, c, row, tmp.data());
    const Step& st = p.steps[c][p.algo == TRV_ALGO_BUCKET ? 0 : p.step_of_row(row)];
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
        // Reduce-Scatter row t, by destination: the block its upstream neighbour passes on; AllGather row t
        // (rows run forwards in both phases), by source: block r - t (mirrored: r + t)
        const int sg = p.steps[c][0].dist;
        for (int r = 0; r < n; ++r) {
            const int off = row < p.S ? sg * (row + 2) : sg * (row - p.S);
            out[r] = blen(((r - off) % n + n) % n);
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
