// Host-side schedule of a Trivance (or comparator) plan: integer work only.
#pragma once
#include <cstddef>
#include <cstdint>
#include <mutex>
#include <memory>
#include <vector>

#include "../../include/trivance.h"

namespace trv {

struct Step {
    int dim;    // torus dimension the step runs along
    int dist;   // ring distance inside that dimension: base^(earlier visits of dim)
};

// What a fused kernel needs to know about one collective (slice).
struct Plan {
    int algo = 0, variant = 0, ndims = 0, n = 0, S = 0, base = 3;
    // concurrent collectives: ndims, or 2 * ndims for a comparator with its mirrored sub-collective
    // (Sec. 2.4); the steps of a mirrored slice carry negated distances
    int nslices = 0;
    int dims[TRV_MAX_DIMS] = {0};
    int stride[TRV_MAX_DIMS] = {0};     // rank = sum_d x_d * stride[d]
    int sdim[TRV_MAX_DIMS] = {0};       // steps in dimension d = log_base a_d
    bool equal_dims = true;
    // steps[c][t]: Reduce-Scatter / latency-form step t of collective c (Sec. 4.1, Sec. 5)
    std::vector<std::vector<Step>> steps;
    // mod[c][t][d] = base^(number of steps <= t of collective c that ran along d): block j is in
    // the message to p at step t iff j_d == p_d (mod mod[c][t][d]) for every d  (closed form Pi)
    std::vector<std::vector<std::vector<int>>> mod;

    // Swing (Sec. 2.4) has no congruence form: reach[c][t][p] = bitset of the blocks rank p still
    // answers for after Reduce-Scatter step t - 1 (its own and all it will forward), t = 0 .. S
    std::vector<std::vector<std::vector<uint64_t>>> reach;
    int words = 0;      // 64-bit words per bitset

    // The ring (Bucket) algorithm on a torus (Sec. 2.4): collective c runs a ring Reduce-Scatter of a_d - 1 steps along
    // dimension c, then along c + 1, ... on the blocks a node still answers for (those that agree with its own coordinates
    // in the dimensions of the earlier phases); the AllGather takes the phases in reverse order.  steps[c][t] = (dimension,
    // +1 or -1 for a mirrored collective) of Reduce-Scatter step t; bk_step[c][t] = the step's number inside its phase,
    // bk_earlier[c][t] = bit mask of the dimensions of the earlier phases, bk_start[c][ph] = first step of phase ph.
    std::vector<std::vector<int>> bk_step, bk_earlier, bk_start;

    // Rings and tori with a side that is no power of three (Sec. 4.4, per dimension as in Sec. 5), bandwidth-optimal
    // form only.  The tree a block follows is the same for every block up to translation, so it is stored once per
    // collective, by the OFFSET o = node - block (coordinate by coordinate, modulo the sides; o is the linear index
    // of that offset vector):  gstep[c][o] = Reduce-Scatter step in which the node at offset o sends its partial on
    // (-1 for the owner, o = 0), along the dimension of that step; gsgn[c][o] = +1 if it sends it to the node `dist`
    // after it, -1 if to the node `dist` before it.
    bool general = false;
    std::vector<std::vector<int8_t>> gstep, gsgn;

    // Host data that the fused launchers derive from the schedule alone, built ONCE by prepare_launch_data() when the plan
    // is created and read-only afterwards (a call writes nothing into the plan): which latency kernel serves the shape
    // (-1: not classified), the line-group kernel's program, the block-tree programs of the stack-machine kernel.
    // Rebuilding them in every call cost 94 us per call on a 27 x 27 torus and 178 us on 32 x 32.
    int lat_kind = -1;
    std::shared_ptr<const void> lines_prog;                     // LnProgram (trv_fused_lines.cu), or empty
    std::vector<std::vector<unsigned short>> tree_progs;        // one per collective (trv_fused_tree.cu), or empty
    bool tree_ready = false;

    // plan-owned scratch for trv_allreduce (STEP family of the latency form), grown on demand under
    // trv_plan_s::scratch_mu; scratch_device = ordinal of the GPU it was allocated on (-1: none yet)
    void* scratch = nullptr;
    size_t scratch_bytes = 0;
    int scratch_device = -1;

    int rows() const { return variant == TRV_BANDWIDTH_OPTIMAL ? 2 * S : S; }
    // schedule step behind a row: AllGather rows mirror the Reduce-Scatter steps
    int step_of_row(int row) const { return row < S ? row : 2 * S - 1 - row; }
    // Bucket: the Reduce-Scatter step with the same dimension, step inside the phase and earlier dimensions as `row`
    // (AllGather rows walk the phases backwards, the steps of a phase forwards)
    int bucket_step(int c, int row) const {
        if (row < S) return row;
        int i = row - S;
        for (int ph = ndims - 1; ph >= 0; --ph) {
            const int len = (ph + 1 < ndims ? bk_start[c][ph + 1] : S) - bk_start[c][ph];
            if (i < len) return bk_start[c][ph] + i;
            i -= len;
        }
        return 0;
    }
    // the schedule step whose (dimension, distance) a row uses
    int row_step(int c, int row) const { return algo == TRV_ALGO_BUCKET ? bucket_step(c, row) : step_of_row(row); }
    int coord(int r, int d) const { return (r / stride[d]) % dims[d]; }
    int shift(int r, int d, int delta) const {
        int a = dims[d], x = coord(r, d);
        int y = ((x + delta) % a + a) % a;
        return r + (y - x) * stride[d];
    }
    // coordinate-wise r - j modulo the sides: the offset of node r from block j (and back: j + o)
    int sub(int r, int j) const {
        int o = 0;
        for (int d = 0; d < ndims; ++d) o += ((coord(r, d) - coord(j, d) + dims[d]) % dims[d]) * stride[d];
        return o;
    }
    int add(int j, int o) const {
        int r = 0;
        for (int d = 0; d < ndims; ++d) r += ((coord(j, d) + coord(o, d)) % dims[d]) * stride[d];
        return r;
    }
};



// element ranges (global indices)
inline int64_t slice_lo(int64_t E, int D, int c) { return (int64_t)(((unsigned __int128)c * (unsigned __int128)E) / D); }
inline int64_t block_lo(int64_t lo, int64_t hi, int n, int j) {
    return lo + (int64_t)(((unsigned __int128)j * (unsigned __int128)(hi - lo)) / n);
}

bool in_send_set(const Plan& p, int c, int t, int dst, int j);
// Bucket: is block j in the message node src passes to its neighbour in `row` (Reduce-Scatter or AllGather)?
bool bucket_sends(const Plan& p, int c, int row, int src, int j);
// peers a rank sends to in step (dim, dist); returns how many; dir = +1 / -1, hops = links crossed
int send_peers(const Plan& p, int r, int dim, int dist, int peer[2], int dir[2], int hops[2]);
// message bytes of one row, indexed by destination (row < S) or by source (AllGather rows)
// (not for general rings)
void message_bytes(const Plan& p, int64_t E, int64_t elem_size, int c, int row, int64_t* out);
// bytes of the message every rank SENDS to its peer number `side` (0: first peer -- Trivance: the
// left one; 1: second peer) in one row; 0 where it sends none.  Every kind of plan.
void message_bytes_side(const Plan& p, int64_t E, int64_t elem_size, int c, int row, int side, int64_t* out);
// sides of any size: what `dst` receives for block j in Reduce-Scatter step t of collective c: bit 0 = a partial
// from the node before it along the step's dimension, bit 1 = one from the node after it
int general_recv_mask(const Plan& p, int c, int t, int dst, int j);

}  // namespace trv

struct trv_plan_s {
    trv::Plan plan;
    std::mutex scratch_mu;      // guards plan.scratch* (the only mutable part of a plan)
};

namespace trv {
trv_status_t build_plan(const int32_t* dims, int32_t ndims, int variant, int algo, trv_plan_s** out);
void prepare_launch_data(Plan& p);      // trv_api.cu: fills lat_kind, lines_prog, tree_progs
}
