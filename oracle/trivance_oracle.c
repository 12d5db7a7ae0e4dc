/*
 * Trivance AllReduce -- plain CPU oracle.  TEST INFRASTRUCTURE ONLY.
 *
 * This file is the slow, literal restatement of what the Trivance paper's
 * AllReduce computes, used to check the CUDA library.  Only tests, the smoke
 * check and the benchmark's CPU-baseline leg may call it; the product never
 * does.  It shares no code, header, table or constant with the CUDA path.
 *
 * What it follows (paper sections):
 *   - problem statement: every rank ends with the element-wise reduction of
 *     all n input vectors (Sec. 2.2);
 *   - peers pi(r,k,n) = (r - 3^k, r + 3^k) mod n (Sec. 4.1);
 *   - latency-optimal form: log3 n steps, whole vector to both peers, joint
 *     reduction of the two received vectors with the local partial (Sec. 4.2);
 *   - bandwidth-optimal form: Reduce-Scatter over n blocks, block sets = the
 *     sets BlockPropagation defines (Algorithm 1, Sec. 4.3), grown step by step
 *     from the peers of each step, then AllGather in reverse order (Sec. 4.1);
 *   - D-dimensional tori: D collectives on 1/D of the vector each, every
 *     collective on a different dimension in every step (Sec. 5);
 *   - congestion c_k = number of messages sharing a link in a step under
 *     deterministic shortest-path routing inside one dimension (Sec. 2.1,
 *     Fig. 1, App. E); Bruck-style, Recursive-Doubling, Swing and ring (Bucket)
 *     schedules, each optionally with its mirrored sub-collective, only as
 *     link-load comparators (Sec. 2.4, Fig. 1, Table 1, App. B);
 *   - rings whose size is no power of three, bandwidth-optimal form (Sec. 4.4):
 *     see the block of comments in front of gen_steps().
 *
 * Readings where the paper is silent:
 *   - a joint reduction adds as (from_left + own) + from_right, where "left"
 *     is the peer r - 3^k.  PARITY UNPINNED by the paper: any fixed order
 *     satisfies every published fact; the tests pin it to this reading with an
 *     independent ternary-tree evaluator.
 *   - slice c of a D-dim torus is elements [floor(cE/D), floor((c+1)E/D));
 *     block j of a slice [lo,hi) is [lo+floor(j*L/n), lo+floor((j+1)*L/n)),
 *     L = hi-lo; ranks are linearised r = x0 + a0*x1 + a0*a1*x2 ...; block j
 *     is owned by linear rank j; collective c uses, at step t, the next
 *     dimension in round-robin order starting at c that still has steps left,
 *     with distance 3^(earlier visits of that dimension).  PARITY UNPINNED by
 *     the paper beyond "collective 0 starts horizontal, collective 1 vertical
 *     and they swap every step" (Sec. 5).
 *   - int32 addition wraps modulo 2^32.
 *   - the mirrored sub-collective of a comparator (Sec. 2.4) is the same pattern with every
 *     displacement and direction of travel reversed, on the second half of the vector; for
 *     Recursive Doubling that is the XOR pattern on the ring counted backwards (r -> -r mod n).
 *     PARITY UNPINNED by the paper for Recursive Doubling (App. B counts one collective's
 *     congestion there); for Swing and the ring algorithm App. B's per-step congestion pins it.
 *   - the ring (Bucket) algorithm sends block (r - t - 1) mod n in Reduce-Scatter step t and block
 *     (r - t) mod n in AllGather step t, always to r + 1: block j ends at node j.  Any such
 *     numbering gives the same loads when the blocks have equal length.
 *     On a torus (Sec. 2.4's two sentences on it) the ring algorithm runs dimension after dimension, collective c
 *     starting with dimension c, each phase on the blocks that agree with the node in the earlier dimensions; the
 *     AllGather takes the phases in reverse order.  PARITY UNPINNED by the paper beyond Table 2's Theta = 1 and the
 *     step count, which the tests check; the sums themselves are pinned by the plain column sums.
 *
 * Floating point: binary32 (or binary64 for the error-bound checks), one add
 * at a time, no contraction, no reassociation.  Compile with
 *   gcc -O2 -ffp-contract=off -fno-fast-math -std=c99
 *
 * All functions work on an element WINDOW [e0,e1) of a global per-rank vector
 * of E elements: columns are independent, so a window gives exactly the values
 * the full run would give for those columns.  Arrays are [n][w], w = e1-e0.
 */
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

#define ORC_MAX_DIMS 8

enum { ORC_OK = 0, ORC_BAD_ARG = 1, ORC_UNDEFINED = 2, ORC_NOMEM = 3, ORC_INTERNAL = 4 };
enum { ORC_TRIVANCE = 0, ORC_BRUCK = 1, ORC_RECDOUB = 2, ORC_SWING = 3, ORC_BUCKET = 4, ORC_MIRROR = 16, ORC_SINGLE = 32 };
enum { ORC_LATENCY = 0, ORC_BANDWIDTH = 1 };
enum { ORC_I32 = 0, ORC_F32 = 1, ORC_F64 = 2 };

typedef struct {
    int algo, ndims, n, S;          /* S = steps per phase, summed over dimensions */
    int nsl;                        /* concurrent collectives (slices): ndims, or 2*ndims when mirrored */
    int base;                       /* 3 (Trivance, Bruck) or 2 (Recursive Doubling, Swing) */
    int dims[ORC_MAX_DIMS];
    int stride[ORC_MAX_DIMS];       /* rank = sum x_d * stride_d */
    int sdim[ORC_MAX_DIMS];         /* steps spent in dimension d = log_base a_d */
} orc_topo;

static int ilog_exact(int a, int base) {       /* log_base a, or -1 if a is no power */
    int s = 0;
    if (a < 1) return -1;
    while (a > 1) { if (a % base) return -1; a /= base; ++s; }
    return s;
}

/* `algo` may carry the ORC_MIRROR flag (comparators on rings only): the collective then runs a
 * second time with every direction reversed, the two sharing the vector half and half -- the
 * "mirrored sub-collective" by which the one-port comparators use both ports (Sec. 2.4). */
static int topo_init(orc_topo *tp, const int32_t *dims, int ndims, int algo) {
    if (!dims || ndims < 1 || ndims > ORC_MAX_DIMS) return ORC_BAD_ARG;
    int mirror = (algo & ORC_MIRROR) ? 1 : 0, single = (algo & ORC_SINGLE) ? 1 : 0;
    algo &= ~(ORC_MIRROR | ORC_SINGLE);
    if (algo < ORC_TRIVANCE || algo > ORC_BUCKET) return ORC_BAD_ARG;
    if (mirror && algo == ORC_TRIVANCE) return ORC_BAD_ARG;
    if (mirror && ndims != 1 && algo != ORC_RECDOUB && algo != ORC_SWING && algo != ORC_BUCKET) return ORC_BAD_ARG;
    /* ORC_SINGLE: ONE collective on the whole vector that walks through the dimensions in turn -- how the
     * latency-optimal Recursive Doubling and Swing use a torus ("only a single port per node", App. B) */
    if (single && (mirror || (algo != ORC_RECDOUB && algo != ORC_SWING))) return ORC_BAD_ARG;
    tp->algo = algo; tp->ndims = ndims; tp->nsl = single ? 1 : ndims * (mirror ? 2 : 1);
    tp->base = (algo == ORC_RECDOUB || algo == ORC_SWING) ? 2 : 3;
    /* Recursive Doubling, Swing and Bucket on tori (Sec. 2.4): one collective per dimension, each with its mirrored
     * sub-collective when asked for (2D collectives on 1/(2D) of the vector each). */
    if (algo == ORC_BUCKET) {
        /* The ring algorithm, any sides >= 2 (Sec. 2.4): a ring Reduce-Scatter of a_d - 1 steps along one dimension
         * after the other on the partially reduced data, then the AllGather phases in reverse order.  Collective c
         * starts with dimension c; see bucket_where. */
        long long nn = 1; tp->S = 0;
        for (int d = 0; d < ndims; ++d) {
            if (dims[d] < 2 || dims[d] > 4096) return ORC_BAD_ARG;
            tp->dims[d] = dims[d]; tp->stride[d] = (int)nn; tp->sdim[d] = dims[d] - 1;
            nn *= dims[d]; tp->S += dims[d] - 1;
            if (nn > 4096) return ORC_BAD_ARG;
        }
        tp->n = (int)nn;
        return ORC_OK;
    }
    long long n = 1; tp->S = 0;
    for (int d = 0; d < ndims; ++d) {
        int s = ilog_exact(dims[d], tp->base);
        if (s < 1) return (dims[d] >= 2) ? ORC_UNDEFINED : ORC_BAD_ARG;
        tp->dims[d] = dims[d]; tp->sdim[d] = s; tp->stride[d] = (int)n;
        n *= dims[d]; tp->S += s;
        if (n > (1 << 20)) return ORC_BAD_ARG;
    }
    tp->n = (int)n;
    return ORC_OK;
}

static int ipow(int b, int e) { int r = 1; while (e-- > 0) r *= b; return r; }

/* Step list of collective (slice) c (Sec. 5): round-robin over dimensions,
 * starting at dimension c, skipping dimensions whose steps are used up; the
 * distance in a dimension grows by the base each time it is revisited. */
/* Swing's signed distance rho(k) = sum_{i<=k} (-2)^i = 1, -1, 3, -5, 11, ... (Sec. 2.4) */
static int swing_rho(int k) { int r = 0, p = 1; for (int i = 0; i <= k; ++i) { r += p; p *= -2; } return r; }

/* A mirrored slice (c >= ndims) gets negated distances: send_peers reverses everything for them. */
static void step_list(const orc_topo *tp, int c, int *sdim_out, int *sdist_out) {
    int visits[ORC_MAX_DIMS] = {0};
    int mir = (c >= tp->ndims) ? -1 : 1;
    int cur = c % tp->ndims;
    for (int t = 0; t < tp->S; ++t) {
        int d = cur;
        while (visits[d] >= tp->sdim[d]) d = (d + 1) % tp->ndims;
        sdim_out[t] = d;
        sdist_out[t] = mir * ((tp->algo == ORC_SWING) ? swing_rho(visits[d]) : ipow(tp->base, visits[d]));
        visits[d]++;
        cur = (d + 1) % tp->ndims;
    }
}

/* rank reached from r by moving delta positions along dimension d (wraps). */
static int shift_rank(const orc_topo *tp, int r, int d, int delta) {
    int a = tp->dims[d], st = tp->stride[d];
    int x = (r / st) % a;
    int y = ((x + delta) % a + a) % a;
    return r + (y - x) * st;
}

/* Bucket on a torus (Sec. 2.4).  Collective c walks the dimensions c, c + 1, ... (mod D); in the phase of dimension d
 * the a_d nodes of every line along d run the ring algorithm on the blocks they still answer for: those that agree
 * with the node's own coordinates in the dimensions of the earlier phases (block j ends at node j).  Row numbering:
 * Reduce-Scatter rows 0 .. S-1 take the phases in order, AllGather rows S .. 2S-1 take them in reverse order; inside
 * a phase the steps s = 0 .. a_d - 2 run forwards in both.  Returns the dimension, the step inside the phase and the
 * bit mask of the dimensions of the earlier phases. */
static void bucket_where(const orc_topo *tp, int c, int row, int *d, int *s, int *earlier) {
    int D = tp->ndims, d0 = c % D, ag = row >= tp->S, i = ag ? row - tp->S : row;
    for (int k = 0; k < D; ++k) {
        int ph = ag ? D - 1 - k : k, dd = (d0 + ph) % D, len = tp->dims[dd] - 1;
        if (i < len) {
            int mask = 0;
            for (int q = 0; q < ph; ++q) mask |= 1 << ((d0 + q) % D);
            *d = dd; *s = i; *earlier = mask;
            return;
        }
        i -= len;
    }
    *d = 0; *s = 0; *earlier = 0;
}

/* The blocks of the message node r passes to its neighbour r + sg e_d in that row: Reduce-Scatter step s carries the
 * blocks whose d-coordinate is r_d - sg (s + 1), AllGather step s those with r_d - sg s (the ring rule "block
 * r - t - 1, then block r - t", Sec. 2.4), both restricted to the blocks that agree with r in the earlier dimensions. */
static void bucket_message(const orc_topo *tp, int r, int row, int d, int s, int earlier, int sg, uint8_t *set) {
    int a = tp->dims[d], ag = row >= tp->S;
    int want = (((r / tp->stride[d]) % a - sg * (s + (ag ? 0 : 1))) % a + a) % a;
    for (int j = 0; j < tp->n; ++j) {
        int ok = ((j / tp->stride[d]) % a) == want;
        for (int q = 0; q < tp->ndims && ok; ++q)
            if (((earlier >> q) & 1) && (j / tp->stride[q]) % tp->dims[q] != (r / tp->stride[q]) % tp->dims[q]) ok = 0;
        set[j] = (uint8_t)ok;
    }
}

/* Peers a rank SENDS to in a step of (dim, dist).  Returns their number;
 * dir = +1/-1 ring direction of travel, hops = links crossed.
 *   Trivance: left = r - dist (travels -), right = r + dist (travels +)  (Sec. 4.1)
 *   Bruck (as drawn in Fig. 1): r + dist and r + 2*dist, both travelling +  (Sec. 2.4)
 *   Recursive Doubling: coordinate XOR dist; the lower rank of a pair sends +. */
static int send_peers(const orc_topo *tp, int r, int d, int dist, int *peer, int *dir, int *hops) {
    if (tp->algo == ORC_TRIVANCE) {
        peer[0] = shift_rank(tp, r, d, -dist); dir[0] = -1; hops[0] = dist;
        peer[1] = shift_rank(tp, r, d, +dist); dir[1] = +1; hops[1] = dist;
        return 2;
    }
    {
        /* comparators: a negative distance is the mirrored collective -- same pattern, every
         * displacement and direction of travel reversed */
        int sg = dist < 0 ? -1 : 1, a = dist < 0 ? -dist : dist;
        if (tp->algo == ORC_BRUCK) {
            peer[0] = shift_rank(tp, r, d, sg * a);     dir[0] = sg; hops[0] = a;
            peer[1] = shift_rank(tp, r, d, sg * 2 * a); dir[1] = sg; hops[1] = 2 * a;
            return 2;
        }
        if (tp->algo == ORC_SWING) {
            /* pi(r,k) = r + rho(k) for even r, r - rho(k) for odd r (Sec. 2.4); here dist = +-rho(k), whose
             * own sign is part of the pattern.  The message travels the short way round: |rho| < n/2. */
            int st = tp->stride[d], x = (r / st) % tp->dims[d];
            int delta = (x % 2 == 0) ? dist : -dist;
            peer[0] = shift_rank(tp, r, d, delta); dir[0] = delta > 0 ? +1 : -1; hops[0] = delta > 0 ? delta : -delta;
            return 1;
        }
        if (tp->algo == ORC_BUCKET) {       /* every step: one block to the next node of the ring */
            peer[0] = shift_rank(tp, r, d, sg); dir[0] = sg; hops[0] = 1;
            return 1;
        }
        {   /* Recursive Doubling: the pair (x, x XOR a); mirrored: the ring read backwards */
            int st = tp->stride[d], x = (r / st) % tp->dims[d];
            int xm = sg > 0 ? x : (tp->dims[d] - x) % tp->dims[d];
            int ym = xm ^ a;
            int y = sg > 0 ? ym : (tp->dims[d] - ym) % tp->dims[d];
            peer[0] = r + (y - x) * st; dir[0] = (ym > xm) ? sg : -sg; hops[0] = a;
            return 1;
        }
    }
}

/* The set Algorithm 1 (BlockPropagation, Sec. 4.3) defines, computed in the oracle's own form:
 * a block that rank r answers for at step `step` reaches, one step at a time, every rank that can
 * be got to from r by hops taken in steps of strictly increasing number step <= k_1 < k_2 < ... < S.
 * So the set grows step by step: the ranks known BEFORE step k (r itself and everything reached in
 * steps step..k-1) each add their peers of step k.  blocks[] gets a 1 for every rank reached; r
 * itself is a source only.  Generalised from the ring's pi(r,k,n) to one collective's step list. */
static void block_propagation(const orc_topo *tp, const int *sdim, const int *sdist,
                              int r, int step, uint8_t *blocks) {
    int n = tp->n, nsrc = 1;
    int *src = (int *)malloc(sizeof(int) * (size_t)n * 2);   /* sources so far, in the order they were reached */
    uint8_t *seen = (uint8_t *)calloc((size_t)n, 1);
    if (!src || !seen) { free(src); free(seen); return; }
    src[0] = r; seen[r] = 1;
    for (int k = step; k < tp->S; ++k) {
        int before = nsrc;                                   /* ranks reached in step k do not send again in step k */
        for (int i = 0; i < before; ++i) {
            int peer[2], dir[2], hops[2];
            int np = send_peers(tp, src[i], sdim[k], sdist[k], peer, dir, hops);
            for (int j = 0; j < np; ++j) {
                blocks[peer[j]] = 1;
                if (!seen[peer[j]] && nsrc < 2 * n) { seen[peer[j]] = 1; src[nsrc++] = peer[j]; }
            }
        }
    }
    free(src); free(seen);
}

/* Blocks a rank sends to peer p in Reduce-Scatter step k: p's own block plus
 * everything p still has to forward in later steps (Sec. 4.1 / 4.3). */
static void send_set(const orc_topo *tp, const int *sdim, const int *sdist, int p, int k, uint8_t *set) {
    memset(set, 0, (size_t)tp->n);
    set[p] = 1;
    block_propagation(tp, sdim, sdist, p, k + 1, set);
}

static void slice_bounds(int64_t E, int D, int c, int64_t *lo, int64_t *hi) {
    *lo = (int64_t)(((__int128)c * E) / D);
    *hi = (int64_t)(((__int128)(c + 1) * E) / D);
}
static int64_t block_bound(int64_t lo, int64_t hi, int n, int j) {
    return lo + (int64_t)(((__int128)j * (hi - lo)) / n);
}
static int64_t clampi(int64_t v, int64_t a, int64_t b) { return v < a ? a : (v > b ? b : v); }

/* ------------------------------------------------------------------ exported helpers */

int orc_num_steps(const int32_t *dims, int ndims, int algo, int *n_out, int *S_out) {
    orc_topo tp; int rc = topo_init(&tp, dims, ndims, algo);
    if (rc) return rc;
    if (n_out) *n_out = tp.n;
    if (S_out) *S_out = tp.S;
    return ORC_OK;
}

int orc_step_list(const int32_t *dims, int ndims, int algo, int c, int32_t *dim_out, int32_t *dist_out) {
    orc_topo tp; int rc = topo_init(&tp, dims, ndims, algo);
    if (rc) return rc;
    if (tp.algo == ORC_BUCKET) return ORC_UNDEFINED;     /* n - 1 single-block steps: see orc_link_loads */
    if (c < 0 || c >= tp.nsl) return ORC_BAD_ARG;
    int sd[64], sx[64];
    step_list(&tp, c, sd, sx);
    for (int t = 0; t < tp.S; ++t) { dim_out[t] = sd[t]; dist_out[t] = sx[t]; }
    return ORC_OK;
}

/* peers_out[2*r+0] = first peer (Trivance: left), [2*r+1] = second (Trivance: right;
 * Recursive Doubling: -1). */
int orc_peers(const int32_t *dims, int ndims, int algo, int c, int step, int32_t *peers_out) {
    orc_topo tp; int rc = topo_init(&tp, dims, ndims, algo);
    if (rc) return rc;
    if (tp.algo == ORC_BUCKET) return ORC_UNDEFINED;     /* n - 1 single-block steps: see orc_link_loads */
    if (c < 0 || c >= tp.nsl || step < 0 || step >= tp.S) return ORC_BAD_ARG;
    int sd[64], sx[64];
    step_list(&tp, c, sd, sx);
    for (int r = 0; r < tp.n; ++r) {
        int peer[2] = {-1, -1}, dir[2], hops[2];
        send_peers(&tp, r, sd[step], sx[step], peer, dir, hops);
        peers_out[2 * r] = peer[0]; peers_out[2 * r + 1] = peer[1];
    }
    return ORC_OK;
}

/* Raw Algorithm 1: marks[] (n bytes, caller-zeroed or not: it is cleared here). */
int orc_block_propagation(const int32_t *dims, int ndims, int algo, int c, int r, int step, uint8_t *marks) {
    orc_topo tp; int rc = topo_init(&tp, dims, ndims, algo);
    if (rc) return rc;
    if (tp.algo == ORC_BUCKET) return ORC_UNDEFINED;     /* n - 1 single-block steps: see orc_link_loads */
    if (c < 0 || c >= tp.nsl || r < 0 || r >= tp.n || step < 0) return ORC_BAD_ARG;
    int sd[64], sx[64];
    step_list(&tp, c, sd, sx);
    memset(marks, 0, (size_t)tp.n);
    block_propagation(&tp, sd, sx, r, step, marks);
    return ORC_OK;
}

/* Blocks sent to peer p in Reduce-Scatter step k of collective c. */
int orc_send_set(const int32_t *dims, int ndims, int algo, int c, int p, int k, uint8_t *set) {
    orc_topo tp; int rc = topo_init(&tp, dims, ndims, algo);
    if (rc) return rc;
    if (tp.algo == ORC_BUCKET) return ORC_UNDEFINED;     /* n - 1 single-block steps: see orc_link_loads */
    if (c < 0 || c >= tp.nsl || p < 0 || p >= tp.n || k < 0 || k >= tp.S) return ORC_BAD_ARG;
    int sd[64], sx[64];
    step_list(&tp, c, sd, sx);
    send_set(&tp, sd, sx, p, k, set);
    return ORC_OK;
}

/* bounds_out[0..n]: element index where block j of slice c starts (global indices). */
int orc_block_bounds(int64_t E, int D, int n, int c, int64_t *bounds_out) {
    if (E < 0 || D < 1 || n < 1 || c < 0 || c >= D) return ORC_BAD_ARG;
    int64_t lo, hi; slice_bounds(E, D, c, &lo, &hi);
    for (int j = 0; j <= n; ++j) bounds_out[j] = block_bound(lo, hi, n, j);
    return ORC_OK;
}

/* Naive sequential binary32 sum over ranks u = 0..n-1, per column. */
void orc_naive_sum_f32(int n, int64_t w, const float *in, float *out) {
    for (int64_t e = 0; e < w; ++e) {
        float acc = in[e];
        for (int u = 1; u < n; ++u) acc = acc + in[(int64_t)u * w + e];
        out[e] = acc;
    }
}

/* ------------------------------------------------------------------ data path (Trivance) */

typedef struct {
    /* all optional (NULL allowed); each is an array of n int64, bytes per rank */
    int64_t *sent_rs;       /* bytes sent in the Reduce-Scatter phase (or the single latency phase) */
    int64_t *sent_ag;       /* bytes sent in the AllGather phase */
    int64_t *reduced;       /* bytes entering the reducer (both messages + local partial) */
} orc_counters;

#define DEFINE_PATH(T, SUFFIX, ADD)                                                                        \
/* Latency-optimal form (Sec. 4.2): each step every rank copies its whole current partial into a          \
 * message for both peers; when both messages are in, it reduces (left + own) + right. */                 \
static int latency_slice_##SUFFIX(const orc_topo *tp, const int *sdim, const int *sdist,                   \
                                  int64_t w, int64_t c0, int64_t c1, const T *in, T *out,                  \
                                  int max_steps, orc_counters *ctr) {                                      \
    int n = tp->n; int64_t wc = c1 - c0;                                                                   \
    if (wc <= 0) return ORC_OK;                                                                            \
    T *partial = (T *)malloc(sizeof(T) * (size_t)n * (size_t)wc);                                          \
    T *message = (T *)malloc(sizeof(T) * (size_t)n * (size_t)wc);                                          \
    if (!partial || !message) { free(partial); free(message); return ORC_NOMEM; }                          \
    for (int r = 0; r < n; ++r) memcpy(partial + (size_t)r * wc, in + (size_t)r * w + c0, sizeof(T) * wc); \
    int steps = (max_steps >= 0 && max_steps < tp->S) ? max_steps : tp->S;                                 \
    for (int t = 0; t < steps; ++t) {                                                                      \
        /* every rank builds its outgoing message first ... */                                            \
        memcpy(message, partial, sizeof(T) * (size_t)n * (size_t)wc);                                      \
        /* ... then every rank, having received both, reduces */                                          \
        for (int p = 0; p < n; ++p) {                                                                      \
            const T *from_left  = message + (size_t)shift_rank(tp, p, sdim[t], -sdist[t]) * wc;            \
            const T *from_right = message + (size_t)shift_rank(tp, p, sdim[t], +sdist[t]) * wc;            \
            T *own = partial + (size_t)p * wc;                                                             \
            for (int64_t e = 0; e < wc; ++e) own[e] = ADD(ADD(from_left[e], own[e]), from_right[e]);       \
            if (ctr && ctr->sent_rs) ctr->sent_rs[p] += 2 * (int64_t)sizeof(T) * wc;                       \
            if (ctr && ctr->reduced) ctr->reduced[p] += 3 * (int64_t)sizeof(T) * wc;                       \
        }                                                                                                  \
    }                                                                                                      \
    for (int r = 0; r < n; ++r) memcpy(out + (size_t)r * w + c0, partial + (size_t)r * wc, sizeof(T) * wc);\
    free(partial); free(message);                                                                          \
    return ORC_OK;                                                                                         \
}                                                                                                          \
                                                                                                           \
/* Bandwidth-optimal form (Sec. 4.1, 4.3): Reduce-Scatter with Algorithm-1 block sets and literal         \
 * messages, then AllGather with the steps in reverse order. */                                           \
static int bandwidth_slice_##SUFFIX(const orc_topo *tp, const int *sdim, const int *sdist,                 \
                                    int64_t slo, int64_t shi, int64_t e0, int64_t e1, int64_t w,           \
                                    const T *in, T *out, orc_counters *ctr) {                              \
    int n = tp->n, S = tp->S, rc = ORC_OK;                                                                 \
    int64_t c0 = clampi(slo, e0, e1) - e0, c1 = clampi(shi, e0, e1) - e0, wc = c1 - c0;                    \
    if (wc <= 0) return ORC_OK;                                                                            \
    /* block j restricted to the window, as columns of the slice-local arrays */                          \
    int64_t *bs = (int64_t *)malloc(sizeof(int64_t) * (size_t)(n + 1));                                    \
    T *partial = (T *)malloc(sizeof(T) * (size_t)n * (size_t)wc);                                          \
    T *msg = (T *)malloc(sizeof(T) * (size_t)n * 2 * (size_t)wc);   /* [rank][side][<=wc] */               \
    int64_t *mlen = (int64_t *)malloc(sizeof(int64_t) * (size_t)n * 2);                                    \
    uint8_t *mset = (uint8_t *)malloc((size_t)n * 2 * (size_t)n);   /* block set of each message */        \
    uint8_t *have = (uint8_t *)calloc((size_t)n, (size_t)n);        /* finished blocks held */             \
    uint8_t *snap = (uint8_t *)malloc((size_t)n * (size_t)n);                                              \
    if (!bs || !partial || !msg || !mlen || !mset || !have || !snap) { rc = ORC_NOMEM; goto done; }        \
    for (int j = 0; j <= n; ++j) bs[j] = clampi(block_bound(slo, shi, n, j), e0, e1) - e0 - c0;            \
    for (int r = 0; r < n; ++r) memcpy(partial + (size_t)r * wc, in + (size_t)r * w + c0, sizeof(T) * wc); \
    /* ---- Reduce-Scatter */                                                                             \
    for (int t = 0; t < S; ++t) {                                                                          \
        for (int r = 0; r < n; ++r) {                                                                      \
            int peer[2], dir[2], hops[2];                                                                  \
            send_peers(tp, r, sdim[t], sdist[t], peer, dir, hops);                                         \
            for (int side = 0; side < 2; ++side) {                                                         \
                uint8_t *set = mset + ((size_t)r * 2 + side) * n;                                          \
                T *m = msg + ((size_t)r * 2 + side) * wc; int64_t len = 0;                                 \
                send_set(tp, sdim, sdist, peer[side], t, set);                                             \
                for (int j = 0; j < n; ++j) if (set[j]) {                                                  \
                    memcpy(m + len, partial + (size_t)r * wc + bs[j], sizeof(T) * (size_t)(bs[j+1]-bs[j]));\
                    len += bs[j + 1] - bs[j];                                                              \
                }                                                                                          \
                mlen[(size_t)r * 2 + side] = len;                                                          \
                if (ctr && ctr->sent_rs) ctr->sent_rs[r] += (int64_t)sizeof(T) * len;                      \
            }                                                                                              \
        }                                                                                                  \
        for (int p = 0; p < n; ++p) {                                                                      \
            int ql = shift_rank(tp, p, sdim[t], -sdist[t]);   /* left peer: its message to ITS right */   \
            int qr = shift_rank(tp, p, sdim[t], +sdist[t]);   /* right peer: its message to ITS left */   \
            const uint8_t *setl = mset + ((size_t)ql * 2 + 1) * n, *setr = mset + ((size_t)qr * 2 + 0) * n;\
            const T *ml = msg + ((size_t)ql * 2 + 1) * wc, *mr = msg + ((size_t)qr * 2 + 0) * wc;          \
            int64_t off = 0;                                                                               \
            if (memcmp(setl, setr, (size_t)n)) { rc = ORC_INTERNAL; goto done; }                           \
            for (int j = 0; j < n; ++j) if (setl[j]) {                                                     \
                T *own = partial + (size_t)p * wc + bs[j]; int64_t bl = bs[j + 1] - bs[j];                 \
                for (int64_t e = 0; e < bl; ++e) own[e] = ADD(ADD(ml[off + e], own[e]), mr[off + e]);      \
                off += bl;                                                                                 \
            }                                                                                              \
            if (off != mlen[(size_t)ql * 2 + 1] || off != mlen[(size_t)qr * 2]) { rc = ORC_INTERNAL; goto done; } \
            if (ctr && ctr->reduced) ctr->reduced[p] += 3 * (int64_t)sizeof(T) * off;                      \
        }                                                                                                  \
    }                                                                                                      \
    /* ---- AllGather: reverse step order, every rank forwards all finished blocks it holds */            \
    for (int r = 0; r < n; ++r) have[(size_t)r * n + r] = 1;                                               \
    for (int t = S - 1; t >= 0; --t) {                                                                     \
        memcpy(snap, have, (size_t)n * (size_t)n);                                                         \
        for (int r = 0; r < n; ++r) {                                                                      \
            T *m = msg + (size_t)r * 2 * wc; int64_t len = 0;       /* same message to both peers */       \
            for (int j = 0; j < n; ++j) if (snap[(size_t)r * n + j]) {                                     \
                memcpy(m + len, partial + (size_t)r * wc + bs[j], sizeof(T) * (size_t)(bs[j+1]-bs[j]));    \
                len += bs[j + 1] - bs[j];                                                                  \
            }                                                                                              \
            if (ctr && ctr->sent_ag) ctr->sent_ag[r] += 2 * (int64_t)sizeof(T) * len;                      \
        }                                                                                                  \
        for (int p = 0; p < n; ++p) {                                                                      \
            for (int side = 0; side < 2; ++side) {                                                         \
                int q = shift_rank(tp, p, sdim[t], side ? +sdist[t] : -sdist[t]);                          \
                const T *m = msg + (size_t)q * 2 * wc; int64_t off = 0;                                    \
                for (int j = 0; j < n; ++j) if (snap[(size_t)q * n + j]) {                                 \
                    int64_t bl = bs[j + 1] - bs[j];                                                        \
                    if (have[(size_t)p * n + j]) { rc = ORC_INTERNAL; goto done; }  /* never twice */      \
                    memcpy(partial + (size_t)p * wc + bs[j], m + off, sizeof(T) * (size_t)bl);             \
                    have[(size_t)p * n + j] = 1; off += bl;                                                \
                }                                                                                          \
            }                                                                                              \
        }                                                                                                  \
    }                                                                                                      \
    for (size_t i = 0; i < (size_t)n * (size_t)n; ++i) if (!have[i]) { rc = ORC_INTERNAL; goto done; }     \
    for (int r = 0; r < n; ++r) memcpy(out + (size_t)r * w + c0, partial + (size_t)r * wc, sizeof(T) * wc);\
done:                                                                                                      \
    free(bs); free(partial); free(msg); free(mlen); free(mset); free(have); free(snap);                    \
    return rc;                                                                                             \
}

#define ADD_WRAP(a, b) ((uint32_t)((a) + (b)))
#define ADD_FP(a, b) ((a) + (b))
DEFINE_PATH(uint32_t, i32, ADD_WRAP)
DEFINE_PATH(float, f32, ADD_FP)
DEFINE_PATH(double, f64, ADD_FP)

/*
 * Trivance AllReduce over the window [e0,e1) of per-rank vectors of E elements.
 *   in, out : [n][w] row-major, w = e1-e0 (out may not alias in)
 *   variant : ORC_LATENCY or ORC_BANDWIDTH
 *   max_steps: latency form only: stop after this many steps (<0 = run all); lets
 *              tests look at the partials after step k.
 *   sent_rs/sent_ag/reduced: optional [n] int64 byte counters (accumulated into).
 */
int orc_allreduce(const int32_t *dims, int ndims, int variant, int dtype,
                  int64_t E, int64_t e0, int64_t e1, const void *in, void *out, int max_steps,
                  int64_t *sent_rs, int64_t *sent_ag, int64_t *reduced) {
    orc_topo tp; int rc = topo_init(&tp, dims, ndims, ORC_TRIVANCE);
    if (rc) return rc;
    if (E < 0 || e0 < 0 || e1 < e0 || e1 > E || !in || !out) return ORC_BAD_ARG;
    if (variant != ORC_LATENCY && variant != ORC_BANDWIDTH) return ORC_BAD_ARG;
    if (dtype != ORC_I32 && dtype != ORC_F32 && dtype != ORC_F64) return ORC_BAD_ARG;
    orc_counters ctr = { sent_rs, sent_ag, reduced };
    int64_t w = e1 - e0;
    for (int c = 0; c < tp.ndims; ++c) {
        int sd[64], sx[64];
        int64_t slo, shi;
        step_list(&tp, c, sd, sx);
        slice_bounds(E, tp.ndims, c, &slo, &shi);
        int64_t c0 = clampi(slo, e0, e1) - e0, c1 = clampi(shi, e0, e1) - e0;
        if (variant == ORC_LATENCY) {
            if (dtype == ORC_I32) rc = latency_slice_i32(&tp, sd, sx, w, c0, c1, (const uint32_t *)in, (uint32_t *)out, max_steps, &ctr);
            else if (dtype == ORC_F32) rc = latency_slice_f32(&tp, sd, sx, w, c0, c1, (const float *)in, (float *)out, max_steps, &ctr);
            else rc = latency_slice_f64(&tp, sd, sx, w, c0, c1, (const double *)in, (double *)out, max_steps, &ctr);
        } else {
            if (dtype == ORC_I32) rc = bandwidth_slice_i32(&tp, sd, sx, slo, shi, e0, e1, w, (const uint32_t *)in, (uint32_t *)out, &ctr);
            else if (dtype == ORC_F32) rc = bandwidth_slice_f32(&tp, sd, sx, slo, shi, e0, e1, w, (const float *)in, (float *)out, &ctr);
            else rc = bandwidth_slice_f64(&tp, sd, sx, slo, shi, e0, e1, w, (const double *)in, (double *)out, &ctr);
        }
        if (rc) return rc;
    }
    return ORC_OK;
}

/* ------------------------------------------------------------------ bytes sent per node */

/*
 * Total bytes every node sends over the whole AllReduce (both phases of the bandwidth form), by
 * walking every message of every step (Sec. 2.3: bandwidth optimality is relative to 2m).
 * sent: [n] int64.
 */
int orc_bytes_sent(const int32_t *dims, int ndims, int variant, int algo, int64_t E, int64_t elem_size, int64_t *sent) {
    orc_topo tp; int rc = topo_init(&tp, dims, ndims, algo);
    if (rc) return rc;
    if (E < 0 || elem_size < 1 || !sent) return ORC_BAD_ARG;
    if (variant != ORC_LATENCY && variant != ORC_BANDWIDTH) return ORC_BAD_ARG;
    int n = tp.n, D = tp.nsl, S = tp.S, T = (variant == ORC_BANDWIDTH) ? 2 * S : S;
    if (tp.algo == ORC_BUCKET) {
        /* Reduce-Scatter step t: node r sends block (r - t - 1) mod n on; AllGather step t: block (r - t) mod n
         * (block j ends at node j); a mirrored collective runs the ring the other way round (Sec. 2.4). */
        if (variant != ORC_BANDWIDTH) return ORC_UNDEFINED;
        uint8_t *msg = (uint8_t *)malloc((size_t)n);
        if (!msg) return ORC_NOMEM;
        memset(sent, 0, sizeof(int64_t) * (size_t)n);
        for (int c = 0; c < D; ++c) {
            int64_t slo, shi; int sg = c >= tp.ndims ? -1 : 1;
            slice_bounds(E, D, c, &slo, &shi);
            for (int row = 0; row < T; ++row) {
                int d, s, earlier;
                bucket_where(&tp, c, row, &d, &s, &earlier);
                for (int r = 0; r < n; ++r) {
                    bucket_message(&tp, r, row, d, s, earlier, sg, msg);
                    for (int j = 0; j < n; ++j)
                        if (msg[j]) sent[r] += (block_bound(slo, shi, n, j + 1) - block_bound(slo, shi, n, j)) * elem_size;
                }
            }
        }
        free(msg);
        return ORC_OK;
    }
    uint8_t *set = (uint8_t *)malloc((size_t)n);
    uint8_t *have = (uint8_t *)malloc((size_t)n * n), *snap = (uint8_t *)malloc((size_t)n * n);
    int64_t *blen = (int64_t *)malloc(sizeof(int64_t) * (size_t)n);
    if (!set || !have || !snap || !blen) { free(set); free(have); free(snap); free(blen); return ORC_NOMEM; }
    memset(sent, 0, sizeof(int64_t) * (size_t)n);
    for (int c = 0; c < D; ++c) {
        int sd[64], sx[64];
        int64_t slo, shi;
        step_list(&tp, c, sd, sx);
        slice_bounds(E, D, c, &slo, &shi);
        for (int j = 0; j < n; ++j) blen[j] = block_bound(slo, shi, n, j + 1) - block_bound(slo, shi, n, j);
        memset(have, 0, (size_t)n * n);
        for (int r = 0; r < n; ++r) have[(size_t)r * n + r] = 1;
        for (int row = 0; row < T; ++row) {
            int t = (row < S) ? row : (2 * S - 1 - row);
            if (row >= S) memcpy(snap, have, (size_t)n * n);
            for (int r = 0; r < n; ++r) {
                int peer[2], dir[2], hops[2];
                int np = send_peers(&tp, r, sd[t], sx[t], peer, dir, hops);
                for (int i = 0; i < np; ++i) {
                    int64_t mbytes = 0;
                    if (variant == ORC_LATENCY) {
                        mbytes = (shi - slo) * elem_size;
                    } else if (row < S) {
                        send_set(&tp, sd, sx, peer[i], t, set);
                        for (int j = 0; j < n; ++j) if (set[j]) mbytes += blen[j] * elem_size;
                    } else {
                        for (int j = 0; j < n; ++j) if (snap[(size_t)r * n + j]) {
                            mbytes += blen[j] * elem_size;
                            have[(size_t)peer[i] * n + j] = 1;
                        }
                    }
                    sent[r] += mbytes;
                }
            }
        }
    }
    free(set); free(have); free(snap); free(blen);
    return ORC_OK;
}

/* ------------------------------------------------------------------ link loads */

/*
 * Per-step, per-directed-link load (Sec. 2.1: c_k; Fig. 1; App. E routing).
 * Rows: T = S (latency form) or 2S (bandwidth form: Reduce-Scatter steps 0..S-1,
 * then the AllGather steps, which mirror S-1..0).
 * msgs/bytes are [T][n][D][2]: link leaving `node` along dimension `dim`,
 * direction index 0 = towards +, 1 = towards -.  Every message walks hop by hop
 * from its source in its direction of travel.  A message's bytes are the real
 * (possibly uneven) lengths of the blocks it carries times elem_size.
 * All four outputs are optional.
 */
int orc_link_loads(const int32_t *dims, int ndims, int variant, int algo, int64_t E, int64_t elem_size,
                   int32_t *msgs, int64_t *bytes, int32_t *max_msgs, int64_t *max_bytes) {
    orc_topo tp; int rc = topo_init(&tp, dims, ndims, algo);
    if (rc) return rc;
    if (E < 0 || elem_size < 1) return ORC_BAD_ARG;
    if (variant != ORC_LATENCY && variant != ORC_BANDWIDTH) return ORC_BAD_ARG;
    int n = tp.n, D = tp.ndims, NSL = tp.nsl, S = tp.S, T = (variant == ORC_BANDWIDTH) ? 2 * S : S;
    if (tp.algo == ORC_BUCKET && variant != ORC_BANDWIDTH) return ORC_UNDEFINED;
    size_t links = (size_t)n * D * 2;
    int32_t *lm = (int32_t *)calloc((size_t)T * links, sizeof(int32_t));
    int64_t *lb = (int64_t *)calloc((size_t)T * links, sizeof(int64_t));
    uint8_t *set = (uint8_t *)malloc((size_t)n);
    uint8_t *have = (uint8_t *)malloc((size_t)n * n), *snap = (uint8_t *)malloc((size_t)n * n);
    int64_t *blen = (int64_t *)malloc(sizeof(int64_t) * (size_t)n);
    if (!lm || !lb || !set || !have || !snap || !blen) { rc = ORC_NOMEM; goto done; }

    if (tp.algo == ORC_BUCKET) {        /* one block per node and step, one hop, always the same way round */
        for (int c = 0; c < NSL; ++c) {
            int64_t slo, shi; int sg = c >= tp.ndims ? -1 : 1;
            slice_bounds(E, NSL, c, &slo, &shi);
            for (int row = 0; row < T; ++row) {
                int d, s, earlier;
                bucket_where(&tp, c, row, &d, &s, &earlier);
                for (int r = 0; r < n; ++r) {       /* one message over the one link from r to its neighbour along d */
                    size_t li = (((size_t)row * n + r) * D + d) * 2 + (sg > 0 ? 0 : 1);
                    bucket_message(&tp, r, row, d, s, earlier, sg, set);
                    lm[li] += 1;
                    for (int j = 0; j < n; ++j)
                        if (set[j]) lb[li] += (block_bound(slo, shi, n, j + 1) - block_bound(slo, shi, n, j)) * elem_size;
                }
            }
        }
    } else
    for (int c = 0; c < NSL; ++c) {
        int sd[64], sx[64];
        int64_t slo, shi;
        step_list(&tp, c, sd, sx);
        slice_bounds(E, NSL, c, &slo, &shi);
        for (int j = 0; j < n; ++j) blen[j] = block_bound(slo, shi, n, j + 1) - block_bound(slo, shi, n, j);
        memset(have, 0, (size_t)n * n);
        for (int r = 0; r < n; ++r) have[(size_t)r * n + r] = 1;
        for (int row = 0; row < T; ++row) {
            int t = (row < S) ? row : (2 * S - 1 - row);      /* AllGather mirrors */
            int d = sd[t], dist = sx[t];
            if (row >= S) memcpy(snap, have, (size_t)n * n);
            for (int r = 0; r < n; ++r) {
                int peer[2], dir[2], hops[2];
                int np = send_peers(&tp, r, d, dist, peer, dir, hops);
                for (int i = 0; i < np; ++i) {
                    int64_t mbytes = 0;
                    if (variant == ORC_LATENCY) {
                        mbytes = (shi - slo) * elem_size;
                    } else if (row < S) {
                        send_set(&tp, sd, sx, peer[i], t, set);
                        for (int j = 0; j < n; ++j) if (set[j]) mbytes += blen[j] * elem_size;
                    } else {
                        for (int j = 0; j < n; ++j) if (snap[(size_t)r * n + j]) {
                            mbytes += blen[j] * elem_size;
                            have[(size_t)peer[i] * n + j] = 1;
                        }
                    }
                    int cur = r;
                    for (int h = 0; h < hops[i]; ++h) {
                        size_t li = (((size_t)row * n + cur) * D + d) * 2 + (dir[i] > 0 ? 0 : 1);
                        lm[li] += 1; lb[li] += mbytes;
                        cur = shift_rank(&tp, cur, d, dir[i]);
                    }
                    if (cur != peer[i]) { rc = ORC_INTERNAL; goto done; }
                }
            }
        }
    }
    for (int row = 0; row < T; ++row) {
        int32_t mm = 0; int64_t mb = 0;
        for (size_t l = 0; l < links; ++l) {
            if (lm[(size_t)row * links + l] > mm) mm = lm[(size_t)row * links + l];
            if (lb[(size_t)row * links + l] > mb) mb = lb[(size_t)row * links + l];
        }
        if (max_msgs) max_msgs[row] = mm;
        if (max_bytes) max_bytes[row] = mb;
    }
    if (msgs) memcpy(msgs, lm, sizeof(int32_t) * (size_t)T * links);
    if (bytes) memcpy(bytes, lb, sizeof(int64_t) * (size_t)T * links);
done:
    free(lm); free(lb); free(set); free(have); free(snap); free(blen);
    return rc;
}

/* ------------------------------------------------------------------ rings of any size (Sec. 4.4) */

/*
 * Bandwidth-optimal Trivance on a ring whose size n is NOT a power of three.
 *
 * What the paper fixes (Sec. 4.4): the first s' = floor(log3 n) steps are the regular ones
 * (distances 3^0 .. 3^(s'-1)); one final step follows in which every node talks to both
 * nodes at distance d = ceil((n - 3^s') / 2); ceil(log3 n) steps in all; blocks travel as in
 * Algorithm 1 with every block forwarded at most once per phase, so a node sends at most m
 * bytes per phase; the final step's congestion is d on every link; for n = 7 a node sends two
 * blocks per direction in the first step and one block, at distance two, in the final one.
 *
 * Reading where the paper is silent (PARITY UNPINNED by the paper):
 * which tree a block follows.  The AllGather of block b runs the steps in reverse order (the
 * distance-d step first).  The nodes that hold the block are kept in the order they got it;
 * in a step every holder, in that order, offers the block first to its left peer (h - dist)
 * and then to its right peer (h + dist); a node that holds the block already -- one that got
 * it earlier in the same step included -- is skipped.  The Reduce-Scatter runs the same tree
 * backwards: in step t every node that received block b in AllGather step t sends its
 * partial of block b to the node it got the block from, and a receiver adds
 * (from_left + own) + from_right, leaving out a side nothing came from.
 * For n a power of three this rule gives the regular schedule (no node is ever skipped).
 */
static int gen_steps(int n, int *dist) {
    int p = 1, s = 0;
    while ((long long)p * 3 <= n) { p *= 3; dist[s++] = p / 3; }
    if (p != n) dist[s++] = (n - p + 1) / 2;
    return s;
}

/* par[b*n+v] = node v got block b from (-1 for v = b); stp[b*n+v] = the step it got it in */
static int gen_build(int n, int S, const int *dist, int32_t *par, int32_t *stp) {
    int *list = (int *)malloc(sizeof(int) * (size_t)n);
    uint8_t *have = (uint8_t *)malloc((size_t)n);
    int rc = ORC_OK;
    if (!list || !have) { free(list); free(have); return ORC_NOMEM; }
    for (int b = 0; b < n && rc == ORC_OK; ++b) {
        int len = 1;
        memset(have, 0, (size_t)n);
        list[0] = b; have[b] = 1; par[(size_t)b * n + b] = -1; stp[(size_t)b * n + b] = -1;
        for (int t = S - 1; t >= 0; --t) {
            int len0 = len;
            for (int i = 0; i < len0; ++i) {
                int h = list[i];
                for (int side = 0; side < 2; ++side) {
                    int v = ((h + (side ? dist[t] : -dist[t])) % n + n) % n;
                    if (have[v]) continue;
                    have[v] = 1; par[(size_t)b * n + v] = h; stp[(size_t)b * n + v] = t; list[len++] = v;
                }
            }
        }
        if (len != n) rc = ORC_INTERNAL;
    }
    free(list); free(have);
    return rc;
}

int orc_gen_num_steps(int n, int *S_out, int32_t *dist_out) {
    if (n < 2 || n > 4096) return ORC_BAD_ARG;
    int dist[32];
    int S = gen_steps(n, dist);
    if (S_out) *S_out = S;
    if (dist_out) for (int t = 0; t < S; ++t) dist_out[t] = dist[t];
    return ORC_OK;
}

int orc_gen_tree(int n, int32_t *par, int32_t *stp) {
    if (n < 2 || n > 4096 || !par || !stp) return ORC_BAD_ARG;
    int dist[32];
    int S = gen_steps(n, dist);
    return gen_build(n, S, dist, par, stp);
}

#define DEFINE_GEN(T, SUFFIX, ADD)                                                                         \
static int gen_allreduce_##SUFFIX(int n, int S, const int *dist, const int32_t *par, const int32_t *stp,   \
                                  int64_t E, int64_t e0, int64_t e1, const T *in, T *out,                  \
                                  orc_counters *ctr) {                                                     \
    int64_t w = e1 - e0;                                                                                   \
    if (w <= 0) return ORC_OK;                                                                             \
    int64_t *bs = (int64_t *)malloc(sizeof(int64_t) * (size_t)(n + 1));                                    \
    T *partial = (T *)malloc(sizeof(T) * (size_t)n * (size_t)w);                                           \
    T *msg = (T *)malloc(sizeof(T) * (size_t)n * (size_t)w);     /* what every node puts on the wire */     \
    if (!bs || !partial || !msg) { free(bs); free(partial); free(msg); return ORC_NOMEM; }                 \
    for (int j = 0; j <= n; ++j) bs[j] = clampi(block_bound(0, E, n, j), e0, e1) - e0;                     \
    memcpy(partial, in, sizeof(T) * (size_t)n * (size_t)w);                                                \
    /* ---- Reduce-Scatter: the tree of every block, leaves first */                                      \
    for (int t = 0; t < S; ++t) {                                                                          \
        memcpy(msg, partial, sizeof(T) * (size_t)n * (size_t)w);                                           \
        for (int b = 0; b < n; ++b) {                                                                      \
            int64_t bl = bs[b + 1] - bs[b];                                                                \
            for (int p = 0; p < n; ++p) {                                                                  \
                int ql = ((p - dist[t]) % n + n) % n, qr = (p + dist[t]) % n;                              \
                int hl = (stp[(size_t)b * n + ql] == t && par[(size_t)b * n + ql] == p);                   \
                int hr = (qr != ql && stp[(size_t)b * n + qr] == t && par[(size_t)b * n + qr] == p);       \
                T *own = partial + (size_t)p * w + bs[b];                                                  \
                const T *ml = msg + (size_t)ql * w + bs[b], *mr = msg + (size_t)qr * w + bs[b];            \
                if (!hl && !hr) continue;                                                                  \
                for (int64_t e = 0; e < bl; ++e) {                                                         \
                    T acc = own[e];                                                                        \
                    if (hl) acc = ADD(ml[e], acc);                                                         \
                    if (hr) acc = ADD(acc, mr[e]);                                                         \
                    own[e] = acc;                                                                          \
                }                                                                                          \
                if (ctr && ctr->sent_rs) {                                                                 \
                    if (hl) ctr->sent_rs[ql] += (int64_t)sizeof(T) * bl;                                   \
                    if (hr) ctr->sent_rs[qr] += (int64_t)sizeof(T) * bl;                                   \
                }                                                                                          \
                if (ctr && ctr->reduced) ctr->reduced[p] += (int64_t)sizeof(T) * bl * (1 + hl + hr);       \
            }                                                                                              \
        }                                                                                                  \
    }                                                                                                      \
    /* ---- AllGather: the same trees, root first */                                                      \
    for (int t = S - 1; t >= 0; --t) {                                                                     \
        memcpy(msg, partial, sizeof(T) * (size_t)n * (size_t)w);                                           \
        for (int b = 0; b < n; ++b)                                                                        \
            for (int v = 0; v < n; ++v) if (stp[(size_t)b * n + v] == t) {                                 \
                int q = par[(size_t)b * n + v]; int64_t bl = bs[b + 1] - bs[b];                            \
                memcpy(partial + (size_t)v * w + bs[b], msg + (size_t)q * w + bs[b], sizeof(T) * (size_t)bl);\
                if (ctr && ctr->sent_ag) ctr->sent_ag[q] += (int64_t)sizeof(T) * bl;                       \
            }                                                                                              \
    }                                                                                                      \
    memcpy(out, partial, sizeof(T) * (size_t)n * (size_t)w);                                               \
    free(bs); free(partial); free(msg);                                                                    \
    return ORC_OK;                                                                                         \
}
DEFINE_GEN(uint32_t, i32, ADD_WRAP)
DEFINE_GEN(float, f32, ADD_FP)
DEFINE_GEN(double, f64, ADD_FP)

/* AllReduce (bandwidth-optimal form) on a ring of any size n >= 2; arguments as orc_allreduce. */
int orc_gen_allreduce(int n, int dtype, int64_t E, int64_t e0, int64_t e1, const void *in, void *out,
                      int64_t *sent_rs, int64_t *sent_ag, int64_t *reduced) {
    if (n < 2 || n > 4096 || E < 0 || e0 < 0 || e1 < e0 || e1 > E || !in || !out) return ORC_BAD_ARG;
    if (dtype != ORC_I32 && dtype != ORC_F32 && dtype != ORC_F64) return ORC_BAD_ARG;
    int dist[32];
    int S = gen_steps(n, dist), rc;
    int32_t *par = (int32_t *)malloc(sizeof(int32_t) * (size_t)n * n), *stp = (int32_t *)malloc(sizeof(int32_t) * (size_t)n * n);
    orc_counters ctr = { sent_rs, sent_ag, reduced };
    if (!par || !stp) { free(par); free(stp); return ORC_NOMEM; }
    rc = gen_build(n, S, dist, par, stp);
    if (rc == ORC_OK) {
        if (dtype == ORC_I32) rc = gen_allreduce_i32(n, S, dist, par, stp, E, e0, e1, (const uint32_t *)in, (uint32_t *)out, &ctr);
        else if (dtype == ORC_F32) rc = gen_allreduce_f32(n, S, dist, par, stp, E, e0, e1, (const float *)in, (float *)out, &ctr);
        else rc = gen_allreduce_f64(n, S, dist, par, stp, E, e0, e1, (const double *)in, (double *)out, &ctr);
    }
    free(par); free(stp);
    return rc;
}

/*
 * Link loads of the same schedule (rows: S Reduce-Scatter steps, then the S AllGather steps in
 * reverse order; arrays [2S][n][1][2] as in orc_link_loads).  All blocks a node sends to one
 * peer in one step form ONE message; it walks dist links in its direction of travel.
 * sent (optional, [n]): bytes every node sends over both phases.
 */
int orc_gen_link_loads(int n, int64_t E, int64_t elem_size, int32_t *msgs, int64_t *bytes,
                       int32_t *max_msgs, int64_t *max_bytes, int64_t *sent) {
    if (n < 2 || n > 4096 || E < 0 || elem_size < 1) return ORC_BAD_ARG;
    int dist[32];
    int S = gen_steps(n, dist), T = 2 * S, rc;
    size_t links = (size_t)n * 2;
    int32_t *par = (int32_t *)malloc(sizeof(int32_t) * (size_t)n * n), *stp = (int32_t *)malloc(sizeof(int32_t) * (size_t)n * n);
    int32_t *lm = (int32_t *)calloc((size_t)T * links, sizeof(int32_t));
    int64_t *lb = (int64_t *)calloc((size_t)T * links, sizeof(int64_t));
    int64_t *mb = (int64_t *)malloc(sizeof(int64_t) * links);       /* [source][side]: bytes of its message */
    int32_t *mc = (int32_t *)malloc(sizeof(int32_t) * links);       /* blocks in it */
    if (!par || !stp || !lm || !lb || !mb || !mc) { rc = ORC_NOMEM; goto done; }
    rc = gen_build(n, S, dist, par, stp);
    if (rc) goto done;
    if (sent) memset(sent, 0, sizeof(int64_t) * (size_t)n);
    for (int row = 0; row < T; ++row) {
        int t = row < S ? row : T - 1 - row;
        memset(mb, 0, sizeof(int64_t) * links); memset(mc, 0, sizeof(int32_t) * links);
        for (int b = 0; b < n; ++b)
            for (int v = 0; v < n; ++v) if (stp[(size_t)b * n + v] == t) {
                int q = par[(size_t)b * n + v];
                /* v is its parent's left peer (tried first, so also when both peers coincide) or right peer */
                int left_child = (v == ((q - dist[t]) % n + n) % n);
                int src = row < S ? v : q;
                int side = row < S ? left_child : !left_child;      /* 0: travels towards -, 1: towards + */
                mb[(size_t)src * 2 + side] += (block_bound(0, E, n, b + 1) - block_bound(0, E, n, b)) * elem_size;
                mc[(size_t)src * 2 + side] += 1;
            }
        for (int src = 0; src < n; ++src)
            for (int side = 0; side < 2; ++side) if (mc[(size_t)src * 2 + side]) {
                int cur = src;
                if (sent) sent[src] += mb[(size_t)src * 2 + side];
                for (int h = 0; h < dist[t]; ++h) {
                    size_t li = ((size_t)row * n + cur) * 2 + (side ? 0 : 1);
                    lm[li] += 1; lb[li] += mb[(size_t)src * 2 + side];
                    cur = ((cur + (side ? 1 : -1)) % n + n) % n;
                }
            }
    }
    for (int row = 0; row < T; ++row) {
        int32_t mm = 0; int64_t mx = 0;
        for (size_t l = 0; l < links; ++l) {
            if (lm[(size_t)row * links + l] > mm) mm = lm[(size_t)row * links + l];
            if (lb[(size_t)row * links + l] > mx) mx = lb[(size_t)row * links + l];
        }
        if (max_msgs) max_msgs[row] = mm;
        if (max_bytes) max_bytes[row] = mx;
    }
    if (msgs) memcpy(msgs, lm, sizeof(int32_t) * (size_t)T * links);
    if (bytes) memcpy(bytes, lb, sizeof(int64_t) * (size_t)T * links);
done:
    free(par); free(stp); free(lm); free(lb); free(mb); free(mc);
    return rc;
}

/* ------------------------------------------------------------------ tori with sides of any size (Sec. 4.4 + Sec. 5) */

/*
 * Bandwidth-optimal Trivance on a D-dimensional torus whose sides a_d >= 2 need not be powers of three.
 *
 * What the paper fixes: Sec. 5 runs one collective per dimension on 1/D of the vector, each collective on a
 * different dimension in every step; Sec. 4.4 gives a ring of any size its step list (the regular distances,
 * then one step at distance ceil((a - 3^floor(log3 a)) / 2)) and says that every block is forwarded at most
 * once per phase.  The paper evaluates such tori (32 x 32, 8 x 64, 16 x 16 x 16) without spelling the
 * combination out.
 *
 * Reading (PARITY UNPINNED by the paper): the two rules are composed literally.
 *   - Step list of collective c: the dimensions in round-robin order starting at c, a dimension that has used
 *     up its ceil(log3 a_d) steps being skipped; the k-th visit of dimension d uses the k-th distance of the
 *     ring of a_d nodes.  S = sum_d ceil(log3 a_d) steps per phase.
 *   - Block b is owned by linear rank b.  Its AllGather runs the steps in reverse; the nodes holding it are
 *     kept in the order they got it; in a step along dimension d every holder, in that order, offers it to
 *     the node `dist` before it along d, then to the node `dist` after it; a node that holds it already is
 *     skipped.  The Reduce-Scatter runs the same tree backwards with (from_left + own) + from_right.
 * For sides that are powers of three nothing is ever skipped and this is the regular schedule of Sec. 5.
 */
typedef struct {
    int ndims, n, S;
    int dims[ORC_MAX_DIMS], stride[ORC_MAX_DIMS];
    int nd[ORC_MAX_DIMS];               /* steps of dimension d */
    int ddist[ORC_MAX_DIMS][32];        /* its distances */
} gent_topo;

static int gent_init(gent_topo *g, const int32_t *dims, int ndims) {
    if (!dims || ndims < 1 || ndims > ORC_MAX_DIMS) return ORC_BAD_ARG;
    long long n = 1;
    g->ndims = ndims; g->S = 0;
    for (int d = 0; d < ndims; ++d) {
        if (dims[d] < 2 || dims[d] > 4096) return ORC_BAD_ARG;
        g->dims[d] = dims[d]; g->stride[d] = (int)n;
        g->nd[d] = gen_steps(dims[d], g->ddist[d]);
        g->S += g->nd[d];
        n *= dims[d];
        if (n > 4096) return ORC_BAD_ARG;
    }
    g->n = (int)n;
    return ORC_OK;
}

static void gent_step_list(const gent_topo *g, int c, int *sdim, int *sdist) {
    int visits[ORC_MAX_DIMS] = {0};
    int cur = c % g->ndims;
    for (int t = 0; t < g->S; ++t) {
        int d = cur;
        while (visits[d] >= g->nd[d]) d = (d + 1) % g->ndims;
        sdim[t] = d; sdist[t] = g->ddist[d][visits[d]];
        visits[d]++;
        cur = (d + 1) % g->ndims;
    }
}

static int gent_shift(const gent_topo *g, int r, int d, int delta) {
    int a = g->dims[d], st = g->stride[d];
    int x = (r / st) % a, y = ((x + delta) % a + a) % a;
    return r + (y - x) * st;
}

/* par[b*n+v] = the node v gets block b from (-1 for v = b); stp[b*n+v] = the step (of collective c) in which */
static int gent_build(const gent_topo *g, const int *sdim, const int *sdist, int32_t *par, int32_t *stp) {
    int n = g->n, rc = ORC_OK;
    int *list = (int *)malloc(sizeof(int) * (size_t)n);
    uint8_t *have = (uint8_t *)malloc((size_t)n);
    if (!list || !have) { free(list); free(have); return ORC_NOMEM; }
    for (int b = 0; b < n && rc == ORC_OK; ++b) {
        int len = 1;
        memset(have, 0, (size_t)n);
        list[0] = b; have[b] = 1; par[(size_t)b * n + b] = -1; stp[(size_t)b * n + b] = -1;
        for (int t = g->S - 1; t >= 0; --t) {
            int len0 = len;
            for (int i = 0; i < len0; ++i) {
                int h = list[i];
                for (int side = 0; side < 2; ++side) {
                    int v = gent_shift(g, h, sdim[t], side ? sdist[t] : -sdist[t]);
                    if (have[v]) continue;
                    have[v] = 1; par[(size_t)b * n + v] = h; stp[(size_t)b * n + v] = t; list[len++] = v;
                }
            }
        }
        if (len != n) rc = ORC_INTERNAL;
    }
    free(list); free(have);
    return rc;
}

int orc_gent_num_steps(const int32_t *dims, int ndims, int *n_out, int *S_out) {
    gent_topo g; int rc = gent_init(&g, dims, ndims);
    if (rc) return rc;
    if (n_out) *n_out = g.n;
    if (S_out) *S_out = g.S;
    return ORC_OK;
}

int orc_gent_step_list(const int32_t *dims, int ndims, int c, int32_t *dim_out, int32_t *dist_out) {
    gent_topo g; int rc = gent_init(&g, dims, ndims);
    if (rc) return rc;
    if (c < 0 || c >= ndims || !dim_out || !dist_out) return ORC_BAD_ARG;
    int sd[256], sx[256];
    gent_step_list(&g, c, sd, sx);
    for (int t = 0; t < g.S; ++t) { dim_out[t] = sd[t]; dist_out[t] = sx[t]; }
    return ORC_OK;
}

int orc_gent_tree(const int32_t *dims, int ndims, int c, int32_t *par, int32_t *stp) {
    gent_topo g; int rc = gent_init(&g, dims, ndims);
    if (rc) return rc;
    if (c < 0 || c >= ndims || !par || !stp) return ORC_BAD_ARG;
    int sd[256], sx[256];
    gent_step_list(&g, c, sd, sx);
    return gent_build(&g, sd, sx, par, stp);
}

/* One collective (slice [slo, shi) of the global vector) on the window [e0, e1); arrays are [n][w], w = e1 - e0. */
#define DEFINE_GENT(T, SUFFIX, ADD)                                                                         \
static int gent_slice_##SUFFIX(const gent_topo *g, const int *sdim, const int *sdist, const int32_t *par,   \
                               const int32_t *stp, int64_t slo, int64_t shi, int64_t e0, int64_t e1,        \
                               T *partial, T *msg, orc_counters *ctr) {                                     \
    int n = g->n, S = g->S;                                                                                 \
    int64_t w = e1 - e0;                                                                                    \
    int64_t *bs = (int64_t *)malloc(sizeof(int64_t) * (size_t)(n + 1));                                     \
    if (!bs) return ORC_NOMEM;                                                                              \
    for (int j = 0; j <= n; ++j) bs[j] = clampi(block_bound(slo, shi, n, j), e0, e1) - e0;                  \
    if (bs[n] <= bs[0]) { free(bs); return ORC_OK; }                                                        \
    /* ---- Reduce-Scatter: every node first puts its current partials on the wire, then all receive */   \
    for (int t = 0; t < S; ++t) {                                                                           \
        for (int p = 0; p < n; ++p)                                                                         \
            memcpy(msg + (size_t)p * w + bs[0], partial + (size_t)p * w + bs[0], sizeof(T) * (size_t)(bs[n] - bs[0])); \
        for (int b = 0; b < n; ++b) {                                                                       \
            int64_t bl = bs[b + 1] - bs[b];                                                                 \
            for (int p = 0; p < n; ++p) {                                                                   \
                int ql = gent_shift(g, p, sdim[t], -sdist[t]), qr = gent_shift(g, p, sdim[t], sdist[t]);    \
                int hl = (stp[(size_t)b * n + ql] == t && par[(size_t)b * n + ql] == p);                    \
                int hr = (qr != ql && stp[(size_t)b * n + qr] == t && par[(size_t)b * n + qr] == p);        \
                if (!hl && !hr) continue;                                                                   \
                T *own = partial + (size_t)p * w + bs[b];                                                   \
                const T *ml = msg + (size_t)ql * w + bs[b], *mr = msg + (size_t)qr * w + bs[b];             \
                for (int64_t e = 0; e < bl; ++e) {                                                          \
                    T acc = own[e];                                                                         \
                    if (hl) acc = ADD(ml[e], acc);                                                          \
                    if (hr) acc = ADD(acc, mr[e]);                                                          \
                    own[e] = acc;                                                                           \
                }                                                                                           \
                if (ctr && ctr->sent_rs) {                                                                  \
                    if (hl) ctr->sent_rs[ql] += (int64_t)sizeof(T) * bl;                                    \
                    if (hr) ctr->sent_rs[qr] += (int64_t)sizeof(T) * bl;                                    \
                }                                                                                           \
                if (ctr && ctr->reduced) ctr->reduced[p] += (int64_t)sizeof(T) * bl * (1 + hl + hr);        \
            }                                                                                               \
        }                                                                                                   \
    }                                                                                                       \
    /* ---- AllGather: the same trees, root first */                                                       \
    for (int t = S - 1; t >= 0; --t) {                                                                      \
        for (int p = 0; p < n; ++p)                                                                         \
            memcpy(msg + (size_t)p * w + bs[0], partial + (size_t)p * w + bs[0], sizeof(T) * (size_t)(bs[n] - bs[0])); \
        for (int b = 0; b < n; ++b)                                                                         \
            for (int v = 0; v < n; ++v) if (stp[(size_t)b * n + v] == t) {                                  \
                int q = par[(size_t)b * n + v]; int64_t bl = bs[b + 1] - bs[b];                             \
                memcpy(partial + (size_t)v * w + bs[b], msg + (size_t)q * w + bs[b], sizeof(T) * (size_t)bl);\
                if (ctr && ctr->sent_ag) ctr->sent_ag[q] += (int64_t)sizeof(T) * bl;                        \
            }                                                                                               \
    }                                                                                                       \
    free(bs);                                                                                               \
    return ORC_OK;                                                                                          \
}
DEFINE_GENT(uint32_t, i32, ADD_WRAP)
DEFINE_GENT(float, f32, ADD_FP)
DEFINE_GENT(double, f64, ADD_FP)

/* AllReduce (bandwidth-optimal form) on a torus with sides of any size >= 2; arguments as orc_allreduce. */
int orc_gent_allreduce(const int32_t *dims, int ndims, int dtype, int64_t E, int64_t e0, int64_t e1, const void *in,
                       void *out, int64_t *sent_rs, int64_t *sent_ag, int64_t *reduced) {
    gent_topo g; int rc = gent_init(&g, dims, ndims);
    if (rc) return rc;
    if (E < 0 || e0 < 0 || e1 < e0 || e1 > E || !in || !out) return ORC_BAD_ARG;
    if (dtype != ORC_I32 && dtype != ORC_F32 && dtype != ORC_F64) return ORC_BAD_ARG;
    int n = g.n;
    int64_t w = e1 - e0;
    size_t es = dtype == ORC_F64 ? 8 : 4;
    if (w == 0) return ORC_OK;
    int32_t *par = (int32_t *)malloc(sizeof(int32_t) * (size_t)n * n), *stp = (int32_t *)malloc(sizeof(int32_t) * (size_t)n * n);
    void *msg = malloc(es * (size_t)n * (size_t)w);
    orc_counters ctr = { sent_rs, sent_ag, reduced };
    if (!par || !stp || !msg) { free(par); free(stp); free(msg); return ORC_NOMEM; }
    memcpy(out, in, es * (size_t)n * (size_t)w);        /* the partials live in `out` */
    for (int c = 0; c < ndims && rc == ORC_OK; ++c) {
        int sd[256], sx[256];
        int64_t slo, shi;
        slice_bounds(E, ndims, c, &slo, &shi);
        if (clampi(shi, e0, e1) <= clampi(slo, e0, e1)) continue;
        gent_step_list(&g, c, sd, sx);
        rc = gent_build(&g, sd, sx, par, stp);
        if (rc) break;
        if (dtype == ORC_I32) rc = gent_slice_i32(&g, sd, sx, par, stp, slo, shi, e0, e1, (uint32_t *)out, (uint32_t *)msg, &ctr);
        else if (dtype == ORC_F32) rc = gent_slice_f32(&g, sd, sx, par, stp, slo, shi, e0, e1, (float *)out, (float *)msg, &ctr);
        else rc = gent_slice_f64(&g, sd, sx, par, stp, slo, shi, e0, e1, (double *)out, (double *)msg, &ctr);
    }
    free(par); free(stp); free(msg);
    return rc;
}

/*
 * Link loads of that schedule: rows = S Reduce-Scatter steps, then the AllGather steps in reverse order;
 * arrays [2S][n][D][2] as in orc_link_loads (index 0: the link leaving the node towards +, 1: towards -).
 * All blocks a node sends to one peer in one step of one collective form ONE message; it walks `dist` links
 * along the step's dimension in its direction of travel.  sent (optional, [n]): bytes a node sends in total.
 */
int orc_gent_link_loads(const int32_t *dims, int ndims, int64_t E, int64_t elem_size, int32_t *msgs, int64_t *bytes,
                        int32_t *max_msgs, int64_t *max_bytes, int64_t *sent) {
    gent_topo g; int rc = gent_init(&g, dims, ndims);
    if (rc) return rc;
    if (E < 0 || elem_size < 1) return ORC_BAD_ARG;
    int n = g.n, S = g.S, T = 2 * S, D = ndims;
    size_t links = (size_t)n * D * 2;
    int32_t *par = (int32_t *)malloc(sizeof(int32_t) * (size_t)n * n), *stp = (int32_t *)malloc(sizeof(int32_t) * (size_t)n * n);
    int32_t *lm = (int32_t *)calloc((size_t)T * links, sizeof(int32_t));
    int64_t *lb = (int64_t *)calloc((size_t)T * links, sizeof(int64_t));
    int64_t *mb = (int64_t *)malloc(sizeof(int64_t) * (size_t)n * 2);
    int32_t *mc = (int32_t *)malloc(sizeof(int32_t) * (size_t)n * 2);
    if (!par || !stp || !lm || !lb || !mb || !mc) { rc = ORC_NOMEM; goto done; }
    if (sent) memset(sent, 0, sizeof(int64_t) * (size_t)n);
    for (int c = 0; c < D; ++c) {
        int sd[256], sx[256];
        int64_t slo, shi;
        slice_bounds(E, D, c, &slo, &shi);
        gent_step_list(&g, c, sd, sx);
        rc = gent_build(&g, sd, sx, par, stp);
        if (rc) goto done;
        for (int row = 0; row < T; ++row) {
            int t = row < S ? row : T - 1 - row, d = sd[t];
            memset(mb, 0, sizeof(int64_t) * (size_t)n * 2); memset(mc, 0, sizeof(int32_t) * (size_t)n * 2);
            for (int b = 0; b < n; ++b)
                for (int v = 0; v < n; ++v) if (stp[(size_t)b * n + v] == t) {
                    int q = par[(size_t)b * n + v];
                    int left_child = (v == gent_shift(&g, q, d, -sx[t]));   /* tried first: also when both peers coincide */
                    int src = row < S ? v : q;
                    int side = row < S ? left_child : !left_child;           /* 0: travels towards -, 1: towards + */
                    mb[(size_t)src * 2 + side] += (block_bound(slo, shi, n, b + 1) - block_bound(slo, shi, n, b)) * elem_size;
                    mc[(size_t)src * 2 + side] += 1;
                }
            for (int src = 0; src < n; ++src)
                for (int side = 0; side < 2; ++side) if (mc[(size_t)src * 2 + side]) {
                    int cur = src;
                    if (sent) sent[src] += mb[(size_t)src * 2 + side];
                    for (int h = 0; h < sx[t]; ++h) {
                        size_t li = (((size_t)row * n + cur) * D + d) * 2 + (side ? 0 : 1);
                        lm[li] += 1; lb[li] += mb[(size_t)src * 2 + side];
                        cur = gent_shift(&g, cur, d, side ? 1 : -1);
                    }
                }
        }
    }
    for (int row = 0; row < T; ++row) {
        int32_t mm = 0; int64_t mx = 0;
        for (size_t l = 0; l < links; ++l) {
            if (lm[(size_t)row * links + l] > mm) mm = lm[(size_t)row * links + l];
            if (lb[(size_t)row * links + l] > mx) mx = lb[(size_t)row * links + l];
        }
        if (max_msgs) max_msgs[row] = mm;
        if (max_bytes) max_bytes[row] = mx;
    }
    if (msgs) memcpy(msgs, lm, sizeof(int32_t) * (size_t)T * links);
    if (bytes) memcpy(bytes, lb, sizeof(int64_t) * (size_t)T * links);
done:
    free(par); free(stp); free(lm); free(lb); free(mb); free(mc);
    return rc;
}

/* ------------------------------------------------------------------ comparator schedules as data paths (Sec. 2.4, 3.1) */

/*
 * The comparison algorithms of the paper -- Bruck with joint reductions (Sec. 3.1; peers r + 3^k and r + 2 3^k),
 * Recursive Doubling (peer r XOR 2^k), Swing (peer r +- rho(k)), the ring (Bucket) algorithm, each optionally with
 * its mirrored sub-collective on the other half of the vector (Sec. 2.4) -- executed literally: in every step every
 * rank puts a message for each of its peers on the wire, then every rank reduces what it received.
 *   latency form   : a message is the sender's whole current partial of the collective's slice;
 *   bandwidth form : Reduce-Scatter: the message to peer p carries the blocks p still answers for after the step
 *                    (p's own and all it forwards later: the same sets the link-load tally uses); AllGather: the
 *                    steps in reverse order, a rank sends every finished block it holds to the step's peers.
 *                    Bucket: step t passes block r - t - 1 (Reduce-Scatter) resp. r - t (AllGather) to r + 1; on a torus
 *                    dimension after dimension on the blocks still answered for (bucket_where, bucket_message).
 * Reading (PARITY UNPINNED by the paper, which never states an association order): a rank that receives m0 from the
 * sender whose FIRST peer it is and m1 from the sender whose SECOND peer it is forms (m1 + own) + m0; with one
 * message own + m0.  For Trivance's peers (first = left, second = right) this is (from_left + own) + from_right.
 */
#define DEFINE_ALGO(T, SUFFIX, ADD)                                                                            \
static int algo_slice_##SUFFIX(const orc_topo *tp, int c, int variant, int64_t slo, int64_t shi, int64_t e0,    \
                               int64_t e1, int64_t w, T *data, orc_counters *ctr) {                             \
    int n = tp->n, S = tp->S, rc = ORC_OK;                                                                      \
    int64_t c0 = clampi(slo, e0, e1) - e0, c1 = clampi(shi, e0, e1) - e0, wc = c1 - c0;                         \
    if (wc <= 0) return ORC_OK;                                                                                 \
    int sd[64], sx[64];                                                                                         \
    int sg = c >= tp->ndims ? -1 : 1, bd = 0, bstep = 0, bearlier = 0;   /* Bucket: direction; dimension, step, earlier dimensions of the row */ \
    if (tp->algo != ORC_BUCKET) step_list(tp, c, sd, sx);                                                       \
    int64_t *bs = (int64_t *)malloc(sizeof(int64_t) * (size_t)(n + 1));                                         \
    T *wire = (T *)malloc(sizeof(T) * (size_t)n * (size_t)wc);       /* what every rank puts on the wire */       \
    int *from = (int *)malloc(sizeof(int) * (size_t)n * 2);          /* from[2p+k]: the sender whose k-th peer is p */\
    uint8_t *set = (uint8_t *)malloc((size_t)n);                                                                \
    uint8_t *have = (uint8_t *)calloc((size_t)n, (size_t)n), *snap = (uint8_t *)malloc((size_t)n * (size_t)n);  \
    if (!bs || !wire || !from || !set || !have || !snap) { rc = ORC_NOMEM; goto done; }                         \
    for (int j = 0; j <= n; ++j) bs[j] = clampi(block_bound(slo, shi, n, j), e0, e1) - e0;                      \
    for (int t = 0; t < S; ++t) {                                   /* ---- latency form, or Reduce-Scatter */   \
        for (int r = 0; r < n; ++r) memcpy(wire + (size_t)r * wc, data + (size_t)r * w + c0, sizeof(T) * (size_t)wc); \
        for (int i = 0; i < 2 * n; ++i) from[i] = -1;                                                           \
        for (int r = 0; r < n; ++r) {                                                                           \
            int peer[2] = {-1, -1}, dir[2], hops[2];                                                            \
            int np = tp->algo == ORC_BUCKET ? 1 : send_peers(tp, r, sd[t], sx[t], peer, dir, hops);             \
            if (tp->algo == ORC_BUCKET) { bucket_where(tp, c, t, &bd, &bstep, &bearlier); peer[0] = shift_rank(tp, r, bd, sg); } \
            for (int k = 0; k < np; ++k) {                                                                      \
                if (from[2 * peer[k] + k] >= 0) { rc = ORC_INTERNAL; goto done; }                               \
                from[2 * peer[k] + k] = r;                                                                      \
            }                                                                                                   \
        }                                                                                                       \
        for (int p = 0; p < n; ++p) {                                                                           \
            int r0 = from[2 * p], r1 = from[2 * p + 1];                                                         \
            if (variant == ORC_LATENCY) memset(set, 1, (size_t)n);                                              \
            else if (tp->algo == ORC_BUCKET) bucket_message(tp, r0, t, bd, bstep, bearlier, sg, set);  /* what its upstream neighbour passes on */ \
            else send_set(tp, sd, sx, p, t, set);                                                               \
            for (int j = 0; j < n; ++j) if (set[j]) {                                                           \
                T *own = data + (size_t)p * w + bs[j];                                                          \
                int64_t bl = bs[j + 1] - bs[j];                                                                 \
                const T *m0 = r0 >= 0 ? wire + (size_t)r0 * wc + (bs[j] - c0) : NULL;                           \
                const T *m1 = r1 >= 0 ? wire + (size_t)r1 * wc + (bs[j] - c0) : NULL;                           \
                for (int64_t e = 0; e < bl; ++e) {                                                              \
                    T acc = own[e];                                                                             \
                    if (m1) acc = ADD(m1[e], acc);                                                              \
                    if (m0) acc = ADD(acc, m0[e]);                                                              \
                    own[e] = acc;                                                                               \
                }                                                                                               \
                if (ctr && ctr->sent_rs) {                                                                      \
                    if (r0 >= 0) ctr->sent_rs[r0] += (int64_t)sizeof(T) * bl;                                   \
                    if (r1 >= 0) ctr->sent_rs[r1] += (int64_t)sizeof(T) * bl;                                   \
                }                                                                                               \
                if (ctr && ctr->reduced) ctr->reduced[p] += (int64_t)sizeof(T) * bl * (1 + (r0 >= 0) + (r1 >= 0)); \
            }                                                                                                   \
        }                                                                                                       \
    }                                                                                                           \
    if (variant == ORC_BANDWIDTH) {                                 /* ---- AllGather */                        \
        for (int r = 0; r < n; ++r) have[(size_t)r * n + r] = 1;                                                \
        for (int row = 0; row < S; ++row) {                                                                     \
            int t = S - 1 - row;                                                                                \
            memcpy(snap, have, (size_t)n * (size_t)n);                                                          \
            for (int r = 0; r < n; ++r) memcpy(wire + (size_t)r * wc, data + (size_t)r * w + c0, sizeof(T) * (size_t)wc); \
            for (int r = 0; r < n; ++r) {                                                                       \
                int peer[2] = {-1, -1}, dir[2], hops[2];                                                        \
                int np = tp->algo == ORC_BUCKET ? 1 : send_peers(tp, r, sd[t], sx[t], peer, dir, hops);         \
                if (tp->algo == ORC_BUCKET) {                                                                   \
                    bucket_where(tp, c, S + row, &bd, &bstep, &bearlier);                                       \
                    peer[0] = shift_rank(tp, r, bd, sg);                                                        \
                    bucket_message(tp, r, S + row, bd, bstep, bearlier, sg, set);                               \
                }                                                                                               \
                for (int k = 0; k < np; ++k)                                                                    \
                    for (int j = 0; j < n; ++j) {                                                               \
                        int sends = tp->algo == ORC_BUCKET ? set[j] : snap[(size_t)r * n + j];                  \
                        if (!sends) continue;                                                                   \
                        if (have[(size_t)peer[k] * n + j]) { rc = ORC_INTERNAL; goto done; }     /* never twice */ \
                        memcpy(data + (size_t)peer[k] * w + bs[j], wire + (size_t)r * wc + (bs[j] - c0),        \
                               sizeof(T) * (size_t)(bs[j + 1] - bs[j]));                                        \
                        have[(size_t)peer[k] * n + j] = 1;                                                      \
                        if (ctr && ctr->sent_ag) ctr->sent_ag[r] += (int64_t)sizeof(T) * (bs[j + 1] - bs[j]);   \
                    }                                                                                           \
            }                                                                                                   \
        }                                                                                                       \
        for (size_t i = 0; i < (size_t)n * (size_t)n; ++i) if (!have[i]) { rc = ORC_INTERNAL; goto done; }      \
    }                                                                                                           \
done:                                                                                                           \
    free(bs); free(wire); free(from); free(set); free(have); free(snap);                                        \
    return rc;                                                                                                  \
}
DEFINE_ALGO(uint32_t, i32, ADD_WRAP)
DEFINE_ALGO(float, f32, ADD_FP)
DEFINE_ALGO(double, f64, ADD_FP)

/* AllReduce by a comparator schedule (algo may carry ORC_MIRROR); arguments as orc_allreduce. */
int orc_allreduce_algo(const int32_t *dims, int ndims, int variant, int algo, int dtype, int64_t E, int64_t e0, int64_t e1,
                       const void *in, void *out, int64_t *sent_rs, int64_t *sent_ag, int64_t *reduced) {
    orc_topo tp; int rc = topo_init(&tp, dims, ndims, algo);
    if (rc) return rc;
    if (E < 0 || e0 < 0 || e1 < e0 || e1 > E || !in || !out) return ORC_BAD_ARG;
    if (variant != ORC_LATENCY && variant != ORC_BANDWIDTH) return ORC_BAD_ARG;
    if (dtype != ORC_I32 && dtype != ORC_F32 && dtype != ORC_F64) return ORC_BAD_ARG;
    if (tp.algo == ORC_BUCKET && variant != ORC_BANDWIDTH) return ORC_UNDEFINED;
    if (tp.S > 64 && tp.algo != ORC_BUCKET) return ORC_BAD_ARG;
    orc_counters ctr = { sent_rs, sent_ag, reduced };
    int64_t w = e1 - e0;
    size_t es = dtype == ORC_F64 ? 8 : 4;
    memcpy(out, in, es * (size_t)tp.n * (size_t)w);         /* the partials live in `out` */
    for (int c = 0; c < tp.nsl && rc == ORC_OK; ++c) {
        int64_t slo, shi;
        slice_bounds(E, tp.nsl, c, &slo, &shi);
        if (dtype == ORC_I32) rc = algo_slice_i32(&tp, c, variant, slo, shi, e0, e1, w, (uint32_t *)out, &ctr);
        else if (dtype == ORC_F32) rc = algo_slice_f32(&tp, c, variant, slo, shi, e0, e1, w, (float *)out, &ctr);
        else rc = algo_slice_f64(&tp, c, variant, slo, shi, e0, e1, w, (double *)out, &ctr);
    }
    return rc;
}
