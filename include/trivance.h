/*
 * trivance.h -- C ABI of the B200 Trivance AllReduce engine.
 *
 * The engine executes the Trivance AllReduce schedule (Juerss, Addanki, Schmid:
 * "Trivance: Latency-Optimal AllReduce by Shortcutting Multiport Networks") over n
 * SIMULATED ranks whose buffers all live in one GPU's memory.  Nothing moves between
 * GPUs.  All entry points are plain C: pointers (each documented as HOST or DEVICE)
 * and sizes.  No entry point throws, aborts or synchronises the device unless it says
 * so.  Every function returns a trv_status_t; argument errors are found on the host
 * before anything is launched.
 *
 * Notation (paper): n ranks on a D-dimensional torus with sides a_0..a_{D-1}, every side
 * a power of three; rank r = x_0 + a_0 x_1 + a_0 a_1 x_2 + ...; S = sum_d log3 a_d steps
 * per phase; every rank owns a vector of `count` 4-byte elements.
 */
#ifndef TRIVANCE_H_
#define TRIVANCE_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct trv_plan_s *trv_plan_t;          /* opaque; owned by the library */

typedef enum {
    TRV_OK = 0,
    TRV_ERR_INVALID_ARG = 1,        /* NULL pointer, bad enum, misaligned or aliasing buffers ... */
    TRV_ERR_UNSUPPORTED = 2,        /* a side that is no power of three in the latency form, too many ranks or dimensions, op != sum */
    TRV_ERR_UNDEFINED_SCHEDULE = 3, /* the schedule does not exist for this n (Recursive Doubling, n != 2^q) */
    TRV_ERR_ALLOC = 4,
    TRV_ERR_CUDA = 5,               /* a CUDA runtime call failed; cudaGetLastError has the reason */
    TRV_ERR_SCRATCH = 6,            /* caller-provided scratch/workspace too small or misaligned */
    TRV_ERR_TOO_LARGE = 7,          /* the call needs more than the fixed capacity of a no-allocation entry point */
    TRV_ERR_TIMEOUT = 8             /* a bounded device-side wait of the PIPELINED kernel ran out (trv_pipeline_status) */
} trv_status_t;

typedef enum { TRV_LATENCY_OPTIMAL = 0, TRV_BANDWIDTH_OPTIMAL = 1 } trv_variant_t;
typedef enum { TRV_ALGO_TRIVANCE = 0, TRV_ALGO_BRUCK = 1, TRV_ALGO_RECDOUB = 2, TRV_ALGO_SWING = 3, TRV_ALGO_BUCKET = 4,
               TRV_ALGO_MIRRORED = 16, TRV_ALGO_SINGLE = 32 /* flags, see trv_plan_create_algo */ } trv_algo_t;
typedef enum { TRV_INT32 = 0, TRV_FLOAT32 = 1 } trv_dtype_t;
typedef enum { TRV_SUM = 0 } trv_op_t;

/* Which kernel family executes the schedule.
 *   STEP : one launch per schedule step, exactly as the paper states the steps (latency form:
 *          ping-pong through scratch; bandwidth form: block-indexed three-input Reduce-Scatter
 *          steps and AllGather copy steps, in place).
 *   FUSED: all steps of a column of elements on chip; one read and one write per element.
 *          Exists for the shapes trv_kernel_supported() reports.
 *   AUTO : FUSED where it exists, else STEP.
 *   PIPELINED: the chunk-level readiness engine the paper sketches for a collective-library
 *          backend (App. D): one persistent kernel; a work item per (rank, step, chunk) runs as soon
 *          as what it reads is marked ready, with no barrier between steps.  Latency form: the chunks
 *          of both peers and the local partial of the previous step.  Bandwidth form (power-of-three
 *          sides): a chunk is a piece of one block; a Reduce-Scatter item binds the two incoming
 *          chunks to the local partial of the same block range, an AllGather item copies the finished
 *          chunk from the peer that holds it.  Never chosen by AUTO.  Needs scratch
 *          (trv_scratch_bytes; for a sharded call of the bandwidth form ask with the GLOBAL count);
 *          all its device-side waits are bounded, see trv_pipeline_status.
 * All families give bit-identical results. */
typedef enum { TRV_KERNEL_AUTO = 0, TRV_KERNEL_STEP = 1, TRV_KERNEL_FUSED = 2, TRV_KERNEL_PIPELINED = 3 } trv_kernel_t;

#define TRV_MAX_DIMS 8
#define TRV_MAX_RANKS 1024

/* ---------------------------------------------------------------- plan (schedule builder)
 *
 * trv_plan_create builds the Trivance schedule for a torus with the given sides:
 * peers pi(r,k,n) = (r - 3^k, r + 3^k) mod n (Sec. 4.1); for D > 1 one collective per
 * dimension on 1/D of the vector, collective c using in step t the next dimension, in
 * round-robin order starting at c, that still has steps left (Sec. 5).
 *   dims  : HOST array of ndims sides (1 <= ndims <= TRV_MAX_DIMS), each 3^k, k >= 1
 *   out   : receives the plan; release with trv_plan_destroy
 * Host-only integer work; makes no CUDA call.  A plan's schedule is immutable: it may be used
 * from several threads and streams at once (the one mutable part, the scratch trv_allreduce may
 * allocate for a few shapes, is described there).
 * Errors: INVALID_ARG (NULL, ndims out of range, side < 2), UNSUPPORTED (side not a power
 * of three, more than TRV_MAX_RANKS ranks).
 *
 * Sides of any other size (Sec. 4.4), bandwidth-optimal variant only.  A ring of n >= 2 nodes, n no power of
 * three, gets ceil(log3 n) steps per phase: the regular distances 3^0 .. 3^(s-1), s = floor(log3 n), then one
 * step at distance ceil((n - 3^s) / 2).  The paper fixes the steps, the distances, that no block is sent twice
 * by a node in a phase and that a node sends at most m bytes per phase; which tree a block follows it leaves
 * open.  This library's reading: the AllGather of a block runs the steps in reverse order; the nodes holding
 * the block are kept in the order they got it; in a step every holder, in that order, offers it to its left
 * peer (h - dist), then to its right peer (h + dist); a node that already holds it is skipped.  The
 * Reduce-Scatter runs the same tree backwards, a receiver adding (from_left + own) + from_right and leaving
 * out a side nothing comes from.
 * A torus with such sides (up to four dimensions; the paper evaluates 32 x 32, 8 x 64 and 16 x 16 x 16)
 * composes this with Sec. 5: one collective per dimension on 1/D of the vector; collective c visits the
 * dimensions in round-robin order from c, a dimension whose ring steps are used up being skipped, the k-th
 * visit of a dimension using its ring's k-th distance; sum over d of ceil(log3 a_d) steps per phase.  Along
 * every dimension a block travels by that ring's tree (the same holder rule applied to the torus gives exactly
 * this product of ring trees).  Block j of every collective is owned by linear rank j.
 * Such plans have a STEP family (one launch per step and collective) and a FUSED kernel that walks the block's
 * tree as a stack machine.  The latency-optimal variant is not defined for these sizes: UNSUPPORTED. */
trv_status_t trv_plan_create(const int32_t *dims, int32_t ndims, trv_variant_t variant, trv_plan_t *out);

/* Same, for a comparator schedule (Sec. 2.4, Fig. 1).  TRV_ALGO_BRUCK: peers r + 3^k and
 * r + 2*3^k, both sent in the + direction.  TRV_ALGO_RECDOUB: peer r XOR 2^k on a ring of
 * 2^q ranks (ndims must be 1), the lower rank of a pair sending in the + direction;
 * UNDEFINED_SCHEDULE for other ring sizes.  TRV_ALGO_SWING: peer r + rho(k) for even r and
 * r - rho(k) for odd r, rho(k) = sum_{i<=k} (-2)^i = 1, -1, 3, -5, ... on a ring of 2^q ranks, each
 * message the short way round; block sets by Algorithm 1.  TRV_ALGO_BUCKET: the ring algorithm,
 * n - 1 steps per phase on a ring of any n >= 2, every step one block to the next node (bandwidth
 * form only; rows 0..n-2 Reduce-Scatter, n-1..2n-3 AllGather, both counted forwards).
 * `algo | TRV_ALGO_MIRRORED` (not Trivance): the collective runs a second time with every
 * direction reversed, the two sharing the vector half and half (the mirrored sub-collective by
 * which these one-port schedules use both ports, Sec. 2.4); the plan then has twice the collectives
 * (trv_plan_slices), the second half with negated distances.
 * Recursive Doubling and Swing also take tori with power-of-two sides (Sec. 2.4; Table 2, App. B): one
 * collective per dimension, visiting the dimensions in round-robin order like Trivance, 2 D collectives when
 * mirrored.  `algo | TRV_ALGO_SINGLE` (these two, not mirrored): ONE collective on the whole vector that walks
 * through the dimensions in turn, which is how their latency-optimal forms use a torus (App. B: "only a
 * single port per node").  Bruck takes power-of-three tori.  Bucket takes tori of any sides >= 2 (Sec. 2.4):
 * collective c runs the ring algorithm along dimension c, then c + 1, ... on the blocks a node still answers for (those
 * that agree with its coordinates in the earlier dimensions), sum of (a_d - 1) steps per phase; the AllGather rows take
 * the dimensions in reverse order; D collectives, 2 D when mirrored.
 * Comparator plans serve trv_link_loads, trv_cost_model and the schedule queries, and they are executable:
 * trv_allreduce / trv_allreduce_ex (TRV_KERNEL_AUTO or TRV_KERNEL_STEP) run them step by step, literally -- at
 * the start of a step every rank's vector is copied to a wire buffer (scratch of n * round_up(count, 64) * 4
 * bytes, trv_scratch_bytes), then every rank reduces what its senders put there: the whole slice in the latency
 * form; in the bandwidth form the blocks the receiver still answers for (Reduce-Scatter) and every finished block
 * the sender holds (AllGather, steps reversed).  TRV_ALGO_BRUCK is Bruck with joint reductions (Sec. 3.1).  The
 * paper states no association order; here a rank that gets m0 from the sender whose first peer it is and m1 from
 * the sender whose second peer it is forms (m1 + own) + m0, with one message own + m0.  They are baselines: no
 * fused or pipelined kernel family exists for them (UNSUPPORTED), and trv_allreduce_host is Trivance only. */
trv_status_t trv_plan_create_algo(const int32_t *dims, int32_t ndims, trv_variant_t variant, trv_algo_t algo,
                                  trv_plan_t *out);

trv_status_t trv_plan_destroy(trv_plan_t plan);

/* n = number of ranks; rows = schedule rows = S for the latency form (Sec. 4.2), 2S for the
 * bandwidth form (Reduce-Scatter steps 0..S-1, then the AllGather steps, which mirror
 * S-1..0, Sec. 4.1).  Any output may be NULL. */
trv_status_t trv_plan_info(trv_plan_t plan, int32_t *n, int32_t *ndims, int32_t *rows);

/* Number of concurrent collectives (slices of the vector): ndims, or 2 * ndims for a mirrored comparator. */
trv_status_t trv_plan_slices(trv_plan_t plan, int32_t *nslices);

/* Row `row` of collective (slice) c: the dimension it runs along and the ring distance. */
trv_status_t trv_plan_step(trv_plan_t plan, int32_t c, int32_t row, int32_t *dim, int32_t *dist);

/* peers: HOST array [n][2]; the ranks each rank sends to in that row (Trivance: left = minus
 * distance, right = plus distance; Recursive Doubling: second entry -1). */
trv_status_t trv_plan_peers(trv_plan_t plan, int32_t c, int32_t row, int32_t *peers);

/* set: HOST array of n bytes; set[j] = 1 iff block j is part of the message sent to rank
 * `dst` in Reduce-Scatter step `step` of collective c (closed form Pi of Sec. 4.3: the
 * blocks that agree with dst modulo 3^(visits so far) in every dimension). */
/* With a side that is no power of three (Sec. 4.4) the two senders' sets differ:
 * set[j] then has bit 0 set if dst receives a partial of block j from the node before it along the
 * step's dimension and bit 1 if it receives one from the node after it. */
trv_status_t trv_plan_send_set(trv_plan_t plan, int32_t c, int32_t step, int32_t dst, uint8_t *set);

/* bounds: HOST array of n+1 global element indices: block j of collective c covers
 * [bounds[j], bounds[j+1]).  Slice c = [floor(c*count/D), floor((c+1)*count/D)), block j of a
 * slice [lo,hi) = [lo + floor(j*(hi-lo)/n), lo + floor((j+1)*(hi-lo)/n)) (Sec. 4.1, Sec. 5). */
trv_status_t trv_plan_block_bounds(trv_plan_t plan, size_t count, int32_t c, int64_t *bounds);

/* ---------------------------------------------------------------- AllReduce
 *
 * In-place AllReduce (Sec. 2.2): on return of the work queued on `cuda_stream`, every
 * rank_buffers[r] holds, element-wise, the sum of all n input vectors, associated in the
 * order the schedule defines: each joint reduction is (from_left + own) + from_right
 * (Sec. 3.1, 4.2).  In the latency form the n results differ in rounding for float32
 * (each rank has its own reduction tree); in the bandwidth form all n are identical.
 *   rank_buffers: HOST array of n DEVICE pointers, each >= count*4 bytes, 16-byte aligned,
 *                 pairwise disjoint; caller-owned, never freed here
 *   count       : elements per rank (0 is allowed: nothing happens)
 *   dtype       : TRV_INT32 adds modulo 2^32; TRV_FLOAT32 is IEEE binary32, round to
 *                 nearest even, no flush to zero
 *   op          : TRV_SUM only
 *   cuda_stream : a cudaStream_t (NULL = the legacy default stream)
 * Asynchronous.  For every shape the FUSED family serves (trv_kernel_supported) the call is a pure launch:
 * it allocates nothing, never synchronises and writes nothing into the plan, so any number of threads and
 * streams may use one plan at once.  (Host-side, the library remembers which streams it has seen: the 9 x 9 x 9
 * kernel for long vectors hands out its tiles from a per-stream counter in a fixed device array.)
 * Shapes that fall to the STEP family of the latency form (e.g. a 243 x 3 torus) need ping-pong scratch.  The
 * plan then allocates it with cudaMalloc on first need -- on the device that is current in that call -- keeps it,
 * grows it when a later call needs more (cudaFree + cudaMalloc: this WAITS FOR THE DEVICE) and frees it in
 * trv_plan_destroy.  That scratch binds the plan to its device: a later such call with another device current
 * returns INVALID_ARG.  The grow path is serialised by a lock inside the plan, so concurrent calls are safe on
 * the host; but all such calls on ONE plan share the one scratch and must not overlap on the device (order them
 * on one stream or by events).  To keep trv_allreduce launch-only for these shapes too, call
 * trv_plan_reserve_scratch once beforehand; to use your own scratch, call trv_allreduce_ex. */
trv_status_t trv_allreduce(trv_plan_t plan, void *const *rank_buffers, size_t count, trv_dtype_t dtype, trv_op_t op,
                           void *cuda_stream);

/* Allocates (or grows) the plan-owned scratch that trv_allreduce needs for vectors of up to `count` elements, on
 * the current device; a no-op for shapes that need none.  May wait for the device (it frees a smaller scratch
 * first).  After it, trv_allreduce calls with count' <= count on this plan allocate and synchronise nothing.
 * Errors: INVALID_ARG (the plan's scratch lives on another device), ALLOC, CUDA, UNSUPPORTED (comparator plan). */
trv_status_t trv_plan_reserve_scratch(trv_plan_t plan, size_t count);

/* Bytes of scratch trv_allreduce_ex needs for this call shape (0 if none). */
trv_status_t trv_scratch_bytes(trv_plan_t plan, size_t count, trv_kernel_t kernel, int32_t in_place, size_t *bytes);

/* 1 if the FUSED family exists for this plan, else 0. */
int32_t trv_kernel_supported(trv_plan_t plan, trv_kernel_t kernel);

/* General form.
 *   in_buffers / out_buffers: HOST arrays of n DEVICE pointers (rules as above).  They may be
 *                 the same array (in place); otherwise no input may overlap any output.
 *   count       : elements per rank held in these buffers
 *   global_count, global_offset: the buffers hold elements [global_offset, global_offset +
 *                 count) of per-rank vectors of global_count elements; slice and block
 *                 membership follow the GLOBAL element index.  This is how a vector is
 *                 sharded by element range over several GPUs without any exchange
 *                 (columns are independent).  Pass count and 0 for an unsharded call.
 *   kernel      : kernel family (see trv_kernel_t)
 *   scratch     : DEVICE pointer, 256-byte aligned, scratch_bytes >= trv_scratch_bytes(...);
 *                 may be NULL when 0 bytes are needed.  Contents are undefined afterwards.
 * Errors: as trv_allreduce, plus SCRATCH. */
trv_status_t trv_allreduce_ex(trv_plan_t plan, const void *const *in_buffers, void *const *out_buffers, size_t count,
                              size_t global_count, size_t global_offset, trv_dtype_t dtype, trv_op_t op,
                              trv_kernel_t kernel, void *scratch, size_t scratch_bytes, void *cuda_stream);

/* AllReduce of HOST vectors, pipelined over element-range windows (columns of elements are independent, Sec. 2.2):
 * window k + 1 is copied to the device while window k is reduced there (trv_allreduce_ex with the global element
 * index) and window k - 1 is copied back; three window slots rotate through `workspace`, so the device holds a few
 * windows, never the whole n x count matrix, and both directions of the host link are busy at once.
 *   host_in / host_out: HOST arrays of n HOST pointers to count*4 bytes each; they may be equal (in place).
 *                 Pinned memory is needed for the copies to overlap; equally spaced rows (rows of one matrix)
 *                 are moved by one 2-D copy per window and direction instead of n copies.
 *   workspace   : DEVICE pointer, 256-byte aligned.  trv_host_workspace_bytes(...) is the size for the preferred
 *                 window (an eighth of the vector, between 64 KiB per rank and 512 MiB over all ranks); a smaller
 *                 workspace is accepted and gives shorter windows; SCRATCH if not even windows of 64 elements fit.
 * Uploads and downloads run on two internal streams that the library creates on the first call on a device (make
 * that call outside any stream capture); kernels run on `cuda_stream`.  The internal streams wait for the work
 * queued on `cuda_stream` before the call, and `cuda_stream` ends up waiting for the last download: to the caller
 * the call is work queued on `cuda_stream`.  It returns without synchronising; the host buffers must stay valid
 * until the stream reaches the end of this work.  Calls that share a workspace must be ordered by the caller. */
trv_status_t trv_allreduce_host(trv_plan_t plan, const void *const *host_in, void *const *host_out, size_t count,
                                trv_dtype_t dtype, trv_op_t op, void *workspace, size_t workspace_bytes,
                                void *cuda_stream);
trv_status_t trv_host_workspace_bytes(trv_plan_t plan, size_t count, size_t *bytes);

/* AllReduce for callers that cannot allocate device memory.  (The paper has no counterpart: this
 * is a packaging of the step-by-step latency form, not a part of the method.)
 *
 * Some callers may not call cudaMalloc or cudaFree at all: code running while a stream is being
 * captured into a CUDA graph, code inside a framework that owns all device memory and forbids
 * allocation outside its pool, or a process whose memory budget is fixed at start-up.  The step
 * family of the latency form needs ping-pong scratch; here that scratch is a fixed array of
 * trv_noalloc_max_scratch_bytes() = 16 MiB that is part of the library image.  Every GPU that
 * loads the library gives up those 16 MiB until the process exits.
 *
 * Semantics are those of trv_allreduce (in place, HOST array of n DEVICE pointers, asynchronous on
 * cuda_stream) for latency-optimal Trivance plans, executed by the STEP kernel family; results are
 * bit-identical to trv_allreduce.  The call makes no cudaMalloc, cudaFree or other allocating call.
 *   - The scratch needed is buffers * n * round_up(count, 64) * 4 bytes, buffers = 1 if the plan
 *     has an even number of steps, 2 if odd (1 for a single step).  A call that needs more than the
 *     16 MiB returns TRV_ERR_TOO_LARGE and launches nothing; other plan kinds return UNSUPPORTED.
 *   - The first call on each device looks up the array's device address (once per device, with that
 *     device current).  Make that first call outside any stream capture.
 *   - All calls in the process share the one array, and it keeps whatever the last call left in it.
 *     Nothing in it has to start at zero (every step writes what it later reads), but two calls that
 *     overlap on the GPU (different streams, or different host threads without ordering) race on
 *     it: order them yourself. */
trv_status_t trv_allreduce_noalloc(trv_plan_t plan, void *const *rank_buffers, size_t count, trv_dtype_t dtype,
                                   trv_op_t op, void *cuda_stream);
size_t trv_noalloc_max_scratch_bytes(void);

/* ---------------------------------------------------------------- one joint reduction on caller-described segments
 *
 * out[s][e] = (left[s][e] + own[s][e]) + right[s][e] for e < counts[s], s < nsegments: the joint reduction of the two
 * received partials with the local one (Sec. 3.1, 4.2), in the association order of trv_allreduce.  A NULL left[s] or
 * right[s] (or a NULL array) leaves that side out: left + own, own + right, or a copy.  It serves schedules whose steps
 * are driven from outside the library, above all the rank-sharded form in which every process holds the partials of its
 * own ranks and the partials of the ranks at distance 3^k arrive in receive buffers (Discussion; App. D).
 *   left, own, right, out: HOST arrays of nsegments DEVICE pointers, 4-byte aligned (16-byte accesses are used where a
 *                 segment's pointers share their alignment); out[s] may equal own[s]; no out[] may overlap a left[] or
 *                 right[] of the same call
 *   counts      : HOST array of element counts
 * Asynchronous on cuda_stream; allocates nothing.  Errors: INVALID_ARG, UNSUPPORTED (a count of 2^40 or more), CUDA. */
trv_status_t trv_joint_reduce(const void *const *left, const void *const *own, const void *const *right, void *const *out,
                              const size_t *counts, size_t nsegments, trv_dtype_t dtype, void *cuda_stream);

/* ---------------------------------------------------------------- PIPELINED family: status
 *
 * The PIPELINED kernel (App. D; Discussion, "Joint Reduction Overheads") waits on readiness entries
 * inside the kernel.  Every such wait gives up after a fixed number of polls (about half a second),
 * records TRV_ERR_TIMEOUT in the first bytes of the call's scratch and ends the kernel; the CUDA
 * context stays usable and the output is then undefined.
 *
 * trv_pipeline_status: synchronises `cuda_stream`, reads that record from the DEVICE scratch of the
 * last PIPELINED call and returns TRV_OK or TRV_ERR_TIMEOUT (TRV_ERR_CUDA if the copy fails).
 *
 * trv_pipeline_selftest_timeout: queues one tiny kernel whose single waiter waits, with a limit of
 * 1000 polls, for an entry that nothing sets; a following trv_pipeline_status on the same scratch
 * (at least 512 bytes, 256-byte aligned, DEVICE) returns TRV_ERR_TIMEOUT.  It exists so that the
 * give-up path can be tested without making any real wait fail. */
trv_status_t trv_pipeline_status(const void *scratch, void *cuda_stream);
trv_status_t trv_pipeline_selftest_timeout(void *scratch, size_t scratch_bytes, void *cuda_stream);

/* Some fused kernels fetch their tile by TMA and wait for it on an mbarrier; that wait is bounded.
 * A thread block whose wait runs out stores nothing and adds one to a per-device counter.
 * trv_tma_giveups reads that counter for the current device (a synchronous copy): 0 in every correct
 * run; anything else means outputs of earlier calls are incomplete.  TRV_ERR_CUDA if it cannot be read.
 * A call that uses such a kernel looks up the counter's device address (cudaGetSymbolAddress) and encodes a
 * tensor map on the host; like the first call of trv_allreduce_noalloc, make the first such call on a device
 * outside any stream capture.  If either step fails the call silently uses the kernel without TMA. */
trv_status_t trv_tma_giveups(uint32_t *count);

/* ---------------------------------------------------------------- link loads
 *
 * Per-step, per-directed-link load of the plan's schedule (Sec. 2.1: c_k = number of
 * messages sharing a link in step k; Fig. 1; App. E: deterministic shortest-path routing
 * inside one dimension).  Tallied on the GPU; synchronous (uses the legacy default stream,
 * allocates and frees a few small device buffers).
 *   count, elem_size: per-rank vector length and bytes per element (message bytes use the
 *                 real, possibly uneven, block lengths)
 *   msgs      : HOST int32 [rows][n][D][2]; link leaving `node` along `dim`, index 0 = towards
 *               +, 1 = towards -; number of messages crossing it in that row
 *   bytes     : HOST int64, same shape; bytes crossing it
 *   max_msgs  : HOST int32 [rows]; max over links    max_bytes: HOST int64 [rows]
 * Any output may be NULL. */
trv_status_t trv_link_loads(trv_plan_t plan, size_t count, size_t elem_size, int32_t *msgs, int64_t *bytes,
                            int32_t *max_msgs, int64_t *max_bytes);

/* bytes: HOST int64 [n].  Row < S (Reduce-Scatter or latency form): bytes of the message a
 * rank RECEIVES from each sender in that row, indexed by destination.  Row >= S (AllGather):
 * bytes of the message a rank SENDS to each of its peers, indexed by source.  Host-only. */
/* UNSUPPORTED for plans with a side that is no power of three (the two messages differ): use the next call. */
trv_status_t trv_plan_message_bytes(trv_plan_t plan, size_t count, size_t elem_size, int32_t c, int32_t row,
                                    int64_t *bytes);

/* bytes: HOST array of n: bytes of the message every rank SENDS in that row to its peer number
 * `side` (0: the first peer of trv_plan_peers -- Trivance: r - dist; 1: the second), always
 * indexed by the sending rank; 0 where no message goes that way.  Every kind of plan.  Host-only. */
trv_status_t trv_plan_message_bytes_side(trv_plan_t plan, size_t count, size_t elem_size, int32_t c, int32_t row,
                                         int32_t side, int64_t *bytes);

/* ---------------------------------------------------------------- cost model
 *
 * Congestion-aware cost of the plan's schedule (Sec. 2.1):
 *     C(m, A) = steps(A) * alpha + sum_k beta * m_k * c_k,
 * where the product m_k * c_k of step k is taken as the largest number of bytes any directed link
 * carries in that step (for Trivance every link carries exactly chunk size x congestion).  The
 * link loads come from the same GPU tally as trv_link_loads; synchronous.
 *   alpha: start-up latency per step (seconds); beta: seconds per byte (1 / link bandwidth)
 * Besides the cost, the three optimality factors of Tables 1 and 2 are returned:
 *   lambda = steps / log3 n                        (latency;   Trivance: 1 or 2)
 *   delta  = bytes a node sends in total / (2 m)   (bandwidth; m = count * elem_size)
 *   theta  = sum_k m_k c_k / (m / D)               (transmission delay) */
typedef struct {
    int32_t steps;
    int64_t bytes_sent_per_node;    /* maximum over nodes */
    int64_t tx_bytes;               /* sum over steps of the most loaded link's bytes */
    double latency_term, tx_term, total;   /* seconds */
    double lambda, delta, theta;
} trv_cost_t;
trv_status_t trv_cost_model(trv_plan_t plan, size_t count, size_t elem_size, double alpha, double beta, trv_cost_t *out);

/* ---------------------------------------------------------------- misc */

const char *trv_strerror(trv_status_t status);

/* Number of kernels this library has launched in this process so far. */
uint64_t trv_launch_count(void);

/* Name of the kernel family member the last trv_allreduce* call of this thread used
 * (static string, e.g. "lat_reg<27>", "step"); for reports. */
const char *trv_last_kernel_name(void);

#ifdef __cplusplus
}
#endif
#endif /* TRIVANCE_H_ */
