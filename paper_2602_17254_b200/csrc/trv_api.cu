// C ABI of the Trivance engine: argument checks, kernel-family choice, host-buffer variant.
#include <algorithm>
#include <cmath>
#include <cstring>
#include <vector>

#include "trv_dev.cuh"
#include "trv_tma.cuh"

namespace trv {
std::atomic<uint64_t> g_launches{0};
thread_local const char* g_last_kernel = "none";

static bool fused_supported(const Plan& p) {
    if (p.general) return fused_tree_supported(p);
    return p.variant == TRV_LATENCY_OPTIMAL ? fused_latency_supported(p) : fused_bandwidth_supported(p);
}

void prepare_launch_data(Plan& p) {
    if (p.algo != TRV_ALGO_TRIVANCE) return;
    if (p.general) tree_prepare(p);
    else if (p.variant == TRV_LATENCY_OPTIMAL) latency_prepare(p);
}

static trv_status_t check_buffers(const Plan& p, const void* const* in, void* const* out, size_t count, bool* in_place) {
    if (!in || !out) return TRV_ERR_INVALID_ARG;
    const int n = p.n;
    bool same = true;
    for (int r = 0; r < n; ++r) {
        if (!in[r] || !out[r]) return TRV_ERR_INVALID_ARG;
        if (((uintptr_t)in[r] | (uintptr_t)out[r]) & 15) return TRV_ERR_INVALID_ARG;
        if (in[r] != out[r]) same = false;
    }
    // pairwise disjoint outputs; inputs either identical to the outputs or disjoint from all of them
    const size_t bytes = count * 4;
    {   // the usual case needs no sorting: equally spaced rows (of one tensor) are disjoint as soon as the spacing holds a
        // row, and two such families either are the same or must not touch (243 ranks: 3 us of a 9 us call otherwise)
        StrideAddr so, si;
        if (n > 1 && uniform_stride((const void* const*)out, n, &so) && so.stride >= bytes &&
            (same || (uniform_stride(in, n, &si) && si.stride >= bytes))) {
            if (!same) {
                const uintptr_t o0 = (uintptr_t)so.base, o1 = o0 + (uintptr_t)so.stride * (n - 1) + bytes;
                const uintptr_t i0 = (uintptr_t)si.base, i1 = i0 + (uintptr_t)si.stride * (n - 1) + bytes;
                if (i0 < o1 && o0 < i1) goto sorted_check;      // the two spans meet: let the general check decide
            }
            *in_place = same;
            return TRV_OK;
        }
    }
sorted_check:
    std::vector<std::pair<uintptr_t, int>> iv;
    iv.reserve(2 * (size_t)n);
    for (int r = 0; r < n; ++r) iv.emplace_back((uintptr_t)out[r], 1);
    if (!same)
        for (int r = 0; r < n; ++r) iv.emplace_back((uintptr_t)in[r], 0);
    std::sort(iv.begin(), iv.end());
    for (size_t i = 1; i < iv.size(); ++i) {
        if (iv[i - 1].first + bytes > iv[i].first) {
            // two inputs may coincide or overlap each other (reading is harmless); anything
            // touching an output may not
            if (iv[i - 1].second == 0 && iv[i].second == 0) continue;
            return TRV_ERR_INVALID_ARG;
        }
    }
    *in_place = same;
    return TRV_OK;
}

static trv_status_t dispatch(Call& c, trv_kernel_t kernel) {
    const Plan& p = *c.plan;
    bool fused = false;
    if (kernel == TRV_KERNEL_PIPELINED)
        return p.variant == TRV_BANDWIDTH_OPTIMAL && !p.general ? run_pipeline_bandwidth(c) : run_pipeline_latency(c);
    if (kernel == TRV_KERNEL_FUSED) {
        if (!fused_supported(p)) return TRV_ERR_UNSUPPORTED;
        fused = true;
    } else if (kernel == TRV_KERNEL_AUTO) {
        fused = fused_supported(p);
    }
    if (fused) {
        const trv_status_t st = p.general ? run_fused_tree(c)
                                : (p.variant == TRV_LATENCY_OPTIMAL ? run_fused_latency(c) : run_fused_bandwidth(c));
        // a fused launcher that cannot serve this call shape: AUTO goes on to the STEP family (which checks the scratch)
        if (st != TRV_ERR_UNSUPPORTED || kernel != TRV_KERNEL_AUTO) return st;
    }
    if (p.general) return run_step_general(c);
    return p.variant == TRV_LATENCY_OPTIMAL ? run_step_latency(c) : run_step_bandwidth(c);
}
}  // namespace trv

using namespace trv;

extern "C" {

trv_status_t trv_plan_create(const int32_t* dims, int32_t ndims, trv_variant_t variant, trv_plan_t* out) {
    return trv_plan_create_algo(dims, ndims, variant, TRV_ALGO_TRIVANCE, out);
}

trv_status_t trv_plan_create_algo(const int32_t* dims, int32_t ndims, trv_variant_t variant, trv_algo_t algo,
                                  trv_plan_t* out) {
    if (!out) return TRV_ERR_INVALID_ARG;
    *out = nullptr;
    const trv_status_t st = build_plan(dims, ndims, (int)variant, (int)algo, out);
    if (st == TRV_OK) prepare_launch_data((*out)->plan);
    return st;
}

trv_status_t trv_plan_destroy(trv_plan_t plan) {
    if (!plan) return TRV_ERR_INVALID_ARG;
    trv_status_t st = TRV_OK;
    if (plan->plan.scratch && cudaFree(plan->plan.scratch) != cudaSuccess) st = TRV_ERR_CUDA;
    delete plan;
    return st;
}

trv_status_t trv_plan_info(trv_plan_t plan, int32_t* n, int32_t* ndims, int32_t* rows) {
    if (!plan) return TRV_ERR_INVALID_ARG;
    if (n) *n = plan->plan.n;
    if (ndims) *ndims = plan->plan.ndims;
    if (rows) *rows = plan->plan.rows();
    return TRV_OK;
}

trv_status_t trv_plan_slices(trv_plan_t plan, int32_t* nslices) {
    if (!plan || !nslices) return TRV_ERR_INVALID_ARG;
    *nslices = plan->plan.nslices;
    return TRV_OK;
}

trv_status_t trv_plan_step(trv_plan_t plan, int32_t c, int32_t row, int32_t* dim, int32_t* dist) {
    if (!plan) return TRV_ERR_INVALID_ARG;
    const Plan& p = plan->plan;
    if (c < 0 || c >= p.nslices || row < 0 || row >= p.rows()) return TRV_ERR_INVALID_ARG;
    const Step& s = p.steps[c][p.row_step(c, row)];
    if (dim) *dim = s.dim;
    if (dist) *dist = s.dist;
    return TRV_OK;
}

trv_status_t trv_plan_peers(trv_plan_t plan, int32_t c, int32_t row, int32_t* peers) {
    if (!plan || !peers) return TRV_ERR_INVALID_ARG;
    const Plan& p = plan->plan;
    if (c < 0 || c >= p.nslices || row < 0 || row >= p.rows()) return TRV_ERR_INVALID_ARG;
    const Step& s = p.steps[c][p.row_step(c, row)];
    for (int r = 0; r < p.n; ++r) {
        int peer[2], dir[2], hops[2];
        send_peers(p, r, s.dim, s.dist, peer, dir, hops);
        peers[2 * r] = peer[0];
        peers[2 * r + 1] = peer[1];
    }
    return TRV_OK;
}

trv_status_t trv_plan_send_set(trv_plan_t plan, int32_t c, int32_t step, int32_t dst, uint8_t* set) {
    if (!plan || !set) return TRV_ERR_INVALID_ARG;
    const Plan& p = plan->plan;
    if (c < 0 || c >= p.nslices || step < 0 || step >= p.S || dst < 0 || dst >= p.n) return TRV_ERR_INVALID_ARG;
    for (int j = 0; j < p.n; ++j)
        set[j] = p.general ? (uint8_t)general_recv_mask(p, c, step, dst, j) : (in_send_set(p, c, step, dst, j) ? 1 : 0);
    return TRV_OK;
}

trv_status_t trv_plan_block_bounds(trv_plan_t plan, size_t count, int32_t c, int64_t* bounds) {
    if (!plan || !bounds) return TRV_ERR_INVALID_ARG;
    const Plan& p = plan->plan;
    if (c < 0 || c >= p.nslices) return TRV_ERR_INVALID_ARG;
    const int64_t lo = slice_lo((int64_t)count, p.nslices, c), hi = slice_lo((int64_t)count, p.nslices, c + 1);
    for (int j = 0; j <= p.n; ++j) bounds[j] = block_lo(lo, hi, p.n, j);
    return TRV_OK;
}

trv_status_t trv_plan_message_bytes(trv_plan_t plan, size_t count, size_t elem_size, int32_t c, int32_t row,
                                    int64_t* bytes) {
    if (!plan || !bytes || elem_size == 0) return TRV_ERR_INVALID_ARG;
    const Plan& p = plan->plan;
    if (c < 0 || c >= p.nslices || row < 0 || row >= p.rows()) return TRV_ERR_INVALID_ARG;
    if (p.general) return TRV_ERR_UNSUPPORTED;
    message_bytes(p, (int64_t)count, (int64_t)elem_size, c, row, bytes);
    return TRV_OK;
}

trv_status_t trv_plan_message_bytes_side(trv_plan_t plan, size_t count, size_t elem_size, int32_t c, int32_t row,
                                         int32_t side, int64_t* bytes) {
    if (!plan || !bytes || elem_size == 0 || side < 0 || side > 1) return TRV_ERR_INVALID_ARG;
    const Plan& p = plan->plan;
    if (c < 0 || c >= p.nslices || row < 0 || row >= p.rows()) return TRV_ERR_INVALID_ARG;
    message_bytes_side(p, (int64_t)count, (int64_t)elem_size, c, row, side, bytes);
    return TRV_OK;
}

int32_t trv_kernel_supported(trv_plan_t plan, trv_kernel_t kernel) {
    if (!plan) return 0;
    if (plan->plan.algo != TRV_ALGO_TRIVANCE) {
        if (plan->plan.algo == TRV_ALGO_BUCKET && plan->plan.variant != TRV_BANDWIDTH_OPTIMAL) return 0;
        return (kernel == TRV_KERNEL_AUTO || kernel == TRV_KERNEL_STEP) ? 1 : 0;
    }
    if (kernel == TRV_KERNEL_FUSED) return fused_supported(plan->plan) ? 1 : 0;
    if (kernel == TRV_KERNEL_PIPELINED) return (pipeline_supported(plan->plan, false) || pipeline_bw_supported(plan->plan)) ? 1 : 0;
    return (kernel == TRV_KERNEL_AUTO || kernel == TRV_KERNEL_STEP) ? 1 : 0;
}

trv_status_t trv_scratch_bytes(trv_plan_t plan, size_t count, trv_kernel_t kernel, int32_t in_place, size_t* bytes) {
    if (!plan || !bytes) return TRV_ERR_INVALID_ARG;
    const Plan& p = plan->plan;
    if (p.algo != TRV_ALGO_TRIVANCE) {      // comparator schedules: the step-by-step executor and its wire buffer
        if (kernel != TRV_KERNEL_AUTO && kernel != TRV_KERNEL_STEP) return TRV_ERR_UNSUPPORTED;
        if (p.algo == TRV_ALGO_BUCKET && p.variant != TRV_BANDWIDTH_OPTIMAL) return TRV_ERR_UNSUPPORTED;
        *bytes = comparator_scratch_bytes(p, count);
        return TRV_OK;
    }
    bool fused = false;
    if (kernel == TRV_KERNEL_PIPELINED) {
        if (pipeline_bw_supported(p)) { *bytes = pipeline_bw_scratch_bytes(p, count); return TRV_OK; }
        if (!pipeline_supported(p, in_place != 0)) return TRV_ERR_UNSUPPORTED;
        *bytes = pipeline_scratch_bytes(p, count);
        return TRV_OK;
    }
    if (kernel == TRV_KERNEL_FUSED) {
        if (!fused_supported(p)) return TRV_ERR_UNSUPPORTED;
        fused = true;
    } else if (kernel == TRV_KERNEL_AUTO) {
        fused = fused_supported(p);
    } else if (kernel != TRV_KERNEL_STEP) {
        return TRV_ERR_INVALID_ARG;
    }
    *bytes = fused ? 0 : step_scratch_bytes(p, count, in_place != 0);
    return TRV_OK;
}

trv_status_t trv_allreduce_ex(trv_plan_t plan, const void* const* in_buffers, void* const* out_buffers, size_t count,
                              size_t global_count, size_t global_offset, trv_dtype_t dtype, trv_op_t op,
                              trv_kernel_t kernel, void* scratch, size_t scratch_bytes, void* cuda_stream) {
    if (!plan) return TRV_ERR_INVALID_ARG;
    const Plan& p = plan->plan;
    if (p.algo != TRV_ALGO_TRIVANCE && kernel != TRV_KERNEL_AUTO && kernel != TRV_KERNEL_STEP) return TRV_ERR_UNSUPPORTED;
    if (p.algo == TRV_ALGO_BUCKET && p.variant != TRV_BANDWIDTH_OPTIMAL) return TRV_ERR_UNSUPPORTED;
    if (dtype != TRV_INT32 && dtype != TRV_FLOAT32) return TRV_ERR_INVALID_ARG;
    if (op != TRV_SUM) return TRV_ERR_UNSUPPORTED;
    if (kernel != TRV_KERNEL_AUTO && kernel != TRV_KERNEL_STEP && kernel != TRV_KERNEL_FUSED && kernel != TRV_KERNEL_PIPELINED)
        return TRV_ERR_INVALID_ARG;
    if (global_offset > global_count || count > global_count - global_offset) return TRV_ERR_INVALID_ARG;
    if (count >= ((size_t)1 << 40)) return TRV_ERR_UNSUPPORTED;
    bool in_place = false;
    trv_status_t st = check_buffers(p, in_buffers, out_buffers, count, &in_place);
    if (st != TRV_OK) return st;
    if (scratch_bytes && (!scratch || ((uintptr_t)scratch & 255))) return TRV_ERR_SCRATCH;
    if (count == 0) return TRV_OK;
    Call c{&p, in_buffers, out_buffers, count, global_count, global_offset, (int)dtype, in_place,
           scratch, scratch_bytes, (cudaStream_t)cuda_stream};
    if (p.algo != TRV_ALGO_TRIVANCE) return run_comparator(c);
    return dispatch(c, kernel);
}

// Grows the plan-owned scratch to `need` bytes on the current device.  Caller holds scratch_mu.
static trv_status_t grow_plan_scratch(Plan& p, size_t need) {
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess) return TRV_ERR_CUDA;
    if (p.scratch && p.scratch_device != dev) return TRV_ERR_INVALID_ARG;   // the scratch lives on another GPU
    if (need <= p.scratch_bytes) return TRV_OK;
    // cudaFree waits for the device: kernels of earlier calls that still use the old scratch finish first
    if (p.scratch) { cudaFree(p.scratch); p.scratch = nullptr; p.scratch_bytes = 0; p.scratch_device = -1; }
    if (cudaMalloc(&p.scratch, need) != cudaSuccess) { (void)cudaGetLastError(); return TRV_ERR_ALLOC; }
    p.scratch_bytes = need;
    p.scratch_device = dev;
    return TRV_OK;
}

trv_status_t trv_plan_reserve_scratch(trv_plan_t plan, size_t count) {
    if (!plan) return TRV_ERR_INVALID_ARG;
    size_t need = 0;
    trv_status_t st = trv_scratch_bytes(plan, count, TRV_KERNEL_AUTO, 1, &need);
    if (st != TRV_OK) return st;
    std::lock_guard<std::mutex> lock(plan->scratch_mu);
    if (need == 0 && !plan->plan.scratch) return TRV_OK;
    return grow_plan_scratch(plan->plan, need);
}

trv_status_t trv_allreduce(trv_plan_t plan, void* const* rank_buffers, size_t count, trv_dtype_t dtype, trv_op_t op,
                           void* cuda_stream) {
    if (!plan) return TRV_ERR_INVALID_ARG;
    Plan& p = plan->plan;
    size_t need = 0;
    trv_status_t st = trv_scratch_bytes(plan, count, TRV_KERNEL_AUTO, 1, &need);
    if (st != TRV_OK) return st;
    if (need == 0)      // the fused kernels: a pure launch, nothing of the plan is written
        return trv_allreduce_ex(plan, (const void* const*)rank_buffers, rank_buffers, count, count, 0, dtype, op,
                                TRV_KERNEL_AUTO, nullptr, 0, cuda_stream);
    // STEP family of the latency form: the plan's own scratch.  The lock is held until the launches are queued, so
    // that a concurrent call which has to grow (and free) the scratch cannot pull it away in between.
    std::lock_guard<std::mutex> lock(plan->scratch_mu);
    if (need > p.scratch_bytes || !p.scratch) {
        bool ip;        // validate before allocating anything
        if (dtype != TRV_INT32 && dtype != TRV_FLOAT32) return TRV_ERR_INVALID_ARG;
        if (op != TRV_SUM) return TRV_ERR_UNSUPPORTED;
        st = check_buffers(p, (const void* const*)rank_buffers, rank_buffers, count, &ip);
        if (st != TRV_OK) return st;
    }
    st = grow_plan_scratch(p, need);
    if (st != TRV_OK) return st;
    return trv_allreduce_ex(plan, (const void* const*)rank_buffers, rank_buffers, count, count, 0, dtype, op,
                            TRV_KERNEL_AUTO, p.scratch, p.scratch_bytes, cuda_stream);
}

trv_status_t trv_tma_giveups(uint32_t* count) {
    if (!count) return TRV_ERR_INVALID_ARG;
    const unsigned v = tma_giveups();
    if (v == ~0u) return TRV_ERR_CUDA;
    *count = v;
    return TRV_OK;
}

trv_status_t trv_pipeline_status(const void* scratch, void* cuda_stream) {
    if (!scratch) return TRV_ERR_INVALID_ARG;
    return pipeline_status(scratch, (cudaStream_t)cuda_stream);
}

trv_status_t trv_pipeline_selftest_timeout(void* scratch, size_t scratch_bytes, void* cuda_stream) {
    if (!scratch || ((uintptr_t)scratch & 255)) return TRV_ERR_SCRATCH;
    return pipeline_selftest_timeout(scratch, scratch_bytes, (cudaStream_t)cuda_stream);
}

trv_status_t trv_link_loads(trv_plan_t plan, size_t count, size_t elem_size, int32_t* msgs, int64_t* bytes,
                            int32_t* max_msgs, int64_t* max_bytes) {
    if (!plan || elem_size == 0) return TRV_ERR_INVALID_ARG;
    return run_link_loads(plan->plan, count, elem_size, msgs, bytes, max_msgs, max_bytes);
}

trv_status_t trv_cost_model(trv_plan_t plan, size_t count, size_t elem_size, double alpha, double beta, trv_cost_t* out) {
    if (!plan || !out || elem_size == 0 || !(alpha >= 0) || !(beta >= 0)) return TRV_ERR_INVALID_ARG;
    const Plan& p = plan->plan;
    const int T = p.rows(), n = p.n, D = p.ndims;
    std::vector<int64_t> max_bytes((size_t)T), mb((size_t)n), sent((size_t)n, 0);
    trv_status_t st = run_link_loads(p, count, elem_size, nullptr, nullptr, nullptr, max_bytes.data());
    if (st != TRV_OK) return st;
    // bytes every node sends: both of its messages in every row of every collective
    for (int c = 0; c < p.nslices; ++c)
        for (int row = 0; row < T; ++row)
            for (int side = 0; side < 2; ++side) {
                message_bytes_side(p, (int64_t)count, (int64_t)elem_size, c, row, side, mb.data());
                for (int r = 0; r < n; ++r) sent[r] += mb[r];
            }
    int64_t tx = 0, smax = 0;
    for (int row = 0; row < T; ++row) tx += max_bytes[row];
    for (int r = 0; r < n; ++r) smax = std::max(smax, sent[r]);
    const double m = (double)count * (double)elem_size;
    const double log3n = std::log((double)n) / std::log(3.0);
    out->steps = T;
    out->bytes_sent_per_node = smax;
    out->tx_bytes = tx;
    out->latency_term = T * alpha;
    out->tx_term = beta * (double)tx;
    out->total = out->latency_term + out->tx_term;
    out->lambda = log3n > 0 ? T / log3n : 0;
    out->delta = m > 0 ? (double)smax / (2.0 * m) : 0;
    out->theta = m > 0 ? (double)tx / (m / D) : 0;
    return TRV_OK;
}

const char* trv_strerror(trv_status_t status) {
    switch (status) {
        case TRV_OK: return "ok";
        case TRV_ERR_INVALID_ARG: return "invalid argument";
        case TRV_ERR_UNSUPPORTED: return "unsupported (side not a power of three, too many ranks, or op/plan kind not executable)";
        case TRV_ERR_UNDEFINED_SCHEDULE: return "schedule undefined for this number of ranks";
        case TRV_ERR_ALLOC: return "allocation failed";
        case TRV_ERR_CUDA: return "CUDA runtime error";
        case TRV_ERR_SCRATCH: return "scratch or workspace too small or misaligned";
        case TRV_ERR_TOO_LARGE: return "size exceeds the fixed scratch capacity of the no-allocation entry point";
        case TRV_ERR_TIMEOUT: return "a bounded device-side wait of the pipelined kernel ran out";
    }
    return "unknown status";
}

uint64_t trv_launch_count(void) { return g_launches.load(std::memory_order_relaxed); }

const char* trv_last_kernel_name(void) { return g_last_kernel; }

}  // extern "C"
