// trv_allreduce_host: AllReduce of vectors that live in HOST memory, as a pipeline of element-range windows.
//
// Columns of elements are independent (Sec. 2.2: the reduction is element-wise), so the vector is cut into
// windows of W elements; window k is uploaded, reduced on the device by trv_allreduce_ex with the GLOBAL
// element index (global_count = count, global_offset = k * W: slice and block membership are unchanged) and
// downloaded.  Three window slots rotate through the caller's workspace, so that the upload of window k + 1,
// the kernel of window k and the download of window k - 1 are in flight together: the two copy directions of
// the host link run concurrently and the kernel hides behind them.  The device workspace is three windows,
// not the whole n * count matrix.
//
// Streams: uploads run on an internal stream, downloads on a second one, kernels on the caller's stream.
// The internal streams start after the work already queued on the caller's stream (event fork) and the
// caller's stream ends by waiting for the last download (event join), so for the caller the call behaves
// like work queued on its stream.  The internal streams and events exist once per device; they are created
// by the first call on that device.
#include <algorithm>
#include <mutex>
#include <vector>

#include "trv_dev.cuh"

namespace {
using namespace trv;

constexpr int kSlots = 3;
constexpr int kMaxDevices = 64;
constexpr size_t kMinWindow = 16384;            // elements: a row copy of at least 64 KiB
constexpr size_t kWindowBudget = 128u << 20;    // elements per window over all ranks (512 MiB); 729 x 32 MiB end to end:
                                                // 42.6 GB/s with 128 MiB windows, 43.7 with 256 MiB, 43.8 with 512 MiB, 41.7 with 1 GiB

struct HostCtx {
    bool ready = false;
    cudaStream_t up = nullptr, down = nullptr;
    cudaEvent_t fork = nullptr, joined = nullptr, in_ready[kSlots] = {}, done[kSlots] = {}, freed[kSlots] = {};
};
std::mutex g_mu;
HostCtx g_ctx[kMaxDevices];

// Caller holds g_mu.
HostCtx* host_ctx() {
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return nullptr;
    HostCtx& c = g_ctx[dev];
    if (c.ready) return &c;
    bool ok = cudaStreamCreateWithFlags(&c.up, cudaStreamNonBlocking) == cudaSuccess &&
              cudaStreamCreateWithFlags(&c.down, cudaStreamNonBlocking) == cudaSuccess &&
              cudaEventCreateWithFlags(&c.fork, cudaEventDisableTiming) == cudaSuccess &&
              cudaEventCreateWithFlags(&c.joined, cudaEventDisableTiming) == cudaSuccess;
    for (int s = 0; s < kSlots && ok; ++s)
        ok = cudaEventCreateWithFlags(&c.in_ready[s], cudaEventDisableTiming) == cudaSuccess &&
             cudaEventCreateWithFlags(&c.done[s], cudaEventDisableTiming) == cudaSuccess &&
             cudaEventCreateWithFlags(&c.freed[s], cudaEventDisableTiming) == cudaSuccess;
    if (!ok) { (void)cudaGetLastError(); return nullptr; }
    c.ready = true;
    return &c;
}

size_t round_up64(size_t v) { return (v + 63) & ~(size_t)63; }

// Window length the call would like: an eighth of the vector (so that even a short vector overlaps its two
// copy directions), at least 64 KiB per row copy, at most 512 MiB per window.
size_t preferred_window(int n, size_t count) {
    size_t w = round_up64((count + 7) / 8);
    const size_t cap = std::max(kMinWindow, (kWindowBudget / (size_t)n) & ~(size_t)63);
    w = std::min(std::max(w, kMinWindow), cap);
    return std::min(w, round_up64(count));
}

trv_status_t slot_bytes(trv_plan_t plan, size_t window, size_t* bytes) {
    size_t scratch = 0;
    const trv_status_t st = trv_scratch_bytes(plan, window, TRV_KERNEL_AUTO, 1, &scratch);
    if (st != TRV_OK) return st;
    *bytes = (size_t)plan->plan.n * window * 4 + ((scratch + 255) & ~(size_t)255);
    return TRV_OK;
}

// rows[r] = base + r * pitch with 0 < pitch <= the largest pitch a 2-D copy takes?
bool uniform_host_rows(const void* const* rows, int n, size_t row_bytes, size_t* pitch) {
    if (n == 1) { *pitch = row_bytes ? row_bytes : 4; return true; }
    const ptrdiff_t d = (const char*)rows[1] - (const char*)rows[0];
    if (d <= 0 || (size_t)d < row_bytes || (size_t)d > 0x7fffffffu) return false;
    for (int r = 2; r < n; ++r)
        if ((const char*)rows[r] - (const char*)rows[r - 1] != d) return false;
    *pitch = (size_t)d;
    return true;
}
}  // namespace

extern "C" {

trv_status_t trv_host_workspace_bytes(trv_plan_t plan, size_t count, size_t* bytes) {
    if (!plan || !bytes) return TRV_ERR_INVALID_ARG;
    if (plan->plan.algo != TRV_ALGO_TRIVANCE) return TRV_ERR_UNSUPPORTED;
    if (count >= ((size_t)1 << 40)) return TRV_ERR_UNSUPPORTED;
    const size_t w = preferred_window(plan->plan.n, std::max<size_t>(count, 1));
    const size_t windows = count ? (count + w - 1) / w : 1;
    size_t one = 0;
    const trv_status_t st = slot_bytes(plan, w, &one);
    if (st != TRV_OK) return st;
    *bytes = one * std::min<size_t>(kSlots, windows);
    return TRV_OK;
}

trv_status_t trv_allreduce_host(trv_plan_t plan, const void* const* host_in, void* const* host_out, size_t count,
                                trv_dtype_t dtype, trv_op_t op, void* workspace, size_t workspace_bytes,
                                void* cuda_stream) {
    if (!plan || !host_in || !host_out) return TRV_ERR_INVALID_ARG;
    const Plan& p = plan->plan;
    const int n = p.n;
    if (p.algo != TRV_ALGO_TRIVANCE) return TRV_ERR_UNSUPPORTED;
    if (dtype != TRV_INT32 && dtype != TRV_FLOAT32) return TRV_ERR_INVALID_ARG;
    if (op != TRV_SUM) return TRV_ERR_UNSUPPORTED;
    if (count >= ((size_t)1 << 40)) return TRV_ERR_UNSUPPORTED;
    for (int r = 0; r < n; ++r)
        if (!host_in[r] || !host_out[r]) return TRV_ERR_INVALID_ARG;
    if (!workspace || ((uintptr_t)workspace & 255)) return TRV_ERR_SCRATCH;
    if (count == 0) return TRV_OK;

    // window length: the preferred one, or what the given workspace has room for (three slots; fewer windows
    // than slots need fewer)
    size_t w = preferred_window(n, count), one = 0;
    trv_status_t st = slot_bytes(plan, w, &one);
    if (st != TRV_OK) return st;
    size_t windows = (count + w - 1) / w;
    if (one * std::min<size_t>(kSlots, windows) > workspace_bytes) {
        size_t unit = 0;                        // bytes of a slot per 64 elements of window (the scratch is linear in it)
        st = slot_bytes(plan, 64, &unit);
        if (st != TRV_OK) return st;
        w = 64 * (workspace_bytes / (kSlots * unit));
        while (w >= 64 && (slot_bytes(plan, w, &one) != TRV_OK || one * kSlots > workspace_bytes)) w -= 64;
        if (w < 64) return TRV_ERR_SCRATCH;
        windows = (count + w - 1) / w;
    }
    const int slots = (int)std::min<size_t>(kSlots, windows);
    const size_t rows_bytes = (size_t)n * w * 4;

    cudaStream_t s = (cudaStream_t)cuda_stream;
    std::vector<void*> dev((size_t)slots * n);
    for (int k = 0; k < slots; ++k)
        for (int r = 0; r < n; ++r) dev[(size_t)k * n + r] = (char*)workspace + (size_t)k * one + (size_t)r * w * 4;
    size_t pitch_in = 0, pitch_out = 0;
    const bool in2d = uniform_host_rows(host_in, n, count * 4, &pitch_in);
    const bool out2d = uniform_host_rows((const void* const*)host_out, n, count * 4, &pitch_out);

    // One call at a time issues into the shared internal streams: record/wait pairs of two calls never interleave.
    std::lock_guard<std::mutex> lock(g_mu);
    HostCtx* c = host_ctx();
    if (!c) return TRV_ERR_CUDA;
    trv_status_t result = TRV_OK;
    auto ok = [&](cudaError_t e) {
        if (e != cudaSuccess && result == TRV_OK) result = TRV_ERR_CUDA;
        return e == cudaSuccess;
    };
    auto window = [&](size_t k) -> bool {
        const int slot = (int)(k % slots);
        const size_t e0 = k * w, len = std::min(w, count - e0);
        void* const* rows = dev.data() + (size_t)slot * n;
        char* const scratch = (char*)workspace + (size_t)slot * one + rows_bytes;
        if (k >= (size_t)slots && !ok(cudaStreamWaitEvent(c->up, c->freed[slot], 0))) return false;   // slot's last download over
        if (in2d) {
            if (!ok(cudaMemcpy2DAsync(rows[0], w * 4, (const char*)host_in[0] + e0 * 4, pitch_in, len * 4, n,
                                      cudaMemcpyHostToDevice, c->up))) return false;
        } else {
            for (int r = 0; r < n; ++r)
                if (!ok(cudaMemcpyAsync(rows[r], (const char*)host_in[r] + e0 * 4, len * 4, cudaMemcpyHostToDevice, c->up)))
                    return false;
        }
        if (!ok(cudaEventRecord(c->in_ready[slot], c->up)) || !ok(cudaStreamWaitEvent(s, c->in_ready[slot], 0))) return false;
        const trv_status_t st2 = trv_allreduce_ex(plan, (const void* const*)rows, rows, len, count, e0, dtype, op, TRV_KERNEL_AUTO,
                                                  one > rows_bytes ? scratch : nullptr, one - rows_bytes, s);
        if (st2 != TRV_OK) { result = st2; return false; }
        if (!ok(cudaEventRecord(c->done[slot], s)) || !ok(cudaStreamWaitEvent(c->down, c->done[slot], 0))) return false;
        if (out2d) {
            if (!ok(cudaMemcpy2DAsync((char*)host_out[0] + e0 * 4, pitch_out, rows[0], w * 4, len * 4, n,
                                      cudaMemcpyDeviceToHost, c->down))) return false;
        } else {
            for (int r = 0; r < n; ++r)
                if (!ok(cudaMemcpyAsync((char*)host_out[r] + e0 * 4, rows[r], len * 4, cudaMemcpyDeviceToHost, c->down)))
                    return false;
        }
        return ok(cudaEventRecord(c->freed[slot], c->down));
    };
    if (!ok(cudaEventRecord(c->fork, s)) || !ok(cudaStreamWaitEvent(c->up, c->fork, 0)) ||
        !ok(cudaStreamWaitEvent(c->down, c->fork, 0)))
        return result;
    for (size_t k = 0; k < windows; ++k)
        if (!window(k)) break;
    // join also after a failure: whatever was queued on the internal streams stays ordered before the caller's next work
    ok(cudaEventRecord(c->joined, c->up));
    ok(cudaStreamWaitEvent(s, c->joined, 0));
    ok(cudaEventRecord(c->joined, c->down));
    ok(cudaStreamWaitEvent(s, c->joined, 0));
    return result;
}

}  // extern "C"
