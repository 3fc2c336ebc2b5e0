// The operator on HOST buffers: chunked copy-in / launch / copy-out pipeline (end-to-end entry point).
// Rows are independent, so a tensor is cut into row chunks; three chunk slots rotate so that the
// host-to-device copies of chunk i+1, the kernel of chunk i and the device-to-host copies of chunk
// i-1 run at the same time on three streams.
#include <string.h>

#include <mutex>

#include "tuner_internal.h"

namespace rt {
namespace {

constexpr int kSlots = 3;
constexpr int64_t kAlign = 256;

struct HostPipe {
    bool ready = false;
    cudaStream_t h2d = nullptr, d2h = nullptr;
    cudaEvent_t loaded[kSlots], computed[kSlots], drained[kSlots], start = nullptr;
};
HostPipe g_pipe[64];
std::mutex g_pipe_mutex;

int64_t round_up(int64_t v, int64_t a) { return (v + a - 1) / a * a; }

int64_t pick_chunk(int64_t n_tokens, int64_t hidden, int dtype, int64_t chunk_tokens)
{
    if (n_tokens <= 0) return 1;
    if (chunk_tokens <= 0) {
        // about 16 MB per tensor per chunk: measured on B200 over PCIe Gen5 x16 (bf16 16384 x 8192, both
        // directions busy), 8-16 MB chunks give the shortest step; 32 MB loses 5% to the pipeline's fill and
        // drain, 2 MB and below lose more to per-copy overhead
        const int64_t row_bytes = hidden * elem_bytes_of(dtype);
        chunk_tokens = std::max<int64_t>(1, (16LL << 20) / std::max<int64_t>(1, row_bytes));
    }
    return std::min(chunk_tokens, n_tokens);
}

int get_pipe(HostPipe** out)
{
    int dev = 0;
    RT_CUDA_OK(cudaGetDevice(&dev));
    if (dev < 0 || dev >= 64) {
        set_error("device index %d out of range", dev);
        return RT_ERR_NO_DEVICE;
    }
    std::lock_guard<std::mutex> lock(g_pipe_mutex);
    HostPipe& p = g_pipe[dev];
    if (!p.ready) {
        RT_CUDA_OK(cudaStreamCreateWithFlags(&p.h2d, cudaStreamNonBlocking));
        RT_CUDA_OK(cudaStreamCreateWithFlags(&p.d2h, cudaStreamNonBlocking));
        for (int i = 0; i < kSlots; ++i) {
            RT_CUDA_OK(cudaEventCreateWithFlags(&p.loaded[i], cudaEventDisableTiming));
            RT_CUDA_OK(cudaEventCreateWithFlags(&p.computed[i], cudaEventDisableTiming));
            RT_CUDA_OK(cudaEventCreateWithFlags(&p.drained[i], cudaEventDisableTiming));
        }
        RT_CUDA_OK(cudaEventCreateWithFlags(&p.start, cudaEventDisableTiming));
        p.ready = true;
    }
    *out = &p;
    return RT_OK;
}

}  // namespace

void host_pipe_shutdown()
{
    std::lock_guard<std::mutex> lock(g_pipe_mutex);
    for (HostPipe& p : g_pipe) {
        if (!p.ready) continue;
        cudaStreamDestroy(p.h2d);
        cudaStreamDestroy(p.d2h);
        for (int i = 0; i < kSlots; ++i) {
            cudaEventDestroy(p.loaded[i]);
            cudaEventDestroy(p.computed[i]);
            cudaEventDestroy(p.drained[i]);
        }
        cudaEventDestroy(p.start);
        p.ready = false;
    }
}

}  // namespace rt

extern "C" {

int64_t rmsnorm_host_workspace_bytes(int64_t n_tokens, int64_t hidden, int dtype, int64_t chunk_tokens)
{
    if (n_tokens < 0 || hidden <= 0 || dtype < 0 || dtype > 2) return -1;
    const int64_t eb = rt::elem_bytes_of(dtype);
    const int64_t chunk = rt::pick_chunk(n_tokens, hidden, dtype, chunk_tokens);
    const int64_t chunk_bytes = rt::round_up(chunk * hidden * eb, rt::kAlign);
    return rt::round_up(hidden * eb, rt::kAlign) + 4 * rt::kSlots * chunk_bytes;
}

int rmsnorm_template_run_host(const rt_params* p, const void* x_host, const void* r_host, const void* w_host,
                              void* y_host, void* r_out_host, int64_t n_tokens, int64_t hidden, float eps, int dtype,
                              void* workspace, int64_t workspace_bytes, int64_t chunk_tokens, void* stream)
{
    if (!p) {
        rt::set_error("params is NULL");
        return RT_ERR_NULL;
    }
    if (dtype < 0 || dtype > 2) {
        rt::set_error("dtype %d unknown", dtype);
        return RT_ERR_DTYPE;
    }
    if (n_tokens < 0 || hidden <= 0) {
        rt::set_error("bad shape");
        return RT_ERR_SHAPE;
    }
    if (n_tokens == 0) return RT_OK;
    if (!x_host || !r_host || !w_host || !y_host || !r_out_host || !workspace) {
        rt::set_error("a buffer pointer is NULL");
        return RT_ERR_NULL;
    }
    const int64_t need = rmsnorm_host_workspace_bytes(n_tokens, hidden, dtype, chunk_tokens);
    if (workspace_bytes < need || ((uintptr_t)workspace & (rt::kAlign - 1))) {
        rt::set_error("workspace of %lld bytes (need %lld, 256-byte aligned)", (long long)workspace_bytes, (long long)need);
        return RT_ERR_CAPACITY;
    }
    rt_limits L;
    int st = rt::current_limits(&L);
    if (st != RT_OK) return st;
    rt::HostPipe* pipe;
    st = rt::get_pipe(&pipe);
    if (st != RT_OK) return st;

    const int64_t eb = rt::elem_bytes_of(dtype);
    const int64_t chunk = rt::pick_chunk(n_tokens, hidden, dtype, chunk_tokens);
    const int64_t chunk_bytes = rt::round_up(chunk * hidden * eb, rt::kAlign);
    char* base = (char*)workspace;
    char* w_dev = base;
    char* slots = base + rt::round_up(hidden * eb, rt::kAlign);
    auto slot_ptr = [&](int slot, int tensor) { return slots + ((int64_t)slot * 4 + tensor) * chunk_bytes; };

    // Plans for a full chunk and for the ragged last chunk (device buffers are 256-byte aligned).
    rt_shape shape;
    memset(&shape, 0, sizeof(shape));
    shape.op = RT_OP_ADD_RMSNORM;
    shape.hidden = hidden;
    shape.dtype = dtype;
    shape.min_ptr_align = 256;
    shape.n_tokens = chunk;
    rt::Plan plan_full, plan_tail;
    st = rt::make_plan(&shape, p, &L, &plan_full);
    if (st != RT_OK) return st;
    const int64_t n_chunks = (n_tokens + chunk - 1) / chunk;
    const int64_t tail_rows = n_tokens - (n_chunks - 1) * chunk;
    shape.n_tokens = tail_rows;
    st = rt::make_plan(&shape, p, &L, &plan_tail);
    if (st != RT_OK) return st;

    cudaStream_t compute = (cudaStream_t)stream;
    // Work queued on the caller's stream before this call stays ordered before ours.
    RT_CUDA_OK(cudaEventRecord(pipe->start, compute));
    RT_CUDA_OK(cudaStreamWaitEvent(pipe->h2d, pipe->start, 0));
    RT_CUDA_OK(cudaStreamWaitEvent(pipe->d2h, pipe->start, 0));
    RT_CUDA_OK(cudaMemcpyAsync(w_dev, w_host, hidden * eb, cudaMemcpyHostToDevice, pipe->h2d));

    for (int64_t c = 0; c < n_chunks; ++c) {
        const int slot = (int)(c % rt::kSlots);
        const int64_t rows = c == n_chunks - 1 ? tail_rows : chunk;
        const int64_t bytes = rows * hidden * eb;
        const int64_t off = c * chunk * hidden * eb;
        // the slot is free once its previous occupant has been copied out
        if (c >= rt::kSlots) RT_CUDA_OK(cudaStreamWaitEvent(pipe->h2d, pipe->drained[slot], 0));
        RT_CUDA_OK(cudaMemcpyAsync(slot_ptr(slot, 0), (const char*)x_host + off, bytes, cudaMemcpyHostToDevice, pipe->h2d));
        RT_CUDA_OK(cudaMemcpyAsync(slot_ptr(slot, 1), (const char*)r_host + off, bytes, cudaMemcpyHostToDevice, pipe->h2d));
        RT_CUDA_OK(cudaEventRecord(pipe->loaded[slot], pipe->h2d));
        RT_CUDA_OK(cudaStreamWaitEvent(compute, pipe->loaded[slot], 0));
        st = rt::launch_plan(c == n_chunks - 1 ? plan_tail : plan_full, slot_ptr(slot, 0), slot_ptr(slot, 1), w_dev,
                             slot_ptr(slot, 2), slot_ptr(slot, 3), rows, hidden, eps, compute);
        if (st != RT_OK) break;
        RT_CUDA_OK(cudaEventRecord(pipe->computed[slot], compute));
        RT_CUDA_OK(cudaStreamWaitEvent(pipe->d2h, pipe->computed[slot], 0));
        RT_CUDA_OK(cudaMemcpyAsync((char*)y_host + off, slot_ptr(slot, 2), bytes, cudaMemcpyDeviceToHost, pipe->d2h));
        RT_CUDA_OK(cudaMemcpyAsync((char*)r_out_host + off, slot_ptr(slot, 3), bytes, cudaMemcpyDeviceToHost, pipe->d2h));
        RT_CUDA_OK(cudaEventRecord(pipe->drained[slot], pipe->d2h));
    }
    cudaError_t e1 = cudaStreamSynchronize(pipe->h2d);
    cudaError_t e2 = cudaStreamSynchronize(compute);
    cudaError_t e3 = cudaStreamSynchronize(pipe->d2h);
    if (st != RT_OK) return st;
    if (e1 != cudaSuccess || e2 != cudaSuccess || e3 != cudaSuccess) {
        rt::set_error("pipeline failed: %s", cudaGetErrorString(e1 != cudaSuccess ? e1 : (e2 != cudaSuccess ? e2 : e3)));
        return RT_ERR_CUDA;
    }
    return RT_OK;
}

}  // extern "C"
