// Instrumented instances of the norm template: the same kernel body with TRACE = true, which stamps SM cycle counts at
// its phase boundaries (entry, released by the previous kernel, inputs arrived, row reduced, outputs issued).  Built for
// the latency-bound shapes, where the time of a launch is a chain of latencies rather than a byte count, so that each
// link can be put beside the hardware figure it should equal.  A measurement aid ("Performance Measurement" in the
// paper times whole kernels only); the instances are few and are not part of the tuner's candidate set.
#include "add_rmsnorm_kernel.cuh"
#include "tuner_internal.h"

namespace rt {
namespace {

struct TraceEntry {
    int dtype, vec_bytes, stage, reduce, unroll, cap;
    const void* fn;
};

#define RT_TRACE_ENTRY(T, DT, VB, ST, RD, U, CAP) \
    TraceEntry{DT, VB, ST, RD, U, (ST) == kStageReg ? (CAP) : 0, (const void*)&add_rmsnorm_kernel<T, VB, ST, RD, U, CAP, true>}

// bf16 and fp32, 16-byte vectors, unroll 1: the register stage with one and two vectors per thread under each
// reduction, and the one-row TMA stage.
const TraceEntry kTraceEntries[] = {
    RT_TRACE_ENTRY(__nv_bfloat16, RT_BF16, 16, kStageReg, kReduceShfl, 1, 1),
    RT_TRACE_ENTRY(__nv_bfloat16, RT_BF16, 16, kStageReg, kReduceShfl, 1, 2),
    RT_TRACE_ENTRY(__nv_bfloat16, RT_BF16, 16, kStageReg, kReduceSmem, 1, 1),
    RT_TRACE_ENTRY(__nv_bfloat16, RT_BF16, 16, kStageReg, kReduceCluster, 1, 1),
    RT_TRACE_ENTRY(__nv_bfloat16, RT_BF16, 16, kStageSmemTma, kReduceShfl, 1, 1),
    RT_TRACE_ENTRY(float, RT_FP32, 16, kStageReg, kReduceShfl, 1, 1),
    RT_TRACE_ENTRY(float, RT_FP32, 16, kStageReg, kReduceShfl, 1, 2),
};

}  // namespace
}  // namespace rt

extern "C" {

int64_t rmsnorm_trace_words(const rt_params* p, int64_t n_tokens, int64_t hidden, int dtype)
{
    if (!p) return -1;
    rt_limits L;
    if (rt::current_limits(&L) != RT_OK) return -1;
    rt_shape s = {};
    s.n_tokens = n_tokens;
    s.hidden = hidden;
    s.dtype = dtype;
    s.min_ptr_align = 256;
    rt::Plan plan;
    if (rt::make_plan(&s, p, &L, &plan) != RT_OK) return -1;
    return (int64_t)plan.grid_x * rt::kTraceWords;
}

int rmsnorm_template_launch_traced(const rt_params* p, const void* x, const void* r, const void* w, void* y, void* r_out,
                                   int64_t n_tokens, int64_t hidden, float eps, int dtype, uint64_t* trace,
                                   int64_t trace_words, void* stream)
{
    if (!p || !trace) {
        rt::set_error("params or trace is NULL");
        return RT_ERR_NULL;
    }
    if (n_tokens > 0 && (!x || !r || !w || !y || !r_out)) {
        rt::set_error("a tensor pointer is NULL");
        return RT_ERR_NULL;
    }
    if ((uintptr_t)trace & 7u) {
        rt::set_error("trace must be 8-byte aligned");
        return RT_ERR_ALIGN;
    }
    rt_limits L;
    int st = rt::current_limits(&L);
    if (st != RT_OK) return st;
    rt_shape s = {};
    s.n_tokens = n_tokens;
    s.hidden = hidden;
    s.dtype = dtype;
    s.min_ptr_align = n_tokens > 0 ? rt::min_pointer_alignment(x, r, w, y, r_out) : 256;
    rt::Plan plan;
    st = rt::make_plan(&s, p, &L, &plan);
    if (st != RT_OK) return st;
    if (trace_words < (int64_t)plan.grid_x * rt::kTraceWords) {
        rt::set_error("trace holds %lld words, the launch's %u CTAs need %lld", (long long)trace_words, plan.grid_x,
                      (long long)plan.grid_x * rt::kTraceWords);
        return RT_ERR_CAPACITY;
    }
    const void* fn = nullptr;
    for (const rt::TraceEntry& e : rt::kTraceEntries)
        if (e.dtype == dtype && e.vec_bytes == p->vec_bytes && e.stage == p->stage && e.reduce == p->reduce &&
            e.unroll == plan.unroll_eff && e.cap == plan.cap)
            fn = e.fn;
    if (!fn) {
        rt::set_error("no instrumented instance for dtype=%d vec=%d stage=%d reduce=%d unroll=%d vectors per thread=%d",
                      dtype, p->vec_bytes, p->stage, p->reduce, plan.unroll_eff, plan.cap);
        return RT_ERR_INFEASIBLE;
    }
    return rt::launch_plan_as(plan, fn, (unsigned long long*)trace, x, r, w, y, r_out, n_tokens, hidden, eps,
                              (cudaStream_t)stream);
}

}  // extern "C"
