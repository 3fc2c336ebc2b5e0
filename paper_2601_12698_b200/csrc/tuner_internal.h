// Internal declarations shared by the host-side translation units of the library.
#pragma once

#include <cuda_runtime.h>
#include <stdint.h>

#include <algorithm>
#include <vector>

#include "rmsnorm_tuner.h"

namespace rt {

// One compiled instance of the kernel template.
struct KernelEntry {
    int op;
    int dtype, vec_bytes, stage, reduce, unroll, cap;  // cap: per-thread row vectors (register stage), else 0
    const void* fn;
    int parts = 0;  // all-reduce-fused norm: partial inputs summed per element
};
struct KernelSlice {
    const KernelEntry* entries;
    int n;
};

// What the compiler and the runtime say about one instance on the current device.
struct KernelInfo {
    int regs_per_thread;
    int local_bytes;   // > 0: the instance spills
    int static_smem;
    int max_threads;   // largest block the instance can be launched with
};

// theta turned into launch geometry; produced only when every hard rule holds.
struct Plan {
    int op;
    int kernel_index;
    int elem_bytes;
    int nvec;         // vectors per row
    int slice_nvec;   // vectors per row per CTA
    int vec_per_thread;
    int cap;          // register-stage capacity actually instantiated (0 otherwise)
    int unroll_eff;
    int vec_per_head; // merge_attn_states: vectors in one head
    int heads;
    int cluster;      // CTAs per row
    int blocks_per_cta;  // pipeline stage: row blocks the busiest CTA of the persistent grid walks over (else 0)
    int block_x, block_y;
    unsigned grid_x;
    size_t dyn_smem;
    size_t static_smem_estimate;
    int reject_reason;  // RejectReason when make_plan fails
};

enum RejectReason { kRejectNone = 0, kRejectArgs = 1, kRejectThreads = 2, kRejectAlign = 3, kRejectRegisters = 4,
                    kRejectSmem = 5, kRejectCluster = 6, kRejectGrid = 7, kRejectReasons = 8 };

void set_error(const char* fmt, ...);
const char* last_error();

inline int elem_bytes_of(int dtype) { return dtype == RT_FP32 ? 4 : 2; }

const std::vector<KernelEntry>& registry();
int find_kernel(int op, int dtype, int vec_bytes, int stage, int reduce, int unroll, int cap, int parts = 0);
// Cached cudaFuncGetAttributes of instance `index` on the current device.
int kernel_info(int index, KernelInfo* out);

// Hard feasibility rules.  limits->have_device selects measured kernel attributes over the model.
int make_plan(const rt_shape* s, const rt_params* p, const rt_limits* limits, Plan* plan);
// Resident CTAs per SM for a plan (runtime query with a device, closed-form model without).
int plan_occupancy(const Plan& plan, const rt_limits* limits, int* regs_per_thread);
// Cached limits of the current device.
int current_limits(rt_limits* out);

int launch_plan(const Plan& plan, const void* x, const void* r, const void* w, void* y, void* r_out,
                int64_t n_tokens, int64_t hidden, float eps, cudaStream_t stream);
int launch_plan_as(const Plan& plan, const void* fn, unsigned long long* trace, const void* x, const void* r, const void* w,
                   void* y, void* r_out, int64_t n_tokens, int64_t hidden, float eps, cudaStream_t stream);
int launch_fp8_plan(const Plan& plan, const void* x, const void* r, const void* w, void* q, float* scale, void* r_out,
                    int64_t n_tokens, int64_t hidden, float eps, cudaStream_t stream);
int launch_allreduce_plan(const Plan& plan, const void* const* x_parts, int n_parts, const void* r, const void* w,
                          void* const* y_outs, int n_y_outs, void* const* r_outs, int n_r_outs, int64_t row_begin,
                          int64_t row_count, int64_t hidden, float eps, cudaStream_t stream);
int launch_merge_plan(const Plan& plan, const void* v_a, const float* s_a, const void* v_b, const float* s_b, void* v_out,
                      float* s_out, int64_t n_tokens, cudaStream_t stream);
int launch_silu_plan(const Plan& plan, const void* x, void* out, int64_t n_tokens, cudaStream_t stream);
int ensure_dynamic_smem(int index, size_t bytes);
int* device_status_word();
void host_pipe_shutdown();  // streams and events of the host-buffer pipeline
void count_launch(int64_t n = 1);

// Raw grid and feasible set (feasible.cu).  counts, when given, has kRejectReasons + 3 entries:
// [0..7] hard rejections by reason, [8] heuristic rejections, [9] feasible, [10] raw.
std::vector<rt_params> raw_grid(const rt_shape& s);
int derive_feasible(const rt_shape& s, const rt_limits& limits, int heuristics, std::vector<rt_params>* out,
                    int32_t* counts);
uint64_t pack_params(const rt_params& p);

int min_pointer_alignment(const void* a, const void* b, const void* c, const void* d, const void* e);

}  // namespace rt

#define RT_CUDA_OK(call)                                                                       \
    do {                                                                                       \
        cudaError_t rt_e_ = (call);                                                            \
        if (rt_e_ != cudaSuccess) {                                                            \
            rt::set_error("%s failed: %s", #call, cudaGetErrorString(rt_e_));                  \
            return RT_ERR_CUDA;                                                                \
        }                                                                                      \
    } while (0)
