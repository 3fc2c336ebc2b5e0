// Instance registry, resource limits r(h), the hard feasibility rules and the launch path.
#include <cuda_runtime.h>
#include <stdarg.h>
#include <stdio.h>
#include <string.h>

#include <atomic>
#include <mutex>
#include <unordered_map>

#include "add_rmsnorm_allreduce_kernel.cuh"
#include "add_rmsnorm_fp8_kernel.cuh"
#include "add_rmsnorm_kernel.cuh"
#include "merge_attn_states_kernel.cuh"
#include "silu_and_mul_kernel.cuh"
#include "tuner_internal.h"

// Each instantiation unit exports its slice of the instance table.
#define RT_DECLARE_SLICE(name) rt::KernelSlice rt_kernel_slice_##name();
#include "instance_units.inc"
#undef RT_DECLARE_SLICE

namespace rt {

static_assert(kMaxParts == RT_MAX_PARTS, "the kernel's argument arrays hold RT_MAX_PARTS pointers");

__device__ int g_status_word = 0;

namespace {

thread_local char tls_error[512] = "";
std::atomic<int64_t> g_launches{0};
std::atomic<int> g_programmatic_launch{1};
std::atomic<int> g_wait_polls{(int)kMbarrierPollLimit};
std::atomic<int> g_drop_tma_copies{0};
std::mutex g_mutex;

constexpr int kMaxDevices = 64;
struct DeviceCache {
    bool limits_ready = false;
    rt_limits limits;
    int* status_ptr = nullptr;
    std::vector<KernelInfo> info;       // per instance
    std::vector<char> info_ready;
    std::vector<size_t> dyn_smem_set;   // largest dynamic shared memory opted in so far
    std::unordered_map<uint64_t, int> occupancy;  // (instance, threads, dynamic shared memory) -> resident CTAs per SM
};
DeviceCache g_dev[kMaxDevices];

uint64_t key_of(int op, int dtype, int vb, int stage, int reduce, int unroll, int cap, int parts = 0)
{
    return ((uint64_t)parts << 56) | ((uint64_t)op << 48) | ((uint64_t)dtype << 40) | ((uint64_t)vb << 32) | ((uint64_t)stage << 28) | ((uint64_t)reduce << 24) |
           ((uint64_t)unroll << 16) | (uint64_t)cap;
}

struct Registry {
    std::vector<KernelEntry> entries;
    std::unordered_map<uint64_t, int> index;
    Registry()
    {
#define RT_DECLARE_SLICE(name)                                             \
    {                                                                      \
        KernelSlice s = rt_kernel_slice_##name();                          \
        for (int i = 0; i < s.n; ++i) entries.push_back(s.entries[i]);     \
    }
#include "instance_units.inc"
#undef RT_DECLARE_SLICE
        for (int i = 0; i < (int)entries.size(); ++i) {
            const KernelEntry& e = entries[i];
            index[key_of(e.op, e.dtype, e.vec_bytes, e.stage, e.reduce, e.unroll, e.cap, e.parts)] = i;
        }
    }
};
Registry& reg()
{
    static Registry r;
    return r;
}

int current_device_cache(DeviceCache** out)
{
    int dev = -1;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess || dev < 0 || dev >= kMaxDevices) {
        (void)cudaGetLastError();
        set_error("no usable CUDA device (%s)", e == cudaSuccess ? "device index out of range" : cudaGetErrorString(e));
        return RT_ERR_NO_DEVICE;
    }
    *out = &g_dev[dev];
    return RT_OK;
}

int next_pow2(int v)
{
    int p = 1;
    while (p < v) p <<= 1;
    return p;
}
bool is_pow2(int v) { return v > 0 && (v & (v - 1)) == 0; }

}  // namespace

void set_error(const char* fmt, ...)
{
    va_list ap;
    va_start(ap, fmt);
    vsnprintf(tls_error, sizeof(tls_error), fmt, ap);
    va_end(ap);
}
const char* last_error() { return tls_error; }
void count_launch(int64_t n) { g_launches.fetch_add(n, std::memory_order_relaxed); }

const std::vector<KernelEntry>& registry() { return reg().entries; }

int find_kernel(int op, int dtype, int vb, int stage, int reduce, int unroll, int cap, int parts)
{
    auto it = reg().index.find(key_of(op, dtype, vb, stage, reduce, unroll, cap, parts));
    return it == reg().index.end() ? -1 : it->second;
}

int current_limits(rt_limits* out)
{
    DeviceCache* dc;
    int st = current_device_cache(&dc);
    if (st != RT_OK) return st;
    std::lock_guard<std::mutex> lock(g_mutex);
    if (!dc->limits_ready) {
        int dev = 0;
        RT_CUDA_OK(cudaGetDevice(&dev));
        cudaDeviceProp prop;
        RT_CUDA_OK(cudaGetDeviceProperties(&prop, dev));
        rt_limits& l = dc->limits;
        memset(&l, 0, sizeof(l));
        l.sm_count = prop.multiProcessorCount;
        l.warp_size = prop.warpSize;
        l.max_threads_per_block = prop.maxThreadsPerBlock;
        l.max_threads_per_sm = prop.maxThreadsPerMultiProcessor;
        l.max_blocks_per_sm = prop.maxBlocksPerMultiProcessor;
        l.regs_per_block = prop.regsPerBlock;
        l.regs_per_sm = prop.regsPerMultiprocessor;
        l.max_regs_per_thread = 255;
        l.max_cluster_size = prop.major >= 9 ? 8 : 1;  // portable cluster size
        l.have_device = 1;
        l.smem_per_block_optin = (int64_t)prop.sharedMemPerBlockOptin;
        l.smem_per_sm = (int64_t)prop.sharedMemPerMultiprocessor;
        l.smem_reserved_per_block = (int64_t)prop.reservedSharedMemPerBlock;
        l.l2_bytes = (int64_t)prop.l2CacheSize;
        dc->limits_ready = true;
    }
    *out = dc->limits;
    return RT_OK;
}

int kernel_info(int index, KernelInfo* out)
{
    DeviceCache* dc;
    int st = current_device_cache(&dc);
    if (st != RT_OK) return st;
    std::lock_guard<std::mutex> lock(g_mutex);
    const size_t n = reg().entries.size();
    if (dc->info.size() != n) {
        dc->info.assign(n, KernelInfo{});
        dc->info_ready.assign(n, 0);
        dc->dyn_smem_set.assign(n, 48 * 1024);
    }
    if (!dc->info_ready[index]) {
        cudaFuncAttributes fa;
        RT_CUDA_OK(cudaFuncGetAttributes(&fa, reg().entries[index].fn));
        KernelInfo& k = dc->info[index];
        k.regs_per_thread = fa.numRegs;
        k.local_bytes = (int)fa.localSizeBytes;
        k.static_smem = (int)fa.sharedSizeBytes;
        k.max_threads = fa.maxThreadsPerBlock;
        dc->info_ready[index] = 1;
    }
    *out = dc->info[index];
    return RT_OK;
}

// Kernels that need more than 48 KB of dynamic shared memory must opt in.  The opt-in is made once per
// instance and device, to the largest size the device allows, so that occupancy queries and launches
// see one fixed setting whatever order they come in.
int ensure_dynamic_smem(int index, size_t bytes)
{
    if (bytes <= 48 * 1024) return RT_OK;
    KernelInfo ki;
    int st = kernel_info(index, &ki);  // also sizes the per-device tables
    if (st != RT_OK) return st;
    rt_limits L;
    st = current_limits(&L);
    if (st != RT_OK) return st;
    DeviceCache* dc;
    st = current_device_cache(&dc);
    if (st != RT_OK) return st;
    std::lock_guard<std::mutex> lock(g_mutex);
    if (dc->dyn_smem_set[index] < bytes) {
        const size_t most = (size_t)L.smem_per_block_optin - (size_t)ki.static_smem;
        if (bytes > most) {
            set_error("%zu bytes of dynamic shared memory exceed the %zu this instance may opt in to", bytes, most);
            return RT_ERR_INFEASIBLE;
        }
        RT_CUDA_OK(cudaFuncSetAttribute(reg().entries[index].fn, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)most));
        dc->dyn_smem_set[index] = most;
    }
    return RT_OK;
}

int* device_status_word()
{
    DeviceCache* dc;
    if (current_device_cache(&dc) != RT_OK) return nullptr;
    std::lock_guard<std::mutex> lock(g_mutex);
    if (!dc->status_ptr) {
        void* p = nullptr;
        if (cudaGetSymbolAddress(&p, g_status_word) != cudaSuccess) {
            set_error("cudaGetSymbolAddress(status word) failed: %s", cudaGetErrorString(cudaGetLastError()));
            return nullptr;
        }
        dc->status_ptr = (int*)p;
    }
    return dc->status_ptr;
}

int min_pointer_alignment(const void* a, const void* b, const void* c, const void* d, const void* e)
{
    const uintptr_t bits = (uintptr_t)a | (uintptr_t)b | (uintptr_t)c | (uintptr_t)d | (uintptr_t)e | 256u;
    return (int)(bits & (~bits + 1));
}

// Registers per thread, static shared memory and spill size of every instance as ptxas reported them for
// this compilation of the library (table generated by the build script).  Used when no device can be asked; with a device the
// runtime's own figures are used instead.
struct InstanceResources {
    int op, dtype, vec_bytes, stage, reduce, unroll, cap, regs, static_smem, spill_bytes, parts;
};
static const InstanceResources kInstanceResources[] = {
#include "instance_resources.inc"
};
static const InstanceResources* build_resources(const KernelEntry& k)
{
    static std::unordered_map<uint64_t, const InstanceResources*> index = [] {
        std::unordered_map<uint64_t, const InstanceResources*> m;
        for (const InstanceResources& r : kInstanceResources)
            m[key_of(r.op, r.dtype, r.vec_bytes, r.stage, r.reduce, r.unroll, r.cap, r.parts)] = &r;
        return m;
    }();
    auto it = index.find(key_of(k.op, k.dtype, k.vec_bytes, k.stage, k.reduce, k.unroll, k.cap, k.parts));
    return it == index.end() ? nullptr : it->second;
}
static int model_regs(const KernelEntry& k, int elem_bytes)
{
    (void)elem_bytes;
    const InstanceResources* r = build_resources(k);
    return r ? r->regs : 255;
}
static int model_static_smem(const KernelEntry& k)
{
    const InstanceResources* r = build_resources(k);
    return r ? r->static_smem : 8192;
}
static int model_spill(const KernelEntry& k)
{
    const InstanceResources* r = build_resources(k);
    return r ? r->spill_bytes : 0;
}

int make_plan(const rt_shape* s, const rt_params* p, const rt_limits* L, Plan* plan)
{
    if (!s || !p || !L || !plan) {
        set_error("make_plan: NULL argument");
        return RT_ERR_NULL;
    }
    memset(plan, 0, sizeof(*plan));
    if (s->dtype < 0 || s->dtype > 2) {
        set_error("dtype %d is not one of bf16(0), fp16(1), fp32(2)", s->dtype);
        plan->reject_reason = kRejectArgs;
        return RT_ERR_DTYPE;
    }
    if (s->op < RT_OP_ADD_RMSNORM || s->op > RT_OP_ADD_RMSNORM_ALLREDUCE) {
        set_error("op %d is not a kernel of this library", s->op);
        plan->reject_reason = kRejectArgs;
        return RT_ERR_SHAPE;
    }
    plan->op = s->op;
    const bool is_silu = s->op == RT_OP_SILU_AND_MUL;
    const bool is_merge = s->op == RT_OP_MERGE_ATTN_STATES;
    const bool no_reduction = is_silu || is_merge;  // element-wise kernels: no reduction axis, no CAP
    const bool is_fp8 = s->op == RT_OP_ADD_RMSNORM_FP8;
    const bool is_allreduce = s->op == RT_OP_ADD_RMSNORM_ALLREDUCE;
    const int eb = elem_bytes_of(s->dtype);
    if (s->n_tokens < 0 || s->hidden <= 0 || s->hidden * eb * (is_silu ? 2 : 1) >= (int64_t)1 << 31) {
        set_error("shape n_tokens=%lld hidden=%lld is out of range", (long long)s->n_tokens, (long long)s->hidden);
        plan->reject_reason = kRejectArgs;
        return RT_ERR_SHAPE;
    }
    const int tpr = p->threads_per_row, rpc = p->rows_per_cta, vb = p->vec_bytes;
    if (!is_pow2(tpr) || tpr < L->warp_size || tpr > 1024) {
        set_error("threads_per_row=%d must be a power of two between the warp size and 1024", tpr);
        plan->reject_reason = kRejectThreads;
        return RT_ERR_INFEASIBLE;
    }
    if (rpc < 1 || rpc > kMaxRowsPerCta) {
        set_error("rows_per_cta=%d outside 1..%d", rpc, kMaxRowsPerCta);
        plan->reject_reason = kRejectThreads;
        return RT_ERR_INFEASIBLE;
    }
    if (tpr * rpc > L->max_threads_per_block) {
        set_error("block of %d x %d threads exceeds the %d threads a CTA may have", tpr, rpc, L->max_threads_per_block);
        plan->reject_reason = kRejectThreads;
        return RT_ERR_INFEASIBLE;
    }
    if (!(vb == 32 || vb == 16 || vb == 8 || vb == 4 || vb == 2) || vb < eb) {
        set_error("vec_bytes=%d is not 32, 16, 8, 4 or 2, or is narrower than one element", vb);
        plan->reject_reason = kRejectArgs;
        return RT_ERR_INFEASIBLE;
    }
    if (!(p->unroll == 1 || p->unroll == 2 || p->unroll == 4)) {
        set_error("unroll=%d is not 1, 2 or 4", p->unroll);
        plan->reject_reason = kRejectArgs;
        return RT_ERR_INFEASIBLE;
    }
    if (p->stage < 0 || p->stage > RT_STAGE_TMA_PIPELINE || p->reduce < 0 || p->reduce > 2) {
        set_error("stage=%d or reduce=%d unknown", p->stage, p->reduce);
        plan->reject_reason = kRejectArgs;
        return RT_ERR_INFEASIBLE;
    }
    const bool realign = p->stage == RT_STAGE_REG_REALIGN;
    if (realign && (s->op != RT_OP_ADD_RMSNORM || (p->vec_bytes != 16 && p->vec_bytes != 32) || p->reduce != RT_REDUCE_SHFL ||
                    p->cluster_size != 1)) {
        set_error("the ragged-row stage belongs to add_rmsnorm and takes 16- or 32-byte chunks and the shuffle reduction "
                  "(op=%d vec=%d reduce=%d cluster=%d)", s->op, p->vec_bytes, p->reduce, p->cluster_size);
        plan->reject_reason = kRejectArgs;
        return RT_ERR_INFEASIBLE;
    }
    const bool pipeline = p->stage == RT_STAGE_TMA_PIPELINE;
    if (pipeline && (s->op != RT_OP_ADD_RMSNORM || p->reduce == RT_REDUCE_CLUSTER || p->cluster_size != 1)) {
        set_error("the pipeline stage belongs to add_rmsnorm and keeps a row inside one CTA (op=%d reduce=%d cluster=%d)",
                  s->op, p->reduce, p->cluster_size);
        plan->reject_reason = kRejectArgs;
        return RT_ERR_INFEASIBLE;
    }
    if (is_merge && (s->head_dim <= 0 || s->hidden % s->head_dim != 0)) {
        set_error("head_dim=%d does not divide hidden=%lld", s->head_dim, (long long)s->hidden);
        plan->reject_reason = kRejectArgs;
        return RT_ERR_SHAPE;
    }
    if (is_fp8 && (s->dtype == RT_FP32 || p->vec_bytes < 16 || p->reduce != RT_REDUCE_SHFL || p->cluster_size != 1 ||
                   p->stage == RT_STAGE_SMEM_LDG)) {
        set_error("the fp8-output norm takes bf16/fp16, 32- or 16-byte vectors, the shuffle reduction and the register or TMA "
                  "stage (dtype=%d vec=%d reduce=%d cluster=%d stage=%d)", s->dtype, p->vec_bytes, p->reduce,
                  p->cluster_size, p->stage);
        plan->reject_reason = kRejectArgs;
        return s->dtype == RT_FP32 ? RT_ERR_DTYPE : RT_ERR_INFEASIBLE;
    }
    if (is_allreduce && !(s->n_parts == 2 || s->n_parts == 4 || s->n_parts == 8)) {
        set_error("n_parts=%d is not 2, 4 or 8", s->n_parts);
        plan->reject_reason = kRejectArgs;
        return RT_ERR_SHAPE;
    }
    if (is_allreduce && (p->vec_bytes < 16 || p->reduce != RT_REDUCE_SHFL || p->cluster_size != 1 || p->stage != RT_STAGE_REG)) {
        set_error("the all-reduce-fused norm takes 32- or 16-byte vectors, the shuffle reduction and the register stage "
                  "(vec=%d reduce=%d cluster=%d stage=%d)", p->vec_bytes, p->reduce, p->cluster_size, p->stage);
        plan->reject_reason = kRejectArgs;
        return RT_ERR_INFEASIBLE;
    }
    if (no_reduction && (p->reduce != RT_REDUCE_SHFL || p->cluster_size != 1 || p->stage == RT_STAGE_SMEM_LDG)) {
        set_error("this kernel has no reduction and no ld.global->shared stage (reduce=%d cluster=%d stage=%d)",
                  p->reduce, p->cluster_size, p->stage);
        plan->reject_reason = kRejectArgs;
        return RT_ERR_INFEASIBLE;
    }
    const int C = p->cluster_size;
    if (p->reduce == RT_REDUCE_CLUSTER) {
        if (!(C == 2 || C == 4 || C == 8) || C > L->max_cluster_size) {
            set_error("cluster_size=%d is not 2, 4 or 8 within the device's limit of %d", C, L->max_cluster_size);
            plan->reject_reason = kRejectCluster;
        return RT_ERR_INFEASIBLE;
        }
    } else if (C != 1) {
        set_error("cluster_size=%d without the cluster reduction", C);
        plan->reject_reason = kRejectCluster;
        return RT_ERR_INFEASIBLE;
    }
    const int64_t row_bytes = s->hidden * eb;
    if (row_bytes % vb != 0 && !realign) {  // the ragged-row stage covers a row of any length with aligned chunks
        set_error("row of %lld bytes is not a multiple of vec_bytes=%d", (long long)row_bytes, vb);
        plan->reject_reason = kRejectAlign;
        return RT_ERR_ALIGN;
    }
    if (is_merge && ((int64_t)s->head_dim * eb) % vb != 0) {
        set_error("a head of %d bytes is not a multiple of vec_bytes=%d", s->head_dim * eb, vb);
        plan->reject_reason = kRejectAlign;
        return RT_ERR_ALIGN;
    }
    if (s->min_ptr_align < vb) {
        set_error("a base pointer is only %d-byte aligned, vec_bytes=%d", s->min_ptr_align, vb);
        plan->reject_reason = kRejectAlign;
        return RT_ERR_ALIGN;
    }
    // silu_and_mul: an input row is 2 * row_bytes long, so 16-byte output rows give 16-byte input rows
    if ((p->stage == RT_STAGE_SMEM_TMA || pipeline) && (row_bytes % 16 != 0 || s->min_ptr_align < 16)) {
        set_error("TMA bulk copies need 16-byte aligned rows and pointers (row %lld bytes, pointers %d)",
                  (long long)row_bytes, s->min_ptr_align);
        plan->reject_reason = kRejectAlign;
        return RT_ERR_ALIGN;
    }

    plan->elem_bytes = eb;
    // ragged rows: the most whole chunks a row can hold (its head and tail elements go one to a thread)
    plan->nvec = realign ? (int)std::max<int64_t>(1, row_bytes / vb) : (int)(row_bytes / vb);
    int slice = (plan->nvec + C - 1) / C;
    const int gran = vb < 16 ? 16 / vb : 1;  // slices start on 16-byte boundaries
    slice = (slice + gran - 1) / gran * gran;
    plan->slice_nvec = slice;
    plan->vec_per_thread = (slice + tpr - 1) / tpr;
    plan->cluster = C;
    if (is_merge) {
        plan->vec_per_head = (int)((int64_t)s->head_dim * eb / vb);
        plan->heads = (int)(s->hidden / s->head_dim);
    }
    plan->block_x = tpr;
    plan->block_y = rpc;
    if ((int64_t)(C - 1) * slice >= plan->nvec && C > 1) {
        set_error("a cluster of %d leaves a CTA without any part of the %d-vector row", C, plan->nvec);
        plan->reject_reason = kRejectCluster;
        return RT_ERR_INFEASIBLE;
    }

    int cap = 0, unroll = p->unroll;
    const bool row_in_registers = (p->stage == RT_STAGE_REG || realign) && !no_reduction;
    if (row_in_registers) {
        cap = next_pow2(plan->vec_per_thread);
        if (unroll > cap) unroll = cap;
    }
    plan->cap = cap;
    plan->unroll_eff = unroll;
    plan->kernel_index = find_kernel(s->op, s->dtype, vb, p->stage, p->reduce, unroll, cap, is_allreduce ? s->n_parts : 0);
    if (plan->kernel_index < 0) {
        if (row_in_registers)
            set_error("a row slice of %d vectors over %d threads needs %d vectors per thread: no register-stage "
                      "instance that large (register budget)", slice, tpr, cap);
        else
            set_error("no compiled instance for dtype=%d vec=%d stage=%d reduce=%d unroll=%d", s->dtype, vb, p->stage,
                      p->reduce, unroll);
        plan->reject_reason = row_in_registers ? kRejectRegisters : kRejectArgs;
        return RT_ERR_INFEASIBLE;
    }
    const KernelEntry& k = registry()[plan->kernel_index];

    if (p->stage == RT_STAGE_SMEM_LDG)
        plan->dyn_smem = (size_t)rpc * slice * (vb / eb) * 4;
    else if (p->stage == RT_STAGE_SMEM_TMA)
        plan->dyn_smem = (size_t)rpc * 2 * slice * vb;
    else if (pipeline)
        plan->dyn_smem = (size_t)p->unroll * rpc * 2 * slice * vb;  // a ring of `unroll` stages per row slot

    int regs, static_smem, local_bytes = 0, max_threads = L->max_threads_per_block;
    if (L->have_device) {
        KernelInfo ki;
        int st = kernel_info(plan->kernel_index, &ki);
        if (st != RT_OK) return st;
        regs = ki.regs_per_thread;
        static_smem = ki.static_smem;
        local_bytes = ki.local_bytes;
        max_threads = ki.max_threads;
    } else {
        regs = model_regs(k, eb);
        static_smem = model_static_smem(k);
        local_bytes = model_spill(k);
    }
    plan->static_smem_estimate = (size_t)static_smem;
    if (regs > L->max_regs_per_thread || local_bytes > 0) {
        set_error("instance needs %d registers per thread and spills %d bytes", regs, local_bytes);
        plan->reject_reason = kRejectRegisters;
        return RT_ERR_INFEASIBLE;
    }
    const int threads = tpr * rpc;
    // registers are allocated per warp in units of 8 per thread
    const int regs_alloc = (regs + 7) / 8 * 8;
    if ((int64_t)regs_alloc * threads > L->regs_per_block || threads > max_threads) {
        set_error("%d threads x %d registers exceed the %d registers of a CTA", threads, regs_alloc, L->regs_per_block);
        plan->reject_reason = kRejectRegisters;
        return RT_ERR_INFEASIBLE;
    }
    if ((int64_t)plan->dyn_smem + static_smem > L->smem_per_block_optin) {
        set_error("%zu + %d bytes of shared memory exceed the %lld a CTA may opt in to", plan->dyn_smem, static_smem,
                  (long long)L->smem_per_block_optin);
        plan->reject_reason = kRejectSmem;
        return RT_ERR_INFEASIBLE;
    }
    const int64_t row_blocks = (s->n_tokens + rpc - 1) / rpc;
    if (row_blocks * C > 0x7fffffffLL) {
        set_error("grid of %lld CTAs is too large", (long long)(row_blocks * C));
        plan->reject_reason = kRejectGrid;
        return RT_ERR_INFEASIBLE;
    }
    plan->grid_x = (unsigned)(row_blocks * C);
    if (pipeline) {
        // persistent: as many CTAs as stay resident on the device, each walking over row blocks
        const int resident = plan_occupancy(*plan, L, nullptr);
        if (resident < 1) {
            set_error("the pipeline's %zu bytes of shared memory leave no CTA resident", plan->dyn_smem);
            plan->reject_reason = kRejectSmem;
            return RT_ERR_INFEASIBLE;
        }
        const int64_t most = (int64_t)resident * L->sm_count;
        plan->grid_x = (unsigned)std::max<int64_t>(1, std::min<int64_t>(row_blocks, most));
        plan->blocks_per_cta = (int)((row_blocks + plan->grid_x - 1) / plan->grid_x);
    }
    return RT_OK;
}

int plan_occupancy(const Plan& plan, const rt_limits* L, int* regs_per_thread)
{
    const KernelEntry& k = registry()[plan.kernel_index];
    const int threads = plan.block_x * plan.block_y;
    if (L->have_device) {
        KernelInfo ki;
        if (kernel_info(plan.kernel_index, &ki) != RT_OK) return 0;
        if (regs_per_thread) *regs_per_thread = ki.regs_per_thread;
        if (ensure_dynamic_smem(plan.kernel_index, plan.dyn_smem) != RT_OK) {
            (void)cudaGetLastError();
            return 0;
        }
        int blocks = 0;
        const uint64_t occ_key = ((uint64_t)plan.kernel_index << 40) | ((uint64_t)threads << 24) | (uint64_t)(plan.dyn_smem >> 4);
        DeviceCache* dc = nullptr;
        bool cached = false;
        if (plan.cluster == 1 && current_device_cache(&dc) == RT_OK) {
            std::lock_guard<std::mutex> lock(g_mutex);
            auto it = dc->occupancy.find(occ_key);
            if (it != dc->occupancy.end()) {
                blocks = it->second;
                cached = true;
            }
        }
        if (cached) return blocks;
        if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&blocks, k.fn, threads, plan.dyn_smem) != cudaSuccess) {
            (void)cudaGetLastError();
            return 0;
        }
        if (plan.cluster == 1 && dc) {
            std::lock_guard<std::mutex> lock(g_mutex);
            dc->occupancy[occ_key] = blocks;
        }
        if (plan.cluster > 1 && blocks > 0) {
            cudaLaunchConfig_t cfg;
            memset(&cfg, 0, sizeof(cfg));
            cfg.gridDim = dim3((unsigned)plan.cluster, 1, 1);
            cfg.blockDim = dim3(plan.block_x, plan.block_y, 1);
            cfg.dynamicSmemBytes = plan.dyn_smem;
            cudaLaunchAttribute attr;
            attr.id = cudaLaunchAttributeClusterDimension;
            attr.val.clusterDim.x = plan.cluster;
            attr.val.clusterDim.y = 1;
            attr.val.clusterDim.z = 1;
            cfg.attrs = &attr;
            cfg.numAttrs = 1;
            int clusters = 0;
            if (cudaOccupancyMaxActiveClusters(&clusters, k.fn, &cfg) != cudaSuccess || clusters < 1) {
                (void)cudaGetLastError();
                return 0;
            }
        }
        return blocks;
    }
    const int regs = model_regs(k, plan.elem_bytes);
    if (regs_per_thread) *regs_per_thread = regs;
    const int regs_alloc = (regs + 7) / 8 * 8;
    int64_t blocks = L->max_blocks_per_sm;
    blocks = std::min<int64_t>(blocks, L->max_threads_per_sm / threads);
    blocks = std::min<int64_t>(blocks, L->regs_per_sm / ((int64_t)regs_alloc * threads));
    const int64_t smem = (int64_t)plan.dyn_smem + (int64_t)plan.static_smem_estimate + L->smem_reserved_per_block;
    blocks = std::min<int64_t>(blocks, L->smem_per_sm / smem);
    return (int)blocks;
}

// Launch attributes common to every kernel of the library: the cluster shape, and - unless switched off through
// rt_set_option - programmatic stream serialization (the kernels wait for their predecessor themselves).
struct LaunchAttrs {
    cudaLaunchAttribute a[2];
};
static void set_launch_attrs(cudaLaunchConfig_t* cfg, LaunchAttrs* la, int cluster)
{
    cfg->numAttrs = 0;
    if (cluster > 1) {
        cudaLaunchAttribute& attr = la->a[cfg->numAttrs++];
        attr.id = cudaLaunchAttributeClusterDimension;
        attr.val.clusterDim.x = cluster;
        attr.val.clusterDim.y = 1;
        attr.val.clusterDim.z = 1;
    }
    if (g_programmatic_launch.load(std::memory_order_relaxed)) {
        cudaLaunchAttribute& attr = la->a[cfg->numAttrs++];
        attr.id = cudaLaunchAttributeProgrammaticStreamSerialization;
        attr.val.programmaticStreamSerializationAllowed = 1;
    }
    cfg->attrs = cfg->numAttrs ? la->a : nullptr;
}

int launch_fp8_plan(const Plan& plan, const void* x, const void* r, const void* w, void* q, float* scale, void* r_out,
                    int64_t n_tokens, int64_t hidden, float eps, cudaStream_t stream)
{
    if (n_tokens == 0) return RT_OK;
    if (plan.op != RT_OP_ADD_RMSNORM_FP8) {
        set_error("plan belongs to another kernel");
        return RT_ERR_INFEASIBLE;
    }
    const KernelEntry& k = registry()[plan.kernel_index];
    int st = ensure_dynamic_smem(plan.kernel_index, plan.dyn_smem);
    if (st != RT_OK) return st;
    Fp8Args a;
    a.x = x; a.r = r; a.w = w; a.q = q; a.scale = scale; a.r_out = r_out;
    a.n_tokens = n_tokens;
    a.hidden = (int)hidden;
    a.nvec = plan.nvec;
    a.eps = eps;
    a.status = device_status_word();
    if (!a.status) return RT_ERR_CUDA;
    cudaLaunchConfig_t cfg;
    memset(&cfg, 0, sizeof(cfg));
    cfg.gridDim = dim3(plan.grid_x, 1, 1);
    cfg.blockDim = dim3(plan.block_x, plan.block_y, 1);
    cfg.dynamicSmemBytes = plan.dyn_smem;
    cfg.stream = stream;
    LaunchAttrs la;
    set_launch_attrs(&cfg, &la, 1);
    void* params[] = {&a};
    cudaError_t e = cudaLaunchKernelExC(&cfg, k.fn, params);
    if (e != cudaSuccess) {
        (void)cudaGetLastError();
        set_error("kernel launch failed: %s", cudaGetErrorString(e));
        return RT_ERR_CUDA;
    }
    count_launch();
    return RT_OK;
}

int launch_allreduce_plan(const Plan& plan, const void* const* x_parts, int n_parts, const void* r, const void* w,
                          void* const* y_outs, int n_y_outs, void* const* r_outs, int n_r_outs, int64_t row_begin,
                          int64_t row_count, int64_t hidden, float eps, cudaStream_t stream)
{
    if (row_count == 0) return RT_OK;
    const KernelEntry& k = registry()[plan.kernel_index];
    if (plan.op != RT_OP_ADD_RMSNORM_ALLREDUCE || k.parts != n_parts) {
        set_error("plan belongs to another kernel");
        return RT_ERR_INFEASIBLE;
    }
    if (n_y_outs < 1 || n_y_outs > kMaxParts || n_r_outs < 1 || n_r_outs > kMaxParts) {
        set_error("n_y_outs=%d or n_r_outs=%d outside 1..%d", n_y_outs, n_r_outs, kMaxParts);
        return RT_ERR_SHAPE;
    }
    AllreduceArgs a;
    memset(&a, 0, sizeof(a));
    for (int i = 0; i < n_parts; ++i) a.x_parts[i] = x_parts[i];
    for (int i = 0; i < n_y_outs; ++i) a.y_outs[i] = y_outs[i];
    for (int i = 0; i < n_r_outs; ++i) a.r_outs[i] = r_outs[i];
    a.r = r; a.w = w;
    a.n_y_outs = n_y_outs;
    a.n_r_outs = n_r_outs;
    a.row_begin = row_begin;
    a.row_end = row_begin + row_count;
    a.hidden = (int)hidden;
    a.nvec = plan.nvec;
    a.eps = eps;
    cudaLaunchConfig_t cfg;
    memset(&cfg, 0, sizeof(cfg));
    cfg.gridDim = dim3(plan.grid_x, 1, 1);
    cfg.blockDim = dim3(plan.block_x, plan.block_y, 1);
    cfg.stream = stream;
    LaunchAttrs la;
    set_launch_attrs(&cfg, &la, 1);
    void* params[] = {&a};
    cudaError_t e = cudaLaunchKernelExC(&cfg, k.fn, params);
    if (e != cudaSuccess) {
        (void)cudaGetLastError();
        set_error("kernel launch failed: %s", cudaGetErrorString(e));
        return RT_ERR_CUDA;
    }
    count_launch();
    return RT_OK;
}

int launch_merge_plan(const Plan& plan, const void* v_a, const float* s_a, const void* v_b, const float* s_b, void* v_out,
                      float* s_out, int64_t n_tokens, cudaStream_t stream)
{
    if (n_tokens == 0) return RT_OK;
    if (plan.op != RT_OP_MERGE_ATTN_STATES) {
        set_error("plan belongs to another kernel");
        return RT_ERR_INFEASIBLE;
    }
    const KernelEntry& k = registry()[plan.kernel_index];
    int st = ensure_dynamic_smem(plan.kernel_index, plan.dyn_smem);
    if (st != RT_OK) return st;
    MergeArgs a;
    a.v_a = v_a; a.v_b = v_b; a.s_a = s_a; a.s_b = s_b; a.v_out = v_out; a.s_out = s_out;
    a.n_tokens = n_tokens;
    a.nvec = plan.nvec;
    a.vec_per_head = plan.vec_per_head;
    a.heads = plan.heads;
    a.head_shift = -1;
    for (int sh = 0; sh < 31; ++sh)
        if ((1 << sh) == plan.vec_per_head) a.head_shift = sh;
    a.status = device_status_word();
    if (!a.status) return RT_ERR_CUDA;
    cudaLaunchConfig_t cfg;
    memset(&cfg, 0, sizeof(cfg));
    cfg.gridDim = dim3(plan.grid_x, 1, 1);
    cfg.blockDim = dim3(plan.block_x, plan.block_y, 1);
    cfg.dynamicSmemBytes = plan.dyn_smem;
    cfg.stream = stream;
    LaunchAttrs la;
    set_launch_attrs(&cfg, &la, 1);
    void* params[] = {&a};
    cudaError_t e = cudaLaunchKernelExC(&cfg, k.fn, params);
    if (e != cudaSuccess) {
        (void)cudaGetLastError();
        set_error("kernel launch failed: %s", cudaGetErrorString(e));
        return RT_ERR_CUDA;
    }
    count_launch();
    return RT_OK;
}

int launch_silu_plan(const Plan& plan, const void* x, void* out, int64_t n_tokens, cudaStream_t stream)
{
    if (n_tokens == 0) return RT_OK;
    if (plan.op != RT_OP_SILU_AND_MUL) {
        set_error("plan belongs to another kernel");
        return RT_ERR_INFEASIBLE;
    }
    const KernelEntry& k = registry()[plan.kernel_index];
    int st = ensure_dynamic_smem(plan.kernel_index, plan.dyn_smem);
    if (st != RT_OK) return st;
    SiluArgs a;
    a.x = x;
    a.out = out;
    a.n_tokens = n_tokens;
    a.nvec = plan.nvec;
    a.status = device_status_word();
    if (!a.status) return RT_ERR_CUDA;
    cudaLaunchConfig_t cfg;
    memset(&cfg, 0, sizeof(cfg));
    cfg.gridDim = dim3(plan.grid_x, 1, 1);
    cfg.blockDim = dim3(plan.block_x, plan.block_y, 1);
    cfg.dynamicSmemBytes = plan.dyn_smem;
    cfg.stream = stream;
    LaunchAttrs la;
    set_launch_attrs(&cfg, &la, 1);
    void* params[] = {&a};
    cudaError_t e = cudaLaunchKernelExC(&cfg, k.fn, params);
    if (e != cudaSuccess) {
        (void)cudaGetLastError();
        set_error("kernel launch failed: %s", cudaGetErrorString(e));
        return RT_ERR_CUDA;
    }
    count_launch();
    return RT_OK;
}

int launch_plan(const Plan& plan, const void* x, const void* r, const void* w, void* y, void* r_out,
                int64_t n_tokens, int64_t hidden, float eps, cudaStream_t stream)
{
    return launch_plan_as(plan, nullptr, nullptr, x, r, w, y, r_out, n_tokens, hidden, eps, stream);
}

// The plan's launch with another compiled function of the same template coordinates in place of the registry's
// (`fn` != NULL: an instrumented instance, which also receives `trace`).
int launch_plan_as(const Plan& plan, const void* fn, unsigned long long* trace, const void* x, const void* r, const void* w,
                   void* y, void* r_out, int64_t n_tokens, int64_t hidden, float eps, cudaStream_t stream)
{
    if (n_tokens == 0) return RT_OK;
    if (plan.op != RT_OP_ADD_RMSNORM) {
        set_error("plan belongs to another kernel");
        return RT_ERR_INFEASIBLE;
    }
    const KernelEntry& k = registry()[plan.kernel_index];
    int st = RT_OK;
    if (!fn) {
        st = ensure_dynamic_smem(plan.kernel_index, plan.dyn_smem);
    } else if (plan.dyn_smem > 48 * 1024) {
        set_error("instrumented instances take at most 48 KB of dynamic shared memory");
        st = RT_ERR_INFEASIBLE;
    }
    if (st != RT_OK) return st;
    KernelArgs a;
    a.trace = trace;
    a.x = x; a.r = r; a.w = w; a.y = y; a.r_out = r_out;
    a.n_tokens = n_tokens;
    a.hidden = (int)hidden;
    a.nvec = plan.nvec;
    a.slice_nvec = plan.slice_nvec;
    a.eps = eps;
    a.status = device_status_word();
    if (!a.status) return RT_ERR_CUDA;
    a.wait_polls = (unsigned)g_wait_polls.load(std::memory_order_relaxed);
    a.drop_copies = g_drop_tma_copies.load(std::memory_order_relaxed);

    cudaLaunchConfig_t cfg;
    memset(&cfg, 0, sizeof(cfg));
    cfg.gridDim = dim3(plan.grid_x, 1, 1);
    cfg.blockDim = dim3(plan.block_x, plan.block_y, 1);
    cfg.dynamicSmemBytes = plan.dyn_smem;
    cfg.stream = stream;
    LaunchAttrs la;
    set_launch_attrs(&cfg, &la, plan.cluster);
    void* params[] = {&a};
    cudaError_t e = cudaLaunchKernelExC(&cfg, fn ? fn : k.fn, params);
    if (e != cudaSuccess) {
        (void)cudaGetLastError();
        set_error("kernel launch failed: %s", cudaGetErrorString(e));
        return RT_ERR_CUDA;
    }
    count_launch();
    return RT_OK;
}

}  // namespace rt

// ---- C ABI -------------------------------------------------------------------------------------

extern "C" {

int rmsnorm_template_launch(const rt_params* p, const void* x, const void* r, const void* w, void* y, void* r_out,
                            int64_t n_tokens, int64_t hidden, float eps, int dtype, void* stream)
{
    if (!p) {
        rt::set_error("params is NULL");
        return RT_ERR_NULL;
    }
    if (n_tokens > 0 && (!x || !r || !w || !y || !r_out)) {
        rt::set_error("a tensor pointer is NULL");
        return RT_ERR_NULL;
    }
    rt_limits L;
    int st = rt::current_limits(&L);
    if (st != RT_OK) return st;
    rt_shape s = {};
    s.n_tokens = n_tokens;
    s.hidden = hidden;
    s.dtype = dtype;
    s.min_ptr_align = n_tokens > 0 ? rt::min_pointer_alignment(x, r, w, y, r_out) : 256;
    s.op = RT_OP_ADD_RMSNORM;
    s.head_dim = 0;
    rt::Plan plan;
    st = rt::make_plan(&s, p, &L, &plan);
    if (st != RT_OK) return st;
    return rt::launch_plan(plan, x, r, w, y, r_out, n_tokens, hidden, eps, (cudaStream_t)stream);
}

int silu_and_mul_template_launch(const rt_params* p, const void* x, void* out, int64_t n_tokens, int64_t d, int dtype,
                                 void* stream)
{
    if (!p) {
        rt::set_error("params is NULL");
        return RT_ERR_NULL;
    }
    if (n_tokens > 0 && (!x || !out)) {
        rt::set_error("a tensor pointer is NULL");
        return RT_ERR_NULL;
    }
    rt_limits L;
    int st = rt::current_limits(&L);
    if (st != RT_OK) return st;
    rt_shape s = {};
    s.n_tokens = n_tokens;
    s.hidden = d;
    s.dtype = dtype;
    s.min_ptr_align = n_tokens > 0 ? rt::min_pointer_alignment(x, out, x, out, x) : 256;
    s.op = RT_OP_SILU_AND_MUL;
    s.head_dim = 0;
    rt::Plan plan;
    st = rt::make_plan(&s, p, &L, &plan);
    if (st != RT_OK) return st;
    return rt::launch_silu_plan(plan, x, out, n_tokens, (cudaStream_t)stream);
}

int rmsnorm_fp8_template_launch(const rt_params* p, const void* x, const void* r, const void* w, void* q, float* scale,
                                void* r_out, int64_t n_tokens, int64_t hidden, float eps, int dtype, void* stream)
{
    if (!p) {
        rt::set_error("params is NULL");
        return RT_ERR_NULL;
    }
    if (n_tokens > 0 && (!x || !r || !w || !q || !scale || !r_out)) {
        rt::set_error("a tensor pointer is NULL");
        return RT_ERR_NULL;
    }
    // q leaves as one vector of vec_bytes / 2 bytes per vector of x
    const uintptr_t q_mask = p->vec_bytes == 32 ? 15u : 7u;
    if (n_tokens > 0 && (((uintptr_t)scale & 3u) || ((uintptr_t)q & q_mask))) {
        rt::set_error("scale must be 4-byte and q %d-byte aligned", (int)q_mask + 1);
        return RT_ERR_ALIGN;
    }
    rt_limits L;
    int st = rt::current_limits(&L);
    if (st != RT_OK) return st;
    rt_shape s = {};
    s.n_tokens = n_tokens;
    s.hidden = hidden;
    s.dtype = dtype;
    s.min_ptr_align = n_tokens > 0 ? rt::min_pointer_alignment(x, r, w, r_out, x) : 256;
    s.op = RT_OP_ADD_RMSNORM_FP8;
    s.head_dim = 0;
    rt::Plan plan;
    st = rt::make_plan(&s, p, &L, &plan);
    if (st != RT_OK) return st;
    return rt::launch_fp8_plan(plan, x, r, w, q, scale, r_out, n_tokens, hidden, eps, (cudaStream_t)stream);
}

int rmsnorm_allreduce_template_launch(const rt_params* p, const void* const* x_parts, int32_t n_parts, const void* r,
                                      const void* w, void* const* y_outs, int32_t n_y_outs, void* const* r_outs,
                                      int32_t n_r_outs, int64_t row_begin, int64_t row_count, int64_t hidden, float eps,
                                      int dtype, void* stream)
{
    if (!p) {
        rt::set_error("params is NULL");
        return RT_ERR_NULL;
    }
    if (!(n_parts == 2 || n_parts == 4 || n_parts == 8)) {
        rt::set_error("n_parts=%d is not 2, 4 or 8", n_parts);
        return RT_ERR_SHAPE;
    }
    if (n_y_outs < 1 || n_y_outs > rt::kMaxParts || n_r_outs < 1 || n_r_outs > rt::kMaxParts) {
        rt::set_error("n_y_outs=%d or n_r_outs=%d outside 1..%d", n_y_outs, n_r_outs, rt::kMaxParts);
        return RT_ERR_SHAPE;
    }
    if (row_begin < 0 || row_count < 0) {
        rt::set_error("row_begin=%lld row_count=%lld out of range", (long long)row_begin, (long long)row_count);
        return RT_ERR_SHAPE;
    }
    if (row_count > 0 && (!x_parts || !y_outs || !r_outs || !r || !w)) {
        rt::set_error("a tensor pointer is NULL");
        return RT_ERR_NULL;
    }
    uintptr_t bits = (uintptr_t)r | (uintptr_t)w | 256u;
    if (row_count > 0) {
        for (int i = 0; i < n_parts; ++i) {
            if (!x_parts[i]) {
                rt::set_error("x_parts[%d] is NULL", i);
                return RT_ERR_NULL;
            }
            bits |= (uintptr_t)x_parts[i];
        }
        for (int pass = 0; pass < 2; ++pass) {
            void* const* outs = pass == 0 ? y_outs : r_outs;
            const int n_dst = pass == 0 ? n_y_outs : n_r_outs;
            for (int i = 0; i < n_dst; ++i) {
                if (!outs[i]) {
                    rt::set_error("%s destination %d is NULL", pass == 0 ? "y" : "r_out", i);
                    return RT_ERR_NULL;
                }
                bits |= (uintptr_t)outs[i];
                for (int k = 0; k < n_parts; ++k)
                    if (outs[i] == x_parts[k]) {
                        rt::set_error("%s destination %d is part %d of x", pass == 0 ? "y" : "r_out", i, k);
                        return RT_ERR_SHAPE;
                    }
            }
        }
    }
    rt_limits L;
    int st = rt::current_limits(&L);
    if (st != RT_OK) return st;
    rt_shape s = {};
    s.n_tokens = row_count;
    s.hidden = hidden;
    s.dtype = dtype;
    s.min_ptr_align = (int32_t)(bits & (~bits + 1));
    s.op = RT_OP_ADD_RMSNORM_ALLREDUCE;
    s.n_parts = n_parts;
    rt::Plan plan;
    st = rt::make_plan(&s, p, &L, &plan);
    if (st != RT_OK) return st;
    return rt::launch_allreduce_plan(plan, x_parts, n_parts, r, w, y_outs, n_y_outs, r_outs, n_r_outs, row_begin, row_count,
                                     hidden, eps, (cudaStream_t)stream);
}

int merge_attn_states_template_launch(const rt_params* p, const void* v_a, const float* s_a, const void* v_b,
                                      const float* s_b, void* v_out, float* s_out, int64_t n_tokens, int64_t heads,
                                      int64_t head_dim, int dtype, void* stream)
{
    if (!p) {
        rt::set_error("params is NULL");
        return RT_ERR_NULL;
    }
    if (n_tokens > 0 && (!v_a || !s_a || !v_b || !s_b || !v_out || !s_out)) {
        rt::set_error("a tensor pointer is NULL");
        return RT_ERR_NULL;
    }
    if (heads <= 0 || head_dim <= 0 || head_dim > 0x7fffffff) {
        rt::set_error("heads=%lld head_dim=%lld out of range", (long long)heads, (long long)head_dim);
        return RT_ERR_SHAPE;
    }
    if (n_tokens > 0 && (((uintptr_t)s_a | (uintptr_t)s_b | (uintptr_t)s_out) & 3u)) {
        rt::set_error("the log-sum-exp tensors must be 4-byte aligned");
        return RT_ERR_ALIGN;
    }
    rt_limits L;
    int st = rt::current_limits(&L);
    if (st != RT_OK) return st;
    rt_shape s = {};
    s.n_tokens = n_tokens;
    s.hidden = heads * head_dim;
    s.dtype = dtype;
    s.min_ptr_align = n_tokens > 0 ? rt::min_pointer_alignment(v_a, v_b, v_out, v_a, v_b) : 256;
    s.op = RT_OP_MERGE_ATTN_STATES;
    s.head_dim = (int32_t)head_dim;
    rt::Plan plan;
    st = rt::make_plan(&s, p, &L, &plan);
    if (st != RT_OK) return st;
    return rt::launch_merge_plan(plan, v_a, s_a, v_b, s_b, v_out, s_out, n_tokens, (cudaStream_t)stream);
}

int rt_query_limits(rt_limits* out)
{
    if (!out) {
        rt::set_error("limits is NULL");
        return RT_ERR_NULL;
    }
    return rt::current_limits(out);
}

void rt_limits_sm100_nominal(rt_limits* out)
{
    if (!out) return;
    memset(out, 0, sizeof(*out));
    out->sm_count = 148;
    out->warp_size = 32;
    out->max_threads_per_block = 1024;
    out->max_threads_per_sm = 2048;
    out->max_blocks_per_sm = 32;
    out->regs_per_block = 65536;
    out->regs_per_sm = 65536;
    out->max_regs_per_thread = 255;
    out->max_cluster_size = 8;
    out->have_device = 0;
    out->smem_per_block_optin = 227 * 1024;
    out->smem_per_sm = 228 * 1024;
    out->smem_reserved_per_block = 1024;
    out->l2_bytes = 126LL * 1024 * 1024;
}

int tuner_check_params(const rt_shape* s, const rt_limits* limits, const rt_params* p)
{
    rt_limits L;
    if (!limits) {
        int st = rt::current_limits(&L);
        if (st != RT_OK) return st;
        limits = &L;
    }
    rt::Plan plan;
    return rt::make_plan(s, p, limits, &plan);
}

const char* rt_status_string(int status)
{
    switch (status) {
        case RT_OK: return "ok";
        case RT_ERR_NULL: return "a required pointer is NULL";
        case RT_ERR_DTYPE: return "unknown dtype";
        case RT_ERR_SHAPE: return "bad shape";
        case RT_ERR_ALIGN: return "pointer or row length not aligned to the vector width";
        case RT_ERR_INFEASIBLE: return "configuration outside the feasible region";
        case RT_ERR_CUDA: return "CUDA runtime error";
        case RT_ERR_MISMATCH: return "output differs from the reference beyond tolerance";
        case RT_ERR_BUDGET: return "search budget allows no evaluation";
        case RT_ERR_DEVICE_TIMEOUT: return "a bounded device-side wait expired";
        case RT_ERR_CAPACITY: return "caller-provided buffer too small";
        case RT_ERR_NO_DEVICE: return "no CUDA device";
        default: return "unknown status";
    }
}

const char* rt_last_error(void) { return rt::last_error(); }

int rt_device_status(void)
{
    int* p = rt::device_status_word();
    if (!p) return RT_ERR_CUDA;
    int v = 0;
    RT_CUDA_OK(cudaDeviceSynchronize());
    RT_CUDA_OK(cudaMemcpy(&v, p, sizeof(int), cudaMemcpyDeviceToHost));
    if (v != 0) {
        RT_CUDA_OK(cudaMemset(p, 0, sizeof(int)));
        rt::set_error("device status word = %d", v);
    }
    return v;
}

int32_t rt_num_kernel_instances(void) { return (int32_t)rt::registry().size(); }

int rt_kernel_instance(int32_t i, int32_t* dtype, int32_t* vec_bytes, int32_t* stage, int32_t* reduce, int32_t* unroll,
                       int32_t* reg_vectors)
{
    if (i < 0 || i >= (int32_t)rt::registry().size()) {
        rt::set_error("instance index %d out of range", i);
        return RT_ERR_CAPACITY;
    }
    const rt::KernelEntry& k = rt::registry()[i];
    if (dtype) *dtype = k.dtype;
    if (vec_bytes) *vec_bytes = k.vec_bytes;
    if (stage) *stage = k.stage;
    if (reduce) *reduce = k.reduce;
    if (unroll) *unroll = k.unroll;
    if (reg_vectors) *reg_vectors = k.cap;
    return RT_OK;
}

int32_t rt_kernel_instance_op(int32_t i)
{
    if (i < 0 || i >= (int32_t)rt::registry().size()) return -1;
    return rt::registry()[i].op;
}

int rt_set_option(int32_t option, int32_t value)
{
    if (option == RT_OPTION_PROGRAMMATIC_LAUNCH && (value == 0 || value == 1)) {
        rt::g_programmatic_launch.store(value);
    } else if (option == RT_OPTION_TMA_WAIT_POLL_LIMIT && value >= 1 && value <= (int32_t)rt::kMbarrierPollLimit) {
        rt::g_wait_polls.store(value);
    } else if (option == RT_OPTION_DEBUG_DROP_TMA_COPIES && (value == 0 || value == 1)) {
        rt::g_drop_tma_copies.store(value);
    } else {
        rt::set_error("unknown option %d or value %d", option, value);
        return RT_ERR_SHAPE;
    }
    return RT_OK;
}

int32_t rt_get_option(int32_t option)
{
    switch (option) {
        case RT_OPTION_PROGRAMMATIC_LAUNCH: return rt::g_programmatic_launch.load();
        case RT_OPTION_TMA_WAIT_POLL_LIMIT: return rt::g_wait_polls.load();
        case RT_OPTION_DEBUG_DROP_TMA_COPIES: return rt::g_drop_tma_copies.load();
        default: return -1;
    }
}

int32_t rt_kernel_instance_parts(int32_t i)
{
    if (i < 0 || i >= (int32_t)rt::registry().size()) return -1;
    return rt::registry()[i].parts;
}

int64_t rt_launch_count(void) { return rt::g_launches.load(); }

}  // extern "C"
