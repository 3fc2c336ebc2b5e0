// Search(S~, x, Theta_feasible): the correctness gate d(.,.) on the device, the timing protocol, and the
// guided search (seeds -> coarse grid -> best-first hill-climb -> Top-K re-test), after Algorithm 1
// (Level 2) and the "Tuning agent" / "Testing agent" roles of the paper.
#include <cuda_fp16.h>
#include <math.h>
#include <string.h>
#include <time.h>

#include <mutex>
#include <unordered_map>

#include "tuner_internal.h"

namespace rt {

// ---- d(.,.): element-wise comparison on the device ---------------------------------------------------

constexpr int kAccSlots = 4;  // accumulator records one evaluation may fill before it reads them back
struct CompareAcc {
    unsigned long long n_bad;
    unsigned int max_bits;  // ULP16: max distance; REL32: float bits of the max relative error; BITS: 0/1
    unsigned int pad;
};

__device__ __forceinline__ unsigned int ulp_distance16(unsigned int g, unsigned int q, unsigned int nan_above)
{
    const unsigned int gm = g & 0x7FFFu, qm = q & 0x7FFFu;
    const bool gn = gm > nan_above, qn = qm > nan_above;
    if (gn || qn) return (gn && qn) ? 0u : 65535u;
    // nan_above is the pattern of infinity: an overflowed value is not "one step" from the largest finite one
    if (gm == nan_above || qm == nan_above) return g == q ? 0u : 65535u;
    const int gi = (g & 0x8000u) ? -(int)gm : (int)gm;
    const int qi = (q & 0x8000u) ? -(int)qm : (int)qm;
    const int d = gi - qi;
    return (unsigned int)(d < 0 ? -d : d);
}

template <int MODE>
__device__ __forceinline__ void compare_word(unsigned int g, unsigned int q, int dtype, double tol,
                                             unsigned long long& bad, unsigned int& worst)
{
    if constexpr (MODE == RT_CMP_BITS) {
        if (dtype == RT_FP32) {
            if (g != q) { ++bad; worst = 1u; }
        } else {
            if ((g & 0xFFFFu) != (q & 0xFFFFu)) { ++bad; worst = 1u; }
            if ((g >> 16) != (q >> 16)) { ++bad; worst = 1u; }
        }
    } else if constexpr (MODE == RT_CMP_ULP16) {
        const unsigned int nan_above = dtype == RT_BF16 ? 0x7F80u : 0x7C00u;
        const unsigned int d0 = ulp_distance16(g & 0xFFFFu, q & 0xFFFFu, nan_above);
        const unsigned int d1 = ulp_distance16(g >> 16, q >> 16, nan_above);
        if ((double)d0 > tol) ++bad;
        if ((double)d1 > tol) ++bad;
        worst = max(worst, max(d0, d1));
    } else {
        const float gf = __uint_as_float(g), qf = __uint_as_float(q);
        const bool gn = gf != gf, qn = qf != qf;
        if (gn || qn) {
            if (!(gn && qn)) { ++bad; worst = 0x7F800000u; }
        } else if (gf != qf && (isinf(gf) || isinf(qf))) {
            ++bad;  // an infinity matches only itself
            worst = 0x7F800000u;
        } else if (gf != qf) {
            const double err = fabs((double)gf - (double)qf);
            const double mag = fabs((double)qf);
            if (!(err <= tol * mag + 1e-30)) ++bad;
            const float rel = (float)(err / fmax(mag, 1e-30));
            worst = max(worst, __float_as_uint(rel));
        }
    }
}

// got/ref viewed as 32-bit words (n_words of them); a trailing 16-bit element, if any, is handled
// by the last thread through the `tail` words (upper half zeroed on both sides).
template <int MODE>
__global__ void compare_kernel(const unsigned int* __restrict__ got, const unsigned int* __restrict__ ref,
                               long long n_words, int has_tail, unsigned int tail_got, unsigned int tail_ref,
                               int dtype, double tol, CompareAcc* acc)
{
    unsigned long long bad = 0;
    unsigned int worst = 0;
    const long long stride = (long long)gridDim.x * blockDim.x;
    for (long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x; i < n_words; i += stride)
        compare_word<MODE>(got[i], ref[i], dtype, tol, bad, worst);
    if (has_tail && blockIdx.x == 0 && threadIdx.x == 0) {
        unsigned long long b2 = 0;
        compare_word<MODE>(tail_got, tail_ref, dtype, tol, b2, worst);
        bad += b2 ? 1 : 0;  // the padded upper halves are equal and add nothing
    }
    for (int off = 16; off >= 1; off >>= 1) {
        bad += __shfl_xor_sync(0xffffffffu, bad, off);
        worst = max(worst, __shfl_xor_sync(0xffffffffu, worst, off));
    }
    if ((threadIdx.x & 31) == 0) {
        if (bad) atomicAdd(&acc->n_bad, bad);
        if (worst) atomicMax(&acc->max_bits, worst);
    }
}

// e4m3 codes: distance in code steps on the value lattice (+0 == -0, NaN matches NaN).
__global__ void compare_e4m3_kernel(const unsigned char* __restrict__ got, const unsigned char* __restrict__ ref,
                                    long long n, int tol_steps, CompareAcc* acc)
{
    unsigned long long bad = 0;
    unsigned int worst = 0;
    const long long stride = (long long)gridDim.x * blockDim.x;
    for (long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x; i < n; i += stride) {
        const unsigned int g = got[i], q = ref[i];
        const bool gn = (g & 0x7Fu) == 0x7Fu, qn = (q & 0x7Fu) == 0x7Fu;
        unsigned int d;
        if (gn || qn) {
            d = (gn && qn) ? 0u : 255u;
        } else {
            const int gi = (g & 0x80u) ? -(int)(g & 0x7Fu) : (int)(g & 0x7Fu);
            const int qi = (q & 0x80u) ? -(int)(q & 0x7Fu) : (int)(q & 0x7Fu);
            d = (unsigned int)(gi > qi ? gi - qi : qi - gi);
        }
        if ((int)d > tol_steps) ++bad;
        worst = max(worst, d);
    }
    for (int off = 16; off >= 1; off >>= 1) {
        bad += __shfl_xor_sync(0xffffffffu, bad, off);
        worst = max(worst, __shfl_xor_sync(0xffffffffu, worst, off));
    }
    if ((threadIdx.x & 31) == 0) {
        if (bad) atomicAdd(&acc->n_bad, bad);
        if (worst) atomicMax(&acc->max_bits, worst);
    }
}

// Mixed tolerance (outputs that may cancel): pass within `tol` ulps (16-bit) / relative (binary32) OR within
// `tol_abs` absolutely.  acc->max_bits receives the float bits of the largest absolute difference.
__device__ __forceinline__ float decode_elem16(unsigned int bits, int dtype)
{
    return dtype == RT_BF16 ? __uint_as_float(bits << 16) : __half2float(__ushort_as_half((unsigned short)bits));
}

__device__ __forceinline__ void mixed_elem(float g, float q, unsigned int ulps, bool use_ulps, double tol, double tol_abs,
                                           unsigned long long& bad, unsigned int& worst)
{
    const bool gn = g != g, qn = q != q;
    if (gn || qn) {
        if (!(gn && qn)) { ++bad; worst = 0x7F800000u; }
        return;
    }
    if (g == q) return;
    if (isinf(g) || isinf(q)) {  // an infinity matches only itself
        ++bad;
        worst = 0x7F800000u;
        return;
    }
    const double diff = fabs((double)g - (double)q);
    const bool ok = diff <= tol_abs || (use_ulps ? (double)ulps <= tol : diff <= tol * fabs((double)q));
    if (!ok) ++bad;
    worst = max(worst, __float_as_uint((float)diff));
}

__global__ void compare_mixed_kernel(const void* __restrict__ got, const void* __restrict__ ref, long long n, int dtype,
                                     double tol, double tol_abs, CompareAcc* acc)
{
    unsigned long long bad = 0;
    unsigned int worst = 0;
    const long long stride = (long long)gridDim.x * blockDim.x;
    for (long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x; i < n; i += stride) {
        if (dtype == RT_FP32) {
            mixed_elem(((const float*)got)[i], ((const float*)ref)[i], 0u, false, tol, tol_abs, bad, worst);
        } else {
            const unsigned int gb = ((const unsigned short*)got)[i], qb = ((const unsigned short*)ref)[i];
            const unsigned int nan_above = dtype == RT_BF16 ? 0x7F80u : 0x7C00u;
            mixed_elem(decode_elem16(gb, dtype), decode_elem16(qb, dtype), ulp_distance16(gb, qb, nan_above), true, tol,
                       tol_abs, bad, worst);
        }
    }
    for (int off = 16; off >= 1; off >>= 1) {
        bad += __shfl_xor_sync(0xffffffffu, bad, off);
        worst = max(worst, __shfl_xor_sync(0xffffffffu, worst, off));
    }
    if ((threadIdx.x & 31) == 0) {
        if (bad) atomicAdd(&acc->n_bad, bad);
        if (worst) atomicMax(&acc->max_bits, worst);
    }
}

// Scratch of the allocation-free comparison entry point: one accumulator record, kept in a fixed
// array that every device loading this library holds until the process exits.  In host code this name
// is only a handle for cudaGetSymbolAddress, never an address a kernel may be given.
constexpr int kStaticScratchBytes = 256;
constexpr int64_t kStaticCompareMaxElems = (int64_t)1 << 40;
static __device__ __align__(256) unsigned char g_static_compare_scratch[kStaticScratchBytes];
static_assert(sizeof(CompareAcc) <= kStaticScratchBytes, "accumulator record larger than the static scratch");

namespace {

// Upper bound of the comparison kernels' grids: 16 CTAs of 256 threads per SM of the current device.
int compare_grid_cap()
{
    rt_limits L;
    return current_limits(&L) == RT_OK ? 16 * std::max(1, L.sm_count) : 16 * 132;
}

// The comparison entry points and the evaluator share one accumulator block per device: calls are serialised.
std::mutex g_compare_mutex;
std::mutex g_scratch_mutex;
CompareAcc* g_static_scratch_addr[64];  // device address of the static scratch, per device

// Set-up of the static scratch for the current device: its device address, looked up once.
int static_scratch(CompareAcc** out)
{
    int dev = 0;
    RT_CUDA_OK(cudaGetDevice(&dev));
    if (dev < 0 || dev >= 64) {
        set_error("device index %d out of range", dev);
        return RT_ERR_NO_DEVICE;
    }
    std::lock_guard<std::mutex> lock(g_scratch_mutex);
    if (!g_static_scratch_addr[dev]) {
        void* p = nullptr;
        cudaError_t e = cudaGetSymbolAddress(&p, g_static_compare_scratch);
        if (e != cudaSuccess || !p) {
            (void)cudaGetLastError();
            set_error("cudaGetSymbolAddress(static compare scratch) failed: %s", cudaGetErrorString(e));
            return RT_ERR_CUDA;
        }
        g_static_scratch_addr[dev] = (CompareAcc*)p;
    }
    *out = g_static_scratch_addr[dev];
    return RT_OK;
}

struct Scratch {
    CompareAcc* dev = nullptr;
    CompareAcc* host = nullptr;  // page-locked
};
Scratch g_scratch[64];

int get_scratch(Scratch** out)
{
    int dev = 0;
    RT_CUDA_OK(cudaGetDevice(&dev));
    if (dev < 0 || dev >= 64) {
        set_error("device index %d out of range", dev);
        return RT_ERR_NO_DEVICE;
    }
    std::lock_guard<std::mutex> lock(g_scratch_mutex);
    Scratch& s = g_scratch[dev];
    if (!s.dev) {
        RT_CUDA_OK(cudaMalloc((void**)&s.dev, kAccSlots * sizeof(CompareAcc)));
        RT_CUDA_OK(cudaMallocHost((void**)&s.host, kAccSlots * sizeof(CompareAcc)));
    }
    *out = &s;
    return RT_OK;
}

// Enqueue one comparison into accumulator slot `slot`; results are read after a stream sync.
int enqueue_compare(const void* got, const void* ref, int64_t n, int dtype, int mode, double tol, CompareAcc* acc,
                    cudaStream_t stream)
{
    const int eb = elem_bytes_of(dtype);
    if (((uintptr_t)got | (uintptr_t)ref) & 3u) {
        set_error("tuner_compare needs 4-byte aligned buffers");
        return RT_ERR_ALIGN;
    }
    const long long n_words = (long long)(n * eb / 4);
    const int has_tail = (n * eb) % 4 != 0;
    unsigned int tail_got = 0, tail_ref = 0;
    if (has_tail) {  // one trailing 16-bit element: fetch it to the host side of the launch
        unsigned short tg = 0, tr = 0;
        RT_CUDA_OK(cudaMemcpyAsync(&tg, (const char*)got + n_words * 4, 2, cudaMemcpyDeviceToHost, stream));
        RT_CUDA_OK(cudaMemcpyAsync(&tr, (const char*)ref + n_words * 4, 2, cudaMemcpyDeviceToHost, stream));
        RT_CUDA_OK(cudaStreamSynchronize(stream));
        tail_got = tg;
        tail_ref = tr;
    }
    const int threads = 256;
    long long want = (n_words + threads * 8 - 1) / (threads * 8);
    const int blocks = (int)std::max<long long>(1, std::min<long long>(want, (long long)compare_grid_cap()));
    const unsigned int* g = (const unsigned int*)got;
    const unsigned int* q = (const unsigned int*)ref;
    if (mode == RT_CMP_BITS)
        compare_kernel<RT_CMP_BITS><<<blocks, threads, 0, stream>>>(g, q, n_words, has_tail, tail_got, tail_ref, dtype, tol, acc);
    else if (mode == RT_CMP_ULP16)
        compare_kernel<RT_CMP_ULP16><<<blocks, threads, 0, stream>>>(g, q, n_words, has_tail, tail_got, tail_ref, dtype, tol, acc);
    else
        compare_kernel<RT_CMP_REL32><<<blocks, threads, 0, stream>>>(g, q, n_words, has_tail, tail_got, tail_ref, dtype, tol, acc);
    RT_CUDA_OK(cudaGetLastError());
    count_launch();
    return RT_OK;
}

int enqueue_compare_e4m3(const void* got, const void* ref, int64_t n, int tol_steps, CompareAcc* acc, cudaStream_t stream)
{
    const int threads = 256;
    const long long want = (n + threads * 16 - 1) / (threads * 16);
    const int blocks = (int)std::max<long long>(1, std::min<long long>(want, (long long)compare_grid_cap()));
    compare_e4m3_kernel<<<blocks, threads, 0, stream>>>((const unsigned char*)got, (const unsigned char*)ref, n, tol_steps, acc);
    RT_CUDA_OK(cudaGetLastError());
    count_launch();
    return RT_OK;
}

int enqueue_compare_mixed(const void* got, const void* ref, int64_t n, int dtype, double tol, double tol_abs,
                          CompareAcc* acc, cudaStream_t stream)
{
    const int threads = 256;
    const long long want = (n + threads * 8 - 1) / (threads * 8);
    const int blocks = (int)std::max<long long>(1, std::min<long long>(want, (long long)compare_grid_cap()));
    compare_mixed_kernel<<<blocks, threads, 0, stream>>>(got, ref, n, dtype, tol, tol_abs, acc);
    RT_CUDA_OK(cudaGetLastError());
    count_launch();
    return RT_OK;
}

int check_compare_args(const void* got, const void* ref, int64_t n, int dtype, int mode)
{
    if (!got || !ref) {
        set_error("tuner_compare: NULL buffer");
        return RT_ERR_NULL;
    }
    if (dtype < 0 || dtype > 2) {
        set_error("dtype %d unknown", dtype);
        return RT_ERR_DTYPE;
    }
    if (n < 0) {
        set_error("n = %lld is negative", (long long)n);
        return RT_ERR_SHAPE;
    }
    if (mode < RT_CMP_BITS || mode > RT_CMP_REL32 || (mode == RT_CMP_ULP16 && dtype == RT_FP32) ||
        (mode == RT_CMP_REL32 && dtype != RT_FP32)) {
        set_error("compare mode %d does not apply to dtype %d", mode, dtype);
        return RT_ERR_DTYPE;
    }
    return RT_OK;
}

double acc_max_err(const CompareAcc& a, int mode)
{
    if (mode == RT_CMP_REL32) {
        float f;
        memcpy(&f, &a.max_bits, sizeof(f));
        return (double)f;
    }
    return (double)a.max_bits;
}

}  // namespace

// ---- evaluation of one theta: gate, then the timing protocol ----------------------------------------

struct Evaluator {
    virtual ~Evaluator() {}
    // Fills rec->status, the gate statistics and the times.  Returns RT_OK unless the evaluation
    // itself could not be carried out (a CUDA failure that is not specific to the candidate).
    virtual int evaluate(const rt_params& p, rt_eval_record* rec) = 0;
    // Top-K re-test of `n` finalists: one record per finalist.  The default measures them one after the other.
    virtual int retest(const rt_params* ps, int n, rt_eval_record* recs)
    {
        for (int i = 0; i < n; ++i) {
            const int st = evaluate(ps[i], &recs[i]);
            if (st != RT_OK) return st;
        }
        return RT_OK;
    }
    // true: a finalist's score becomes its re-test time (all finalists were re-timed side by side, under one clock
    // regime); false: the mean of its two measurements.
    virtual bool retest_replaces() const { return false; }
};

static float median_of(std::vector<float> v)
{
    std::sort(v.begin(), v.end());
    const size_t n = v.size();
    return n % 2 ? v[n / 2] : 0.5f * (v[n / 2 - 1] + v[n / 2]);
}

static double monotonic_seconds()
{
    timespec ts;
    clock_gettime(CLOCK_MONOTONIC, &ts);
    return (double)ts.tv_sec + 1e-9 * (double)ts.tv_nsec;
}

struct DeviceEvaluator : Evaluator {
    rt_shape shape;
    rt_budget budget;
    rt_workspace ws;
    rt_limits limits;

    cudaStream_t stream() const { return (cudaStream_t)ws.stream; }
    int elem_bytes() const { return elem_bytes_of(shape.dtype); }
    size_t set_bytes() const { return (size_t)shape.n_tokens * shape.hidden * elem_bytes(); }
    size_t lse_bytes(const Plan& plan) const  // merge_attn_states: one log-sum-exp tensor
    {
        return shape.op == RT_OP_MERGE_ATTN_STATES ? (size_t)shape.n_tokens * plan.heads * sizeof(float) : 0;
    }

    // One launch of the plan on ring set k (set 0 when the workspace has one set).
    int launch_set(const Plan& plan, int k) const
    {
        const int sets = ws.ring_sets > 0 ? ws.ring_sets : 1;
        const int eb = elem_bytes();
        const size_t set = (size_t)(k % sets);
        const size_t off = set * (size_t)ws.ring_stride_bytes;
        switch (shape.op) {
            case RT_OP_ADD_RMSNORM_ALLREDUCE: {
                // the parts of x lie one after the other in ws.x; one destination
                const void* parts[RT_MAX_PARTS];
                for (int j = 0; j < shape.n_parts; ++j)
                    parts[j] = (const char*)ws.x + (size_t)shape.n_parts * off + (size_t)j * set_bytes();
                void* y_out = (char*)ws.y + off;
                void* r_out = (char*)ws.r_out + off;
                return launch_allreduce_plan(plan, parts, shape.n_parts, (const char*)ws.r + off, ws.w, &y_out, 1, &r_out, 1,
                                             0, shape.n_tokens, shape.hidden, ws.eps, stream());
            }
            case RT_OP_ADD_RMSNORM_FP8:
                return launch_fp8_plan(plan, (const char*)ws.x + off, (const char*)ws.r + off, ws.w, (char*)ws.y + off / eb,
                                       (float*)((char*)ws.aux_out + set * shape.n_tokens * sizeof(float)),
                                       (char*)ws.r_out + off, shape.n_tokens, shape.hidden, ws.eps, stream());
            case RT_OP_MERGE_ATTN_STATES: {
                const size_t so = set * lse_bytes(plan);
                return launch_merge_plan(plan, (const char*)ws.x + off, (const float*)((const char*)ws.w + so),
                                         (const char*)ws.r + off, (const float*)((const char*)ws.aux + so),
                                         (char*)ws.y + off, (float*)((char*)ws.r_out + so), shape.n_tokens, stream());
            }
            case RT_OP_SILU_AND_MUL:  // the input rows are twice as long as the output rows
                return launch_silu_plan(plan, (const char*)ws.x + 2 * off, (char*)ws.y + off, shape.n_tokens, stream());
            default:
                return launch_plan(plan, (const char*)ws.x + off, (const char*)ws.r + off, ws.w, (char*)ws.y + off,
                                   (char*)ws.r_out + off, shape.n_tokens, shape.hidden, ws.eps, stream());
        }
    }

    // Reads and clears the device status word.  A bounded wait that expired marks the candidate, not the search.
    int status_word_clear(rt_eval_record* rec) const
    {
        int* word = device_status_word();
        if (!word) return RT_ERR_CUDA;
        int flag = 0;
        RT_CUDA_OK(cudaMemcpy(&flag, word, sizeof(int), cudaMemcpyDeviceToHost));
        if (flag) {
            RT_CUDA_OK(cudaMemset(word, 0, sizeof(int)));
            rec->status = RT_ERR_DEVICE_TIMEOUT;
        }
        return RT_OK;
    }

    // theta -> plan; rec->status carries a refusal.  Returns false when the candidate was refused.
    bool plan_for(const rt_params& p, Plan* plan, rt_eval_record* rec) const
    {
        memset(rec, 0, sizeof(*rec));
        rec->params = p;
        const int st = make_plan(&shape, &p, &limits, plan);
        if (st != RT_OK) {
            rec->status = st;
            return false;
        }
        int regs = 0;
        rec->occupancy_blocks_per_sm = plan_occupancy(*plan, &limits, &regs);
        rec->regs_per_thread = regs;
        return true;
    }

    // The correctness gate: one launch on set 0 compared with the uploaded references.  rec->status = RT_OK,
    // RT_ERR_MISMATCH, RT_ERR_DEVICE_TIMEOUT or the launch's refusal.  Outputs are poisoned first (all-ones is NaN
    // in all three types), so that values left by an earlier candidate cannot pass for this one's.
    int gate(const rt_params& p, const Plan& plan, rt_eval_record* rec) const
    {
        const int eb = elem_bytes();
        const int64_t n_ref = ws.n_ref_tokens;
        Scratch* sc;
        int st = get_scratch(&sc);
        if (st != RT_OK) return st;
        const bool is_silu = shape.op == RT_OP_SILU_AND_MUL;
        const bool is_merge = shape.op == RT_OP_MERGE_ATTN_STATES;
        const bool is_fp8 = shape.op == RT_OP_ADD_RMSNORM_FP8;
        cudaStream_t s = stream();
        RT_CUDA_OK(cudaMemsetAsync(ws.y, 0xFF, is_fp8 ? set_bytes() / eb : set_bytes(), s));
        if (is_fp8) RT_CUDA_OK(cudaMemsetAsync(ws.aux_out, 0xFF, (size_t)shape.n_tokens * sizeof(float), s));
        if (is_merge) RT_CUDA_OK(cudaMemsetAsync(ws.r_out, 0xFF, lse_bytes(plan), s));
        else if (!is_silu) RT_CUDA_OK(cudaMemsetAsync(ws.r_out, 0xFF, set_bytes(), s));
        RT_CUDA_OK(cudaMemsetAsync(sc->dev, 0, kAccSlots * sizeof(CompareAcc), s));
        st = launch_set(plan, 0);
        if (st != RT_OK) {
            rec->status = st;
            return RT_OK;
        }
        const int y_mode = shape.dtype == RT_FP32 ? RT_CMP_REL32 : RT_CMP_ULP16;
        const double y_tol = shape.dtype == RT_FP32 ? 1e-5 : 2.0;
        if (is_fp8) {
            // residual bit-exact; codes within one e4m3 step; per-token scales within 1e-5 relative
            st = enqueue_compare(ws.r_out, ws.r_ref, n_ref * shape.hidden, shape.dtype, RT_CMP_BITS, 0.0, sc->dev, s);
            if (st != RT_OK) return st;
            st = enqueue_compare_e4m3(ws.y, ws.y_ref, n_ref * shape.hidden, 1, sc->dev + 1, s);
            if (st != RT_OK) return st;
            st = enqueue_compare(ws.aux_out, ws.aux_ref, n_ref, RT_FP32, RT_CMP_REL32, 1e-5, sc->dev + 2, s);
            if (st != RT_OK) return st;
        } else if (is_merge) {
            // outputs that may cancel: 2 ulp / 1e-5 relative, or 1e-5 absolute; the merged log-sum-exp likewise
            st = enqueue_compare_mixed(ws.r_out, ws.r_ref, n_ref * plan.heads, RT_FP32, 1e-5, 1e-5, sc->dev, s);
            if (st != RT_OK) return st;
            st = enqueue_compare_mixed(ws.y, ws.y_ref, n_ref * shape.hidden, shape.dtype, y_tol, 1e-5, sc->dev + 1, s);
            if (st != RT_OK) return st;
        } else {
            if (!is_silu) {
                st = enqueue_compare(ws.r_out, ws.r_ref, n_ref * shape.hidden, shape.dtype, RT_CMP_BITS, 0.0, sc->dev, s);
                if (st != RT_OK) return st;
            }
            st = enqueue_compare(ws.y, ws.y_ref, n_ref * shape.hidden, shape.dtype, y_mode, y_tol, sc->dev + 1, s);
            if (st != RT_OK) return st;
        }
        RT_CUDA_OK(cudaMemcpyAsync(sc->host, sc->dev, kAccSlots * sizeof(CompareAcc), cudaMemcpyDeviceToHost, s));
        cudaError_t e = cudaStreamSynchronize(s);
        if (e != cudaSuccess) {
            set_error("candidate faulted: %s", cudaGetErrorString(e));
            return RT_ERR_CUDA;  // a sticky error: nothing further can run in this context
        }
        rec->r_bad = (int64_t)sc->host[0].n_bad;
        rec->y_bad = (int64_t)sc->host[1].n_bad + (is_fp8 ? (int64_t)sc->host[2].n_bad : 0);
        if (is_fp8)
            rec->y_max_ulp = (int32_t)sc->host[1].max_bits;  // e4m3 code steps
        else if (shape.dtype == RT_FP32 || is_merge)
            rec->y_max_rel = (float)acc_max_err(sc->host[1], RT_CMP_REL32);  // merge: largest absolute difference
        else
            rec->y_max_ulp = (int32_t)sc->host[1].max_bits;
        if (p.stage == RT_STAGE_SMEM_TMA || p.stage == RT_STAGE_TMA_PIPELINE) {
            st = status_word_clear(rec);
            if (st != RT_OK) return st;
            if (rec->status != RT_OK) return RT_OK;
        }
        if (rec->r_bad || rec->y_bad) rec->status = RT_ERR_MISMATCH;
        return RT_OK;
    }

    // The timed block as one CUDA graph of `iters` launches, replayed once untimed.  A candidate that cannot be
    // captured gets rec->status; *exec stays NULL.
    int capture_block(const Plan& plan, int iters, cudaGraphExec_t* exec, rt_eval_record* rec) const
    {
        *exec = nullptr;
        if (!stream()) {
            set_error("use_graph needs a non-default stream");
            return RT_ERR_CUDA;
        }
        cudaGraph_t graph = nullptr;
        RT_CUDA_OK(cudaStreamBeginCapture(stream(), cudaStreamCaptureModeThreadLocal));
        int cap_st = RT_OK;
        for (int i = 0; i < iters && cap_st == RT_OK; ++i) cap_st = launch_set(plan, i);
        cudaError_t ce = cudaStreamEndCapture(stream(), &graph);
        if (cap_st != RT_OK || ce != cudaSuccess) {
            if (graph) cudaGraphDestroy(graph);
            (void)cudaGetLastError();
            rec->status = cap_st != RT_OK ? cap_st : RT_ERR_CUDA;
            return RT_OK;
        }
        ce = cudaGraphInstantiate(exec, graph, 0);
        cudaGraphDestroy(graph);
        if (ce != cudaSuccess) {
            *exec = nullptr;
            set_error("cudaGraphInstantiate failed: %s", cudaGetErrorString(ce));
            return RT_ERR_CUDA;
        }
        RT_CUDA_OK(cudaGraphLaunch(*exec, stream()));  // one untimed replay
        return RT_OK;
    }

    // `iters` launches between two events; *us = block time / iters.
    int timed_block(const Plan& plan, cudaGraphExec_t exec, int iters, cudaEvent_t e0, cudaEvent_t e1, float* us) const
    {
        int fail = RT_OK;
        cudaEventRecord(e0, stream());
        if (exec) {
            if (cudaGraphLaunch(exec, stream()) != cudaSuccess) fail = RT_ERR_CUDA;
            count_launch(iters);
        } else {
            for (int i = 0; i < iters && fail == RT_OK; ++i) fail = launch_set(plan, i);
        }
        cudaEventRecord(e1, stream());
        if (cudaEventSynchronize(e1) != cudaSuccess) fail = RT_ERR_CUDA;
        float ms = 0.f;
        if (fail == RT_OK && cudaEventElapsedTime(&ms, e0, e1) != cudaSuccess) fail = RT_ERR_CUDA;
        if (fail != RT_OK) {
            cudaError_t le = cudaGetLastError();
            set_error("timing failed: %s", cudaGetErrorString(le));
            return RT_ERR_CUDA;
        }
        *us = ms * 1000.f / (float)iters;
        return RT_OK;
    }

    // Keeps the device busy with launches of `plan` for budget.preheat_ms, so that what is timed next runs at the
    // clocks of a loaded device (a B200 under a memory-bound kernel settles some 15% below its idle SM clock once its
    // power limit is reached) rather than at those of a device that was just waiting for the host.
    int preheat(const Plan& plan) const
    {
        if (budget.preheat_ms <= 0) return RT_OK;
        const double t_end = monotonic_seconds() + 1e-3 * (double)budget.preheat_ms;
        int k = 0;
        do {
            for (int i = 0; i < 64; ++i) {
                const int st = launch_set(plan, k++);
                if (st != RT_OK) return st;
            }
            RT_CUDA_OK(cudaStreamSynchronize(stream()));
        } while (monotonic_seconds() < t_end);
        return RT_OK;
    }
    bool heated = false;  // the first candidate that passes its gate pre-heats the device for the whole search

    static void fill_times(const std::vector<float>& block_us, rt_eval_record* rec)
    {
        float sum = 0.f, mn = block_us[0];
        for (float v : block_us) {
            sum += v;
            mn = std::min(mn, v);
        }
        rec->us = median_of(block_us);
        rec->us_min_block = mn;
        rec->us_mean = sum / (float)block_us.size();
    }

    int evaluate(const rt_params& p, rt_eval_record* rec) override
    {
        std::lock_guard<std::mutex> serial(g_compare_mutex);
        Plan plan;
        if (!plan_for(p, &plan, rec)) return RT_OK;
        int st = gate(p, plan, rec);
        if (st != RT_OK || rec->status != RT_OK) return st;
        if (!heated) {
            heated = true;
            st = preheat(plan);
            if (st != RT_OK) return st;
        }

        // Timing: `warmup` launches, then `repeats` blocks of `iters` launches between two events.
        for (int i = 0; i < budget.warmup; ++i) {
            st = launch_set(plan, i);
            if (st != RT_OK) {
                rec->status = st;
                return RT_OK;
            }
        }
        const int iters = budget.iters > 0 ? budget.iters : 1;
        const int repeats = budget.repeats > 0 ? budget.repeats : 1;
        cudaGraphExec_t graph_exec = nullptr;
        if (budget.use_graph) {
            st = capture_block(plan, iters, &graph_exec, rec);
            if (st != RT_OK || rec->status != RT_OK) return st;
        }
        cudaEvent_t e0, e1;
        RT_CUDA_OK(cudaEventCreate(&e0));
        RT_CUDA_OK(cudaEventCreate(&e1));
        std::vector<float> block_us;
        st = RT_OK;
        for (int rep = 0; rep < repeats && st == RT_OK; ++rep) {
            float us = 0.f;
            st = timed_block(plan, graph_exec, iters, e0, e1, &us);
            if (st == RT_OK) block_us.push_back(us);
        }
        cudaEventDestroy(e0);
        cudaEventDestroy(e1);
        if (graph_exec) cudaGraphExecDestroy(graph_exec);
        if (st != RT_OK) return st;
        fill_times(block_us, rec);
        // a bounded wait may also expire in a timed launch: such a time is not a time of the operator
        if (p.stage == RT_STAGE_SMEM_TMA || p.stage == RT_STAGE_TMA_PIPELINE) return status_word_clear(rec);
        return RT_OK;
    }

    // Re-timing of several thetas side by side: every theta passes the gate once, then `rounds` rounds; in a round
    // every theta runs one block (warm-up launches, then `iters` timed launches) before any theta runs its next
    // block, and the order rotates by one from round to round.  Clock and power changes during the measurement
    // therefore meet every theta alike.  recs[i]: status, gate statistics, median / fastest / mean block of theta i;
    // blocks (may be NULL): one record per (round, theta) block in the order they ran.
    int interleaved(const rt_params* ps, int n, int rounds, rt_eval_record* recs, rt_block_record* blocks,
                    int* n_blocks_out = nullptr)
    {
        std::lock_guard<std::mutex> serial(g_compare_mutex);
        const int iters = budget.iters > 0 ? budget.iters : 1;
        std::vector<Plan> plans((size_t)n);
        std::vector<cudaGraphExec_t> execs((size_t)n, nullptr);
        std::vector<std::vector<float>> times((size_t)n);
        int st = RT_OK;
        for (int i = 0; i < n && st == RT_OK; ++i) {
            if (!plan_for(ps[i], &plans[i], &recs[i])) continue;
            st = gate(ps[i], plans[i], &recs[i]);
            if (st == RT_OK && recs[i].status == RT_OK && budget.use_graph)
                st = capture_block(plans[i], iters, &execs[i], &recs[i]);
        }
        for (int i = 0; i < n && st == RT_OK; ++i)
            if (recs[i].status == RT_OK) {  // the side-by-side comparison is made on a loaded device
                st = preheat(plans[i]);
                break;
            }
        cudaEvent_t e0 = nullptr, e1 = nullptr;
        if (st == RT_OK && (cudaEventCreate(&e0) != cudaSuccess || cudaEventCreate(&e1) != cudaSuccess)) {
            set_error("cudaEventCreate failed");
            st = RT_ERR_CUDA;
        }
        int n_blocks = 0;
        for (int round = 0; round < rounds && st == RT_OK; ++round)
            for (int j = 0; j < n && st == RT_OK; ++j) {
                const int i = (j + round) % n;
                if (recs[i].status != RT_OK) continue;
                for (int k = 0; k < budget.warmup && st == RT_OK; ++k) st = launch_set(plans[i], k);
                if (st != RT_OK) break;
                if (cudaStreamSynchronize(stream()) != cudaSuccess) {
                    set_error("warm-up faulted");
                    st = RT_ERR_CUDA;
                    break;
                }
                float us = 0.f;
                const double t0 = monotonic_seconds();
                st = timed_block(plans[i], execs[i], iters, e0, e1, &us);
                const double t1 = monotonic_seconds();
                if (st != RT_OK) break;
                times[i].push_back(us);
                if (blocks) {
                    rt_block_record& b = blocks[n_blocks];
                    b.theta_index = i;
                    b.round = round;
                    b.us = us;
                    b.reserved = 0;
                    b.t_begin_s = t0;
                    b.t_end_s = t1;
                }
                ++n_blocks;
            }
        if (n_blocks_out) *n_blocks_out = n_blocks;
        if (e0) cudaEventDestroy(e0);
        if (e1) cudaEventDestroy(e1);
        for (cudaGraphExec_t g : execs)
            if (g) cudaGraphExecDestroy(g);
        if (st != RT_OK) return st;
        for (int i = 0; i < n; ++i) {
            if (recs[i].status != RT_OK) continue;
            if (times[i].empty()) {
                recs[i].status = RT_ERR_BUDGET;  // rounds < 1: gated, not timed
                continue;
            }
            fill_times(times[i], &recs[i]);
            if (ps[i].stage == RT_STAGE_SMEM_TMA || ps[i].stage == RT_STAGE_TMA_PIPELINE) {
                // the word is shared: an expired wait is charged to every TMA candidate of this re-test
                rt_eval_record probe = recs[i];
                st = status_word_clear(&probe);
                if (st != RT_OK) return st;
                if (probe.status != RT_OK)
                    for (int k = 0; k < n; ++k)
                        if (recs[k].status == RT_OK && (ps[k].stage == RT_STAGE_SMEM_TMA || ps[k].stage == RT_STAGE_TMA_PIPELINE))
                            recs[k].status = RT_ERR_DEVICE_TIMEOUT;
            }
        }
        return RT_OK;
    }

    int retest(const rt_params* ps, int n, rt_eval_record* recs) override
    {
        return interleaved(ps, n, budget.repeats > 0 ? budget.repeats : 1, recs, nullptr);
    }
    bool retest_replaces() const override { return true; }
};

// The launch floor: an empty kernel timed with the same protocol, so that the share of launch overhead in
// the time of a latency-bound shape is visible.
__global__ void empty_kernel() {}

static int time_launch_floor(const rt_budget& b, cudaStream_t stream, float* out_us)
{
    const int iters = b.iters > 0 ? b.iters : 1, repeats = b.repeats > 0 ? b.repeats : 1;
    for (int i = 0; i < b.warmup; ++i) empty_kernel<<<1, 32, 0, stream>>>();
    cudaGraphExec_t graph_exec = nullptr;
    if (b.use_graph) {
        if (!stream) {
            set_error("use_graph needs a non-default stream");
            return RT_ERR_CUDA;
        }
        cudaGraph_t graph = nullptr;
        RT_CUDA_OK(cudaStreamBeginCapture(stream, cudaStreamCaptureModeThreadLocal));
        for (int i = 0; i < iters; ++i) empty_kernel<<<1, 32, 0, stream>>>();
        RT_CUDA_OK(cudaStreamEndCapture(stream, &graph));
        cudaError_t ce = cudaGraphInstantiate(&graph_exec, graph, 0);
        cudaGraphDestroy(graph);
        if (ce != cudaSuccess) {
            set_error("cudaGraphInstantiate failed: %s", cudaGetErrorString(ce));
            return RT_ERR_CUDA;
        }
        RT_CUDA_OK(cudaGraphLaunch(graph_exec, stream));
    }
    cudaEvent_t e0, e1;
    RT_CUDA_OK(cudaEventCreate(&e0));
    RT_CUDA_OK(cudaEventCreate(&e1));
    std::vector<float> block_us;
    for (int rep = 0; rep < repeats; ++rep) {
        cudaEventRecord(e0, stream);
        if (graph_exec) {
            cudaGraphLaunch(graph_exec, stream);
        } else {
            for (int i = 0; i < iters; ++i) empty_kernel<<<1, 32, 0, stream>>>();
        }
        cudaEventRecord(e1, stream);
        float ms = 0.f;
        if (cudaEventSynchronize(e1) == cudaSuccess && cudaEventElapsedTime(&ms, e0, e1) == cudaSuccess)
            block_us.push_back(ms * 1000.f / iters);
    }
    count_launch((int64_t)repeats * iters + b.warmup);
    cudaEventDestroy(e0);
    cudaEventDestroy(e1);
    if (graph_exec) cudaGraphExecDestroy(graph_exec);
    RT_CUDA_OK(cudaGetLastError());
    if (block_us.empty()) {
        set_error("launch-floor timing failed");
        return RT_ERR_CUDA;
    }
    *out_us = median_of(block_us);
    return RT_OK;
}

struct CallbackEvaluator : Evaluator {
    rt_evaluate_fn fn;
    void* user;
    int evaluate(const rt_params& p, rt_eval_record* rec) override
    {
        memset(rec, 0, sizeof(*rec));
        rec->params = p;
        const double t = fn(&p, user);
        if (!(t >= 0.0) || isinf(t)) {
            rec->status = RT_ERR_MISMATCH;
        } else {
            rec->us = rec->us_min_block = rec->us_mean = (float)t;
            rec->status = RT_OK;
        }
        return RT_OK;
    }
};

// ---- the search --------------------------------------------------------------------------------------

namespace {

int level_of(const int* levels, int n, int v)
{
    for (int i = 0; i < n; ++i)
        if (levels[i] == v) return i;
    return -1;
}
const int kTpr[] = {32, 64, 128, 256, 512, 1024};
const int kRpc[] = {1, 2, 4, 8};
const int kUnr[] = {1, 2, 4};
const int kVec[] = {2, 4, 8, 16, 32};
const int kClu[] = {1, 2, 4, 8};
constexpr float kStageLeaderMargin = 1.03f;
constexpr float kRetestTie = 1.005f;  // re-test times this close count as a tie
constexpr int kCentreVectorsPerThread = 1;  // vectors a thread owns at the centre level of the threads-per-row axis  // a stage's fastest point is climbed from while it is this close to the leader

struct SearchState {
    std::vector<rt_params> cand;
    std::unordered_map<uint64_t, int> index;
    std::vector<float> time_us;   // < 0: not evaluated; +inf: failed its gate
    std::vector<char> expanded;
    int used = 0, failed = 0;
    int max_evals = 0;
    rt_eval_record* log = nullptr;
    int log_cap = 0, n_log = 0;
    Evaluator* ev = nullptr;

    int add(const rt_params& p)
    {
        auto it = index.find(pack_params(p));
        if (it != index.end()) return it->second;
        cand.push_back(p);
        time_us.push_back(-1.f);
        expanded.push_back(0);
        index[pack_params(p)] = (int)cand.size() - 1;
        return (int)cand.size() - 1;
    }
    bool budget_left(int reserve) const { return used < max_evals - reserve; }

    // One evaluation (counts against the budget).  Returns a hard error or RT_OK.
    int run(int idx, int phase, float* out_us)
    {
        rt_eval_record rec;
        int st = ev->evaluate(cand[idx], &rec);
        rec.phase = phase;
        rec.eval_index = used;
        ++used;
        if (log && n_log < log_cap) log[n_log++] = rec;
        if (st != RT_OK) return st;
        if (rec.status != RT_OK) {
            ++failed;
            *out_us = INFINITY;
        } else {
            *out_us = rec.us;
        }
        return RT_OK;
    }

    // One-step neighbours: +-1 level on one ordered axis, or another stage, or another reduction.
    std::vector<int> neighbours(int idx) const
    {
        std::vector<int> out;
        const rt_params& p = cand[idx];
        auto probe = [&](rt_params q) {
            auto it = index.find(pack_params(q));
            if (it != index.end() && it->second != idx) out.push_back(it->second);
        };
        // A step along the block-shape or vector axis can land where the current unroll depth is pruned as a
        // duplicate (more threads per row or wider vectors leave a thread fewer vectors than the batch is deep):
        // the neighbour is then that point with the deepest unroll that exists there.
        auto step = [&](const int* levels, int n, int rt_params::*field) {
            const int l = level_of(levels, n, p.*field);
            for (int d = -1; d <= 1; d += 2) {
                if (l + d < 0 || l + d >= n || l < 0) continue;
                rt_params q = p;
                q.*field = levels[l + d];
                if (field != &rt_params::unroll)
                    while (q.unroll > 1 && index.find(pack_params(q)) == index.end()) q.unroll /= 2;
                probe(q);
            }
        };
        step(kTpr, 6, &rt_params::threads_per_row);
        step(kRpc, 4, &rt_params::rows_per_cta);
        step(kUnr, 3, &rt_params::unroll);
        step(kVec, 5, &rt_params::vec_bytes);
        // Two diagonal steps that keep what a thread does unchanged: half the vector width with twice the unroll (the
        // same bytes in flight per thread, in narrower instructions), and half the vector width with twice the threads per
        // row (the same vectors per thread), and their reverses.  Along a single axis both halves of such a move are
        // usually worse than the point they start from, so a climb over single steps does not cross them.
        {
            const int lv = level_of(kVec, 5, p.vec_bytes), lu = level_of(kUnr, 3, p.unroll),
                      lt = level_of(kTpr, 6, p.threads_per_row);
            for (int d = -1; d <= 1; d += 2) {
                if (lv < 0 || lv + d < 0 || lv + d >= 5) continue;
                if (lu >= 0 && lu - d >= 0 && lu - d < 3) {
                    rt_params q = p;
                    q.vec_bytes = kVec[lv + d];
                    q.unroll = kUnr[lu - d];
                    probe(q);
                }
                if (lt >= 0 && lt - d >= 0 && lt - d < 6) {
                    rt_params q = p;
                    q.vec_bytes = kVec[lv + d];
                    q.threads_per_row = kTpr[lt - d];
                    while (q.unroll > 1 && index.find(pack_params(q)) == index.end()) q.unroll /= 2;
                    probe(q);
                }
            }
        }
        // another stage at the same vector width; where that stage has no such point (the ragged-row stage is
        // all 16-byte chunks while the other stages of a misaligned shape are narrower), at its widest width
        for (int stage = 0; stage <= RT_STAGE_TMA_PIPELINE; ++stage) {
            rt_params q = p;
            q.stage = stage;
            if (index.find(pack_params(q)) == index.end()) {
                if (stage == RT_STAGE_REG_REALIGN) q.reduce = RT_REDUCE_SHFL, q.cluster_size = 1;
                for (int k = 4; k >= 0; --k) {
                    q.vec_bytes = kVec[k];
                    if (index.find(pack_params(q)) != index.end()) break;
                }
            }
            probe(q);
        }
        for (int reduce = 0; reduce < 3; ++reduce)
            for (int c : kClu) {
                if ((reduce == RT_REDUCE_CLUSTER) != (c > 1)) continue;
                rt_params q = p;
                q.reduce = reduce;
                q.cluster_size = c;
                probe(q);
            }
        return out;
    }
};

// The centre of the threads-per-row axis for a point's mode: the level at which a thread owns about one vector of its
// CTA's slice of the row at the stage's widest vector (8192 bf16 elements in 32-byte vectors: 512 threads; the same
// row split over a cluster of 8: 64).  The optima of the recorded sweeps sit at that level or next to it, so the grid
// and the small-budget order are laid out from there instead of from a fixed 256.
int centre_level(const rt_shape& s, const rt_params& p, int vec_bytes)
{
    const int64_t slice_vectors =
        std::max<int64_t>(1, s.hidden * (s.dtype == RT_FP32 ? 4 : 2) / vec_bytes / std::max(1, p.cluster_size));
    int level = 0;
    while (level < 5 && kTpr[level] * kCentreVectorsPerThread < slice_vectors) ++level;
    return level;
}

// The coarse grid: every other level of the ordered axes (threads per row: the centre level and every second level
// from it; rows per CTA 1/4; unroll 1 and the deepest feasible), the widest vector of the point's stage, every stage
// and reduction mode.
bool on_coarse_grid(const rt_shape& s, const rt_params& p, int widest_vec, bool deepest_unroll)
{
    const int lt = level_of(kTpr, 6, p.threads_per_row) - centre_level(s, p, widest_vec);
    const int lr = level_of(kRpc, 4, p.rows_per_cta), lu = level_of(kUnr, 3, p.unroll);
    // the two ends of the unroll axis: 1, and the deepest unroll that is feasible beside these other parameters
    // (4 where a thread owns that many vectors; with wide vectors and many threads per row it is 2, and the
    // step from 1 to 2 can be the steepest of the whole space)
    return (lt % 2 == 0) && (lr % 2 == 0) && (lu == 0 || deepest_unroll) && p.vec_bytes == widest_vec;
}

// When the budget cannot cover the whole coarse grid, the part that is evaluated must still touch every
// stage x reduction mode: the grid points are ordered mode by mode in rounds - first every mode's point
// nearest its centre (the centre level of threads per row, one row per CTA, unroll 1), then every mode's
// second nearest, and so on - and the first `keep` of that order are taken.
std::vector<int> stratified(const rt_shape& s, const std::vector<int>& coarse, const std::vector<rt_params>& cand, int keep)
{
    if (keep <= 0) return {};
    if ((int)coarse.size() <= keep) return coarse;
    auto mode_of = [](const rt_params& p) { return (p.reduce * 16 + p.cluster_size) * 4 + p.stage; };
    auto off_centre = [&](const rt_params& p) {
        return 2 * abs(level_of(kTpr, 6, p.threads_per_row) - centre_level(s, p, p.vec_bytes)) + level_of(kRpc, 4, p.rows_per_cta) +
               level_of(kUnr, 3, p.unroll);
    };
    std::vector<int> order = coarse;
    std::stable_sort(order.begin(), order.end(), [&](int x, int y) {
        const int mx = mode_of(cand[x]), my = mode_of(cand[y]);
        if (mx != my) return mx < my;
        return off_centre(cand[x]) < off_centre(cand[y]);
    });
    // rank of each point inside its mode, then round-robin over the modes
    std::vector<std::pair<int, int>> keyed;  // (rank in mode, position in `order`)
    int rank = 0;
    for (size_t i = 0; i < order.size(); ++i) {
        rank = (i > 0 && mode_of(cand[order[i]]) == mode_of(cand[order[i - 1]])) ? rank + 1 : 0;
        keyed.push_back({rank, (int)i});
    }
    std::stable_sort(keyed.begin(), keyed.end(), [](const std::pair<int, int>& x, const std::pair<int, int>& y) {
        return x.first < y.first;
    });
    std::vector<int> out;
    for (int i = 0; i < keep; ++i) out.push_back(order[keyed[i].second]);
    return out;
}

int run_search(const rt_shape& shape, const rt_limits& limits, const rt_budget& b, Evaluator& ev, rt_result* out,
               rt_eval_record* log, int32_t log_cap)
{
    memset(out, 0, sizeof(*out));
    if (b.max_evals < 1) {
        set_error("max_evals = %d allows no evaluation", b.max_evals);
        return RT_ERR_BUDGET;
    }
    std::vector<rt_params> feasible;
    int st = derive_feasible(shape, limits, b.heuristics, &feasible, nullptr);
    if (st != RT_OK) return st;
    if (feasible.empty()) {
        set_error("the feasible set is empty for this shape");
        return RT_ERR_INFEASIBLE;
    }
    SearchState S;
    S.ev = &ev;
    S.max_evals = b.max_evals;
    S.log = log;
    S.log_cap = log ? log_cap : 0;
    for (const rt_params& p : feasible) S.add(p);
    out->n_candidates = (int32_t)feasible.size();

    const int top_k = std::max(0, std::min<int>(b.top_k, b.max_evals / 4));  // re-tests are part of the budget
    float t;

    if (b.strategy == RT_SEARCH_EXHAUSTIVE) {
        for (int i = 0; i < (int)S.cand.size() && S.budget_left(top_k); ++i) {
            st = S.run(i, RT_PHASE_SWEEP, &t);
            if (st != RT_OK) return st;
            S.time_us[i] = t;
        }
    } else {
        // 1. seeds: configurations found on other shapes, if they are feasible here
        for (int k = 0; k < b.n_seeds && b.seeds && S.budget_left(top_k); ++k) {
            Plan plan;
            if (make_plan(&shape, &b.seeds[k], &limits, &plan) != RT_OK) continue;
            const int idx = S.add(b.seeds[k]);
            if (S.time_us[idx] >= 0.f) continue;
            st = S.run(idx, RT_PHASE_SEED, &t);
            if (st != RT_OK) return st;
            S.time_us[idx] = t;
        }
        // 2. coarse grid, cut to half of what is left of the budget (mode by mode, nearest each mode's centre first)
        int widest[RT_STAGE_TMA_PIPELINE + 1] = {0, 0, 0, 0, 0};  // per stage: the ragged-row stage is wider than the others
        for (const rt_params& p : feasible) widest[p.stage] = std::max(widest[p.stage], p.vec_bytes);
        std::vector<int> coarse;
        for (int i = 0; i < (int)feasible.size(); ++i) {
            bool deepest = true;  // no feasible point with these parameters and a deeper unroll
            for (int u = S.cand[i].unroll * 2; u <= 4 && deepest; u *= 2) {
                rt_params q = S.cand[i];
                q.unroll = u;
                if (S.index.find(pack_params(q)) != S.index.end()) deepest = false;
            }
            if (on_coarse_grid(shape, S.cand[i], widest[S.cand[i].stage], deepest)) coarse.push_back(i);
        }
        if (coarse.empty())
            for (int i = 0; i < (int)feasible.size(); ++i) coarse.push_back(i);
        const int grid_budget = std::max(1, (S.max_evals - top_k - S.used) / 2);
        for (int idx : stratified(shape, coarse, S.cand, grid_budget)) {
            if (!S.budget_left(top_k)) break;
            if (S.time_us[idx] >= 0.f) continue;
            st = S.run(idx, RT_PHASE_GRID, &t);
            if (st != RT_OK) return st;
            S.time_us[idx] = t;
        }
        // 3. best-first hill-climb: expand the neighbours of the fastest point not yet expanded, among
        //    the three fastest found so far (and the stage leaders, below).  When those are all expanded and budget is left, the frontier
        //    widens by three at a time (up to the twelve fastest): an optimum two steps away from every
        //    leader - a narrower vector that only pays with a deeper unroll, say - is reached through a
        //    runner-up.  Stops when the widest frontier is expanded or the budget is spent.
        int frontier = 3;
        while (S.budget_left(top_k)) {
            std::vector<int> order;
            for (int i = 0; i < (int)S.cand.size(); ++i)
                if (S.time_us[i] >= 0.f && isfinite(S.time_us[i])) order.push_back(i);
            std::sort(order.begin(), order.end(), [&](int a, int c) { return S.time_us[a] < S.time_us[c]; });
            // the stages are separate basins, and the coarse grid may have met one of them only two levels away from
            // its optimum: after the leader itself, the fastest point of every stage is climbed from once while it is
            // within 3 % of the leader; then the rest of the `frontier` fastest points
            int pick = -1;
            if (!order.empty() && !S.expanded[order[0]]) pick = order[0];
            bool seen[RT_STAGE_TMA_PIPELINE + 1] = {false, false, false, false, false};
            for (int k = 0; k < (int)order.size() && pick < 0; ++k) {
                if (S.time_us[order[k]] > kStageLeaderMargin * S.time_us[order[0]]) break;
                const int s = S.cand[order[k]].stage;
                if (!seen[s] && !S.expanded[order[k]]) pick = order[k];
                seen[s] = true;
            }
            for (int k = 0; k < (int)order.size() && k < frontier && pick < 0; ++k)
                if (!S.expanded[order[k]]) pick = order[k];
            if (pick < 0) {
                if (frontier >= 12 || frontier >= (int)order.size()) break;
                frontier += 3;
                continue;
            }
            S.expanded[pick] = 1;
            for (int nb : S.neighbours(pick)) {
                if (!S.budget_left(top_k)) break;
                if (S.time_us[nb] >= 0.f) continue;
                st = S.run(nb, RT_PHASE_CLIMB, &t);
                if (st != RT_OK) return st;
                S.time_us[nb] = t;
            }
        }
    }

    // 4. Top-K confirmation re-test ("Tuning agent": the finalists are measured again before the winner is
    //    declared).  The K fastest are re-timed together (on the device: interleaved block by block, so that they
    //    share one clock regime) and the winner is the fastest of those that pass again; a finalist that fails
    //    its re-test - a gate that passes once and fails once is what the re-test is there to catch - drops out,
    //    and while budget remains the next runner-up is re-tested in its place.
    std::vector<int> order;
    for (int i = 0; i < (int)S.cand.size(); ++i)
        if (S.time_us[i] >= 0.f && isfinite(S.time_us[i])) order.push_back(i);
    std::sort(order.begin(), order.end(), [&](int a, int c) { return S.time_us[a] < S.time_us[c]; });
    std::vector<int> confirmed;
    std::vector<float> first_us = S.time_us;  // the times the finalists were ranked by, before their re-test replaces them
    size_t next = 0;
    int want = top_k;
    for (int pass = 0; pass < 2 && want > 0; ++pass) {
        std::vector<int> batch;
        while (next < order.size() && (int)batch.size() < want && S.used + (int)batch.size() < S.max_evals)
            batch.push_back(order[next++]);
        if (batch.empty()) break;
        std::vector<rt_params> ps;
        for (int idx : batch) ps.push_back(S.cand[idx]);
        std::vector<rt_eval_record> recs(batch.size());
        st = ev.retest(ps.data(), (int)ps.size(), recs.data());
        int dropped = 0;
        for (size_t k = 0; k < batch.size(); ++k) {
            rt_eval_record& rec = recs[k];
            rec.phase = RT_PHASE_TOPK;
            rec.eval_index = S.used++;
            if (S.log && S.n_log < S.log_cap) S.log[S.n_log++] = rec;
            if (st != RT_OK) continue;
            if (rec.status != RT_OK) {
                ++S.failed;
                ++dropped;
                S.time_us[batch[k]] = INFINITY;
            } else {
                S.time_us[batch[k]] = ev.retest_replaces() ? rec.us : 0.5f * (S.time_us[batch[k]] + rec.us);
                confirmed.push_back(batch[k]);
            }
        }
        if (st != RT_OK) return st;
        want = dropped;
    }
    int best = -1;
    for (int i : confirmed.empty() ? order : confirmed)
        if (isfinite(S.time_us[i]) && (best < 0 || S.time_us[i] < S.time_us[best])) best = i;
    // A re-test that cannot separate two finalists does not overturn their first ranking: among the confirmed finalists
    // within kRetestTie of the fastest re-test time, the one that was faster when the search first timed it wins (a
    // configuration can read 3-4 % slow for the length of one re-test - where its CTAs landed - and then lose a
    // photo finish to a point it leads by that much everywhere else).
    if (best >= 0 && !confirmed.empty()) {
        const float limit = S.time_us[best] * kRetestTie;
        for (int i : confirmed)
            if (isfinite(S.time_us[i]) && S.time_us[i] <= limit && first_us[i] >= 0.f && first_us[i] < first_us[best]) best = i;
    }

    out->evals_used = S.used;
    out->n_log = S.n_log;
    out->n_failed_gate = S.failed;
    if (best < 0) {
        set_error("no candidate passed the correctness gate (%d evaluated)", S.used);
        return RT_ERR_MISMATCH;
    }
    out->best = S.cand[best];
    out->best_us = S.time_us[best];
    return RT_OK;
}

int check_workspace(const rt_shape* s, const rt_workspace* ws)
{
    if (!s || !ws) {
        set_error("shape or workspace is NULL");
        return RT_ERR_NULL;
    }
    const bool is_silu = s->op == RT_OP_SILU_AND_MUL;
    if (!ws->x || !ws->y || !ws->y_ref || (!is_silu && (!ws->r || !ws->w || !ws->r_out || !ws->r_ref)) ||
        (s->op == RT_OP_MERGE_ATTN_STATES && !ws->aux) || (s->op == RT_OP_ADD_RMSNORM_FP8 && (!ws->aux_out || !ws->aux_ref))) {
        set_error("a workspace pointer is NULL");
        return RT_ERR_NULL;
    }
    if (s->n_tokens < 1 || ws->n_ref_tokens < 1 || ws->n_ref_tokens > s->n_tokens) {
        set_error("n_ref_tokens=%lld must lie in 1..n_tokens=%lld", (long long)ws->n_ref_tokens, (long long)s->n_tokens);
        return RT_ERR_SHAPE;
    }
    if (ws->x == ws->y || (!is_silu && ws->r == ws->r_out)) {
        set_error("the tuner's workspace must not alias inputs and outputs (launches repeat)");
        return RT_ERR_SHAPE;
    }
    if (ws->ring_sets > 1 && ws->ring_stride_bytes <= 0) {
        set_error("ring_sets=%d needs a positive ring_stride_bytes", ws->ring_sets);
        return RT_ERR_SHAPE;
    }
    // the comparison kernels read 32-bit words
    if (((uintptr_t)ws->y | (uintptr_t)ws->y_ref | (uintptr_t)ws->r_out | (uintptr_t)ws->r_ref | (uintptr_t)ws->aux_out |
         (uintptr_t)ws->aux_ref) & 3u) {
        set_error("outputs and references must be 4-byte aligned");
        return RT_ERR_ALIGN;
    }
    return RT_OK;
}

// The alignment every address the evaluator will hand to a kernel is known to have: the caller's claim
// (rt_shape.min_ptr_align) cut down to what the workspace pointers, the ring stride and the offsets derived from
// them (the parts of the all-reduce-fused norm, the byte-wide codes of the fp8-output norm) really share.  The
// feasible set and every plan are derived from this value, so a sliced tensor or an odd ring stride narrows the
// vectors or refuses the TMA stages instead of launching a misaligned access.
int32_t effective_alignment(const rt_shape& s, const rt_workspace& ws)
{
    const int eb = elem_bytes_of(s.dtype);
    uintptr_t bits = (uintptr_t)ws.x | (uintptr_t)ws.y | 256u;
    const bool vectors_in_r = s.op != RT_OP_SILU_AND_MUL;
    if (vectors_in_r) bits |= (uintptr_t)ws.r;
    if (s.op == RT_OP_ADD_RMSNORM_FP8) {
        // q leaves as vectors half as wide as those of x: its alignment counts double
        bits = ((uintptr_t)ws.x | (uintptr_t)ws.r | (uintptr_t)ws.w | (uintptr_t)ws.r_out | ((uintptr_t)ws.y << 1) | 256u);
    } else if (s.op != RT_OP_MERGE_ATTN_STATES && s.op != RT_OP_SILU_AND_MUL) {
        bits |= (uintptr_t)ws.w | (uintptr_t)ws.r_out;  // merge_attn_states: w and r_out are binary32 scalars per head
    }
    if (ws.ring_sets > 1) {
        bits |= (uintptr_t)ws.ring_stride_bytes;
        if (s.op == RT_OP_ADD_RMSNORM_FP8) bits |= (uintptr_t)(ws.ring_stride_bytes / eb) << 1;
    }
    if (s.op == RT_OP_ADD_RMSNORM_ALLREDUCE) bits |= (uintptr_t)((uint64_t)s.n_tokens * (uint64_t)s.hidden * eb);
    const int32_t have = (int32_t)(bits & (~bits + 1));
    return std::min<int32_t>(s.min_ptr_align > 0 ? s.min_ptr_align : 1, have);
}

rt_budget normalised(const rt_budget* b)
{
    rt_budget n = *b;
    if (n.warmup < 0) n.warmup = 0;
    if (n.iters < 1) n.iters = 1;
    if (n.repeats < 1) n.repeats = 1;
    if (n.preheat_ms < 0) n.preheat_ms = 0;
    if (n.preheat_ms > 5000) n.preheat_ms = 5000;
    return n;
}

}  // namespace
}  // namespace rt

// ---- C ABI -------------------------------------------------------------------------------------------

extern "C" {

int tuner_compare(const void* got, const void* ref, int64_t n, int dtype, int mode, double tol, double* max_err,
                  int64_t* n_bad, void* stream)
{
    std::lock_guard<std::mutex> serial(rt::g_compare_mutex);
    int st = rt::check_compare_args(got, ref, n, dtype, mode);
    if (st != RT_OK) return st;
    if (!max_err || !n_bad) {
        rt::set_error("tuner_compare: NULL result pointer");
        return RT_ERR_NULL;
    }
    *max_err = 0.0;
    *n_bad = 0;
    if (n == 0) return RT_OK;
    rt::Scratch* sc;
    st = rt::get_scratch(&sc);
    if (st != RT_OK) return st;
    cudaStream_t s = (cudaStream_t)stream;
    RT_CUDA_OK(cudaMemsetAsync(sc->dev, 0, sizeof(rt::CompareAcc), s));
    st = rt::enqueue_compare(got, ref, n, dtype, mode, tol, sc->dev, s);
    if (st != RT_OK) return st;
    RT_CUDA_OK(cudaMemcpyAsync(sc->host, sc->dev, sizeof(rt::CompareAcc), cudaMemcpyDeviceToHost, s));
    RT_CUDA_OK(cudaStreamSynchronize(s));
    *max_err = rt::acc_max_err(sc->host[0], mode);
    *n_bad = (int64_t)sc->host[0].n_bad;
    return RT_OK;
}

int tuner_compare_e4m3(const void* got, const void* ref, int64_t n, int32_t tol_steps, int32_t* max_steps, int64_t* n_bad,
                       void* stream)
{
    std::lock_guard<std::mutex> serial(rt::g_compare_mutex);
    if (!got || !ref || !max_steps || !n_bad) {
        rt::set_error("tuner_compare_e4m3: NULL argument");
        return RT_ERR_NULL;
    }
    if (n < 0) {
        rt::set_error("n = %lld is negative", (long long)n);
        return RT_ERR_SHAPE;
    }
    *max_steps = 0;
    *n_bad = 0;
    if (n == 0) return RT_OK;
    rt::Scratch* sc;
    int st = rt::get_scratch(&sc);
    if (st != RT_OK) return st;
    cudaStream_t s = (cudaStream_t)stream;
    RT_CUDA_OK(cudaMemsetAsync(sc->dev, 0, sizeof(rt::CompareAcc), s));
    st = rt::enqueue_compare_e4m3(got, ref, n, tol_steps, sc->dev, s);
    if (st != RT_OK) return st;
    RT_CUDA_OK(cudaMemcpyAsync(sc->host, sc->dev, sizeof(rt::CompareAcc), cudaMemcpyDeviceToHost, s));
    RT_CUDA_OK(cudaStreamSynchronize(s));
    *max_steps = (int32_t)sc->host[0].max_bits;
    *n_bad = (int64_t)sc->host[0].n_bad;
    return RT_OK;
}

int tuner_compare_mixed(const void* got, const void* ref, int64_t n, int dtype, double tol, double tol_abs,
                        double* max_abs, int64_t* n_bad, void* stream)
{
    std::lock_guard<std::mutex> serial(rt::g_compare_mutex);
    int st = rt::check_compare_args(got, ref, n, dtype, RT_CMP_BITS);
    if (st != RT_OK) return st;
    if (!max_abs || !n_bad) {
        rt::set_error("tuner_compare_mixed: NULL result pointer");
        return RT_ERR_NULL;
    }
    *max_abs = 0.0;
    *n_bad = 0;
    if (n == 0) return RT_OK;
    rt::Scratch* sc;
    st = rt::get_scratch(&sc);
    if (st != RT_OK) return st;
    cudaStream_t s = (cudaStream_t)stream;
    RT_CUDA_OK(cudaMemsetAsync(sc->dev, 0, sizeof(rt::CompareAcc), s));
    st = rt::enqueue_compare_mixed(got, ref, n, dtype, tol, tol_abs, sc->dev, s);
    if (st != RT_OK) return st;
    RT_CUDA_OK(cudaMemcpyAsync(sc->host, sc->dev, sizeof(rt::CompareAcc), cudaMemcpyDeviceToHost, s));
    RT_CUDA_OK(cudaStreamSynchronize(s));
    *max_abs = rt::acc_max_err(sc->host[0], RT_CMP_REL32);
    *n_bad = (int64_t)sc->host[0].n_bad;
    return RT_OK;
}

int tuner_compare_static(const void* got, const void* ref, int64_t n, int dtype, int mode, double tol, double* max_err,
                         int64_t* n_bad, void* stream)
{
    int st = rt::check_compare_args(got, ref, n, dtype, mode);
    if (st != RT_OK) return st;
    if (!max_err || !n_bad) {
        rt::set_error("tuner_compare_static: NULL result pointer");
        return RT_ERR_NULL;
    }
    if (n > rt::kStaticCompareMaxElems) {
        rt::set_error("tuner_compare_static: n = %lld exceeds the limit of %lld elements", (long long)n,
                      (long long)rt::kStaticCompareMaxElems);
        return RT_ERR_CAPACITY;
    }
    *max_err = 0.0;
    *n_bad = 0;
    if (n == 0) return RT_OK;
    rt::CompareAcc* acc = nullptr;
    st = rt::static_scratch(&acc);
    if (st != RT_OK) return st;
    cudaStream_t s = (cudaStream_t)stream;
    // The record still holds the previous call's result: clear it on the same stream first.
    RT_CUDA_OK(cudaMemsetAsync(acc, 0, sizeof(rt::CompareAcc), s));
    st = rt::enqueue_compare(got, ref, n, dtype, mode, tol, acc, s);
    if (st != RT_OK) return st;
    rt::CompareAcc result;
    RT_CUDA_OK(cudaMemcpyAsync(&result, acc, sizeof(result), cudaMemcpyDeviceToHost, s));
    RT_CUDA_OK(cudaStreamSynchronize(s));
    *max_err = rt::acc_max_err(result, mode);
    *n_bad = (int64_t)result.n_bad;
    return RT_OK;
}

int tuner_evaluate(const rt_shape* s, const rt_params* p, const rt_budget* b, const rt_workspace* ws, rt_eval_record* out)
{
    if (!p || !b || !out) {
        rt::set_error("tuner_evaluate: NULL argument");
        return RT_ERR_NULL;
    }
    int st = rt::check_workspace(s, ws);
    if (st != RT_OK) return st;
    rt::DeviceEvaluator ev;
    ev.shape = *s;
    ev.shape.min_ptr_align = rt::effective_alignment(*s, *ws);
    ev.budget = rt::normalised(b);
    ev.ws = *ws;
    st = rt::current_limits(&ev.limits);
    if (st != RT_OK) return st;
    return ev.evaluate(*p, out);
}

int tuner_retest_interleaved(const rt_shape* s, const rt_params* thetas, int32_t n_thetas, const rt_budget* b,
                             const rt_workspace* ws, int32_t rounds, rt_eval_record* out, rt_block_record* blocks,
                             int32_t* n_blocks)
{
    if (!thetas || !b || !out) {
        rt::set_error("tuner_retest_interleaved: NULL argument");
        return RT_ERR_NULL;
    }
    if (n_thetas < 1 || rounds < 1) {
        rt::set_error("tuner_retest_interleaved: n_thetas=%d and rounds=%d must be positive", n_thetas, rounds);
        return RT_ERR_BUDGET;
    }
    int st = rt::check_workspace(s, ws);
    if (st != RT_OK) return st;
    rt::DeviceEvaluator ev;
    ev.shape = *s;
    ev.shape.min_ptr_align = rt::effective_alignment(*s, *ws);
    ev.budget = rt::normalised(b);
    ev.ws = *ws;
    st = rt::current_limits(&ev.limits);
    if (st != RT_OK) return st;
    if (blocks) memset(blocks, 0, sizeof(rt_block_record) * (size_t)rounds * (size_t)n_thetas);
    int ran = 0;
    st = ev.interleaved(thetas, n_thetas, rounds, out, blocks, &ran);
    if (n_blocks) *n_blocks = ran;
    return st;
}

int tuner_search(const rt_shape* s, const rt_budget* b, const rt_workspace* ws, rt_result* out, rt_eval_record* log,
                 int32_t log_cap)
{
    if (!b || !out) {
        rt::set_error("tuner_search: NULL argument");
        return RT_ERR_NULL;
    }
    int st = rt::check_workspace(s, ws);
    if (st != RT_OK) return st;
    rt::DeviceEvaluator ev;
    ev.shape = *s;
    ev.shape.min_ptr_align = rt::effective_alignment(*s, *ws);
    ev.budget = rt::normalised(b);
    ev.ws = *ws;
    st = rt::current_limits(&ev.limits);
    if (st != RT_OK) return st;
    return rt::run_search(ev.shape, ev.limits, ev.budget, ev, out, log, log_cap);
}

int tuner_search_with(const rt_shape* s, const rt_limits* limits, const rt_budget* b, rt_evaluate_fn evaluate, void* user,
                      rt_result* out, rt_eval_record* log, int32_t log_cap)
{
    if (!s || !limits || !b || !evaluate || !out) {
        rt::set_error("tuner_search_with: NULL argument");
        return RT_ERR_NULL;
    }
    rt::CallbackEvaluator ev;
    ev.fn = evaluate;
    ev.user = user;
    return rt::run_search(*s, *limits, rt::normalised(b), ev, out, log, log_cap);
}

int tuner_launch_floor(const rt_budget* b, void* stream, float* us)
{
    if (!b || !us) {
        rt::set_error("tuner_launch_floor: NULL argument");
        return RT_ERR_NULL;
    }
    return rt::time_launch_floor(rt::normalised(b), (cudaStream_t)stream, us);
}

void rt_shutdown(void)
{
    rt::host_pipe_shutdown();
    std::lock_guard<std::mutex> serial(rt::g_compare_mutex);
    std::lock_guard<std::mutex> lock(rt::g_scratch_mutex);
    for (rt::Scratch& s : rt::g_scratch) {
        if (s.dev) cudaFree(s.dev);
        if (s.host) cudaFreeHost(s.host);
        s.dev = nullptr;
        s.host = nullptr;
    }
}

}  // extern "C"
