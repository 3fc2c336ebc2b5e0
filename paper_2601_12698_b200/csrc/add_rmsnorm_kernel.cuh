// Fused residual-add + RMSNorm as one explicitly parameterised kernel template (sm_100a).
//
// The template is the "parameterizable template" S~ of the paper's Algorithm 1 (Level 2) for the
// kernel `fused_add_rmsnorm`; its axes are the execution-strategy dimensions named in "Tuning
// parameter selection and search space derivation": thread-level granularity (threads per row,
// rows per CTA: run-time block shape), vectorisation (VB bytes per ld/st: 32 - the 256-bit global accesses
// of sm_100 -, 16 or 8), unrolling (U independent
// loads in flight), and the organisation of shared memory and registers (STAGE, REDUCE).
//
// Compile-time axes: element type, VB, STAGE, REDUCE, U and - for the two register stages - CAP, the
// number of row vectors one thread keeps.  Run-time axes: blockDim.x = threads per row,
// blockDim.y = rows per CTA, cluster size.  In the persistent pipeline stage U is the depth of the ring of
// shared-memory stages ("loop scheduling"): the grid is as large as the device keeps resident, and a CTA walks
// over row blocks with the bulk copies of its next U - 1 blocks in flight.
//
// Per row:  s = fp32(x) + fp32(r);  r_out = rn(s);  y = rn(s * rsqrt(mean(s^2) + eps) * w).
// The sum of squares is combined in a fixed order (no atomics): results are deterministic.
#pragma once

#include <cuda_bf16.h>
#include <cuda_fp16.h>
#include <stddef.h>
#include <stdint.h>

#include <type_traits>

namespace rt {

constexpr int kStageReg = 0;
constexpr int kStageSmemLdg = 1;
constexpr int kStageSmemTma = 2;
constexpr int kStageRegRealign = 3;
constexpr int kStageTmaPipeline = 4;
constexpr int kMaxPipelineDepth = 4;
constexpr int kReduceShfl = 0;
constexpr int kReduceSmem = 1;
constexpr int kReduceCluster = 2;

constexpr int kMaxRowsPerCta = 8;
constexpr int kMaxClusterSize = 8;
constexpr int kDeviceTimeoutCode = 9;           // written to the status word when a bounded wait expires
constexpr unsigned kMbarrierPollLimit = 1u << 24;        // polls of mbarrier.try_wait before giving up ...
constexpr long long kMbarrierCycleLimit = 2000000000LL;  // ... or about one second of SM clock, whichever is first

struct KernelArgs {
    const void* x;
    const void* r;
    const void* w;
    void* y;
    void* r_out;
    long long n_tokens;
    int hidden;
    int nvec;        // vectors of VB bytes in one row
    int slice_nvec;  // vectors of one row owned by one CTA (== nvec unless the row is split over a cluster)
    float eps;
    int* status;     // device status word
    unsigned wait_polls;  // polls a bounded mbarrier wait may take (kMbarrierPollLimit unless the caller lowered it)
    int drop_copies;      // diagnostic: 1 = the TMA stages post no copy, so their waits run out and report it
    unsigned long long* trace;  // instrumented instances only: kTraceWords words per CTA
};

// Phase stamps of the instrumented instances (TRACE = true): SM cycle counts taken by the CTA's first thread at entry,
// after the wait for the previous kernel, when its share of x and r has arrived and been summed, after the row
// reduction, and after its last store was issued; plus the global nanosecond timer at entry and exit and the SM
// the CTA ran on.  Kept in registers and written once at the end, so that the stamps disturb the kernel as little
// as a stamp can.  With TRACE = false every member is empty and compiles to nothing.
constexpr int kTraceWords = 8;
enum { kTraceEntry = 0, kTraceReleased = 1, kTraceLoaded = 2, kTraceReduced = 3, kTraceStored = 4 };
template <bool TRACE>
struct PhaseTrace {
    long long cycles[TRACE ? 5 : 1];
    unsigned long long ns_entry;
    __device__ __forceinline__ void begin()
    {
        if constexpr (TRACE) {
#pragma unroll
            for (int k = 0; k < 5; ++k) cycles[k] = 0;
            asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(ns_entry));
            cycles[kTraceEntry] = clock64();
        }
    }
    __device__ __forceinline__ void mark(int phase)
    {
        if constexpr (TRACE) cycles[phase] = clock64();
    }
    __device__ __forceinline__ void flush(const KernelArgs& a)
    {
        if constexpr (TRACE) {
            if (threadIdx.x == 0 && threadIdx.y == 0 && a.trace) {
                unsigned long long ns_exit;
                unsigned smid;
                asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(ns_exit));
                asm volatile("mov.u32 %0, %%smid;" : "=r"(smid));
                unsigned long long* out = a.trace + (size_t)blockIdx.x * kTraceWords;
                out[0] = ns_entry;
#pragma unroll
                for (int k = 0; k < 5; ++k) out[1 + k] = (unsigned long long)cycles[k];
                out[6] = ns_exit;
                out[7] = smid;
            }
        }
    }
};

// ---- vectors of VB bytes ------------------------------------------------------------------------

template <int VB>
struct Vec {
    uint32_t w[(VB + 3) / 4];  // VB == 2 uses the low half of w[0]
};

// Streaming loads of x and r: read once, keep them out of L1.  Volatile, so that the order of
// global loads and stores in the program is the order in the instruction stream: a batch of U loads
// is issued together, and the next batch is not hoisted above this batch's stores.
template <int VB>
__device__ __forceinline__ Vec<VB> ld_stream(const void* p)
{
    Vec<VB> v;
    if constexpr (VB == 32) {
        asm volatile("ld.global.L1::no_allocate.v8.u32 {%0,%1,%2,%3,%4,%5,%6,%7}, [%8];"
                     : "=r"(v.w[0]), "=r"(v.w[1]), "=r"(v.w[2]), "=r"(v.w[3]), "=r"(v.w[4]), "=r"(v.w[5]), "=r"(v.w[6]),
                       "=r"(v.w[7]) : "l"(p));
    } else if constexpr (VB == 16) {
        asm volatile("ld.global.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];"
                     : "=r"(v.w[0]), "=r"(v.w[1]), "=r"(v.w[2]), "=r"(v.w[3]) : "l"(p));
    } else if constexpr (VB == 8) {
        asm volatile("ld.global.L1::no_allocate.v2.u32 {%0,%1}, [%2];" : "=r"(v.w[0]), "=r"(v.w[1]) : "l"(p));
    } else if constexpr (VB == 4) {
        asm volatile("ld.global.L1::no_allocate.u32 %0, [%1];" : "=r"(v.w[0]) : "l"(p));
    } else {
        unsigned short h;
        asm volatile("ld.global.L1::no_allocate.u16 %0, [%1];" : "=h"(h) : "l"(p));
        v.w[0] = h;
    }
    return v;
}

// Stores of r_out and y.  EVICT_FIRST marks the written lines as the first to leave L2 (st.global.cs): the
// outputs are not read again by this kernel, and measured on B200 this is 1-3% faster where x and r come in
// through ld.global, but not where they come in through TMA bulk copies - so the stage decides.
template <int VB, bool EVICT_FIRST = false>
__device__ __forceinline__ void st_stream(void* p, const Vec<VB>& v)
{
    if constexpr (VB == 32 && EVICT_FIRST) {
        asm volatile("st.global.cs.v8.u32 [%0], {%1,%2,%3,%4,%5,%6,%7,%8};" ::"l"(p), "r"(v.w[0]), "r"(v.w[1]), "r"(v.w[2]),
                     "r"(v.w[3]), "r"(v.w[4]), "r"(v.w[5]), "r"(v.w[6]), "r"(v.w[7]) : "memory");
    } else if constexpr (VB == 32) {
        asm volatile("st.global.v8.u32 [%0], {%1,%2,%3,%4,%5,%6,%7,%8};" ::"l"(p), "r"(v.w[0]), "r"(v.w[1]), "r"(v.w[2]),
                     "r"(v.w[3]), "r"(v.w[4]), "r"(v.w[5]), "r"(v.w[6]), "r"(v.w[7]) : "memory");
    } else if constexpr (VB == 16 && EVICT_FIRST) {
        asm volatile("st.global.cs.v4.u32 [%0], {%1,%2,%3,%4};" ::"l"(p), "r"(v.w[0]), "r"(v.w[1]), "r"(v.w[2]),
                     "r"(v.w[3]) : "memory");
    } else if constexpr (VB == 8 && EVICT_FIRST) {
        asm volatile("st.global.cs.v2.u32 [%0], {%1,%2};" ::"l"(p), "r"(v.w[0]), "r"(v.w[1]) : "memory");
    } else if constexpr (VB == 16) {
        asm volatile("st.global.v4.u32 [%0], {%1,%2,%3,%4};" ::"l"(p), "r"(v.w[0]), "r"(v.w[1]), "r"(v.w[2]),
                     "r"(v.w[3]) : "memory");
    } else if constexpr (VB == 8) {
        asm volatile("st.global.v2.u32 [%0], {%1,%2};" ::"l"(p), "r"(v.w[0]), "r"(v.w[1]) : "memory");
    } else if constexpr (VB == 4) {
        asm volatile("st.global.u32 [%0], %1;" ::"l"(p), "r"(v.w[0]) : "memory");
    } else {
        asm volatile("st.global.u16 [%0], %1;" ::"l"(p), "h"((unsigned short)v.w[0]) : "memory");
    }
}

// The weight vector is shared by every row: read-only path, cached.
template <int VB>
__device__ __forceinline__ Vec<VB> ld_weight(const void* p)
{
    Vec<VB> v;
    if constexpr (VB == 32) {
        const uint4 q = __ldg(reinterpret_cast<const uint4*>(p)), h = __ldg(reinterpret_cast<const uint4*>(p) + 1);
        v.w[0] = q.x; v.w[1] = q.y; v.w[2] = q.z; v.w[3] = q.w;
        v.w[4] = h.x; v.w[5] = h.y; v.w[6] = h.z; v.w[7] = h.w;
    } else if constexpr (VB == 16) {
        const uint4 q = __ldg(reinterpret_cast<const uint4*>(p));
        v.w[0] = q.x; v.w[1] = q.y; v.w[2] = q.z; v.w[3] = q.w;
    } else if constexpr (VB == 8) {
        const uint2 q = __ldg(reinterpret_cast<const uint2*>(p));
        v.w[0] = q.x; v.w[1] = q.y;
    } else if constexpr (VB == 4) {
        v.w[0] = __ldg(reinterpret_cast<const unsigned int*>(p));
    } else {
        v.w[0] = __ldg(reinterpret_cast<const unsigned short*>(p));
    }
    return v;
}

// The same load pinned in program order (volatile): used to put the weight fetch ahead of the row
// reduction, so that its latency overlaps the barrier instead of following it.
template <int VB>
__device__ __forceinline__ Vec<VB> ld_weight_early(const void* p)
{
    Vec<VB> v;
    if constexpr (VB == 32) {
        asm volatile("ld.global.nc.v4.u32 {%0,%1,%2,%3}, [%4];"
                     : "=r"(v.w[0]), "=r"(v.w[1]), "=r"(v.w[2]), "=r"(v.w[3]) : "l"(p));
        asm volatile("ld.global.nc.v4.u32 {%0,%1,%2,%3}, [%4];"
                     : "=r"(v.w[4]), "=r"(v.w[5]), "=r"(v.w[6]), "=r"(v.w[7]) : "l"(reinterpret_cast<const unsigned char*>(p) + 16));
    } else if constexpr (VB == 16) {
        asm volatile("ld.global.nc.v4.u32 {%0,%1,%2,%3}, [%4];"
                     : "=r"(v.w[0]), "=r"(v.w[1]), "=r"(v.w[2]), "=r"(v.w[3]) : "l"(p));
    } else if constexpr (VB == 8) {
        asm volatile("ld.global.nc.v2.u32 {%0,%1}, [%2];" : "=r"(v.w[0]), "=r"(v.w[1]) : "l"(p));
    } else if constexpr (VB == 4) {
        asm volatile("ld.global.nc.u32 %0, [%1];" : "=r"(v.w[0]) : "l"(p));
    } else {
        unsigned short h;
        asm volatile("ld.global.nc.u16 %0, [%1];" : "=h"(h) : "l"(p));
        v.w[0] = h;
    }
    return v;
}

template <int VB>
__device__ __forceinline__ Vec<VB> ld_shared(const void* p)
{
    Vec<VB> v;
    if constexpr (VB == 32) {
        const uint4 q = *reinterpret_cast<const uint4*>(p), h = *(reinterpret_cast<const uint4*>(p) + 1);
        v.w[0] = q.x; v.w[1] = q.y; v.w[2] = q.z; v.w[3] = q.w;
        v.w[4] = h.x; v.w[5] = h.y; v.w[6] = h.z; v.w[7] = h.w;
    } else if constexpr (VB == 16) {
        const uint4 q = *reinterpret_cast<const uint4*>(p);
        v.w[0] = q.x; v.w[1] = q.y; v.w[2] = q.z; v.w[3] = q.w;
    } else if constexpr (VB == 8) {
        const uint2 q = *reinterpret_cast<const uint2*>(p);
        v.w[0] = q.x; v.w[1] = q.y;
    } else if constexpr (VB == 4) {
        v.w[0] = *reinterpret_cast<const unsigned int*>(p);
    } else {
        v.w[0] = *reinterpret_cast<const unsigned short*>(p);
    }
    return v;
}

// ---- element codecs -----------------------------------------------------------------------------

template <typename T, int VB>
struct Codec {
    static constexpr int EPV = VB / (int)sizeof(T);
    static_assert(EPV >= 1, "vector narrower than one element");

    static __device__ __forceinline__ void unpack(const Vec<VB>& v, float (&f)[EPV])
    {
        if constexpr (sizeof(T) == 4) {
#pragma unroll
            for (int i = 0; i < EPV; ++i) f[i] = __uint_as_float(v.w[i]);
        } else if constexpr (EPV == 1) {
            f[0] = to_float16(v.w[0] & 0xFFFFu);
        } else {
#pragma unroll
            for (int i = 0; i < EPV / 2; ++i) {
                f[2 * i] = to_float16(v.w[i] & 0xFFFFu);
                f[2 * i + 1] = to_float16(v.w[i] >> 16);
            }
        }
    }

    static __device__ __forceinline__ Vec<VB> pack(const float (&f)[EPV])
    {
        Vec<VB> v;
        if constexpr (sizeof(T) == 4) {
#pragma unroll
            for (int i = 0; i < EPV; ++i) v.w[i] = __float_as_uint(f[i]);
        } else if constexpr (EPV == 1) {
            v.w[0] = from_float16(f[0]);
        } else {
#pragma unroll
            for (int i = 0; i < EPV / 2; ++i) v.w[i] = from_float16x2(f[2 * i], f[2 * i + 1]);
        }
        return v;
    }

    static __device__ __forceinline__ float to_float16(uint32_t bits)
    {
        if constexpr (sizeof(T) == 4) {
            return 0.f;
        } else if constexpr (std::is_same<T, __nv_bfloat16>::value) {
            return __uint_as_float(bits << 16);  // bf16 is the top half of a binary32
        } else {
            return __half2float(__ushort_as_half((unsigned short)bits));
        }
    }
    static __device__ __forceinline__ uint32_t from_float16(float a)  // round to nearest even
    {
        if constexpr (sizeof(T) == 4) {
            return 0u;
        } else if constexpr (std::is_same<T, __nv_bfloat16>::value) {
            return __bfloat16_as_ushort(__float2bfloat16_rn(a));
        } else {
            return __half_as_ushort(__float2half_rn(a));
        }
    }
    static __device__ __forceinline__ uint32_t from_float16x2(float lo, float hi)
    {
        if constexpr (sizeof(T) == 4) {
            return 0u;
        } else if constexpr (std::is_same<T, __nv_bfloat16>::value) {
            const __nv_bfloat162 p = __floats2bfloat162_rn(lo, hi);
            return *reinterpret_cast<const uint32_t*>(&p);
        } else {
            const __half2 p = __floats2half2_rn(lo, hi);
            return *reinterpret_cast<const uint32_t*>(&p);
        }
    }
};

// ---- ragged rows (STAGE == kStageRegRealign) -----------------------------------------------------
//
// A row whose byte length is not a multiple of the chunk width VB (16 or 32 bytes) starts at a different offset
// inside a chunk from one row to the next, so no vector that wide divides it.  This stage cuts the row at the
// VB-byte boundaries of the tensor instead: a head of fewer than EPV elements up to the first boundary, the whole
// aligned chunks (moved as VB-byte vectors, kept in registers like the register stage), and a tail of fewer than EPV
// elements.  Head and tail elements go one to a thread, so no byte outside the row is touched.  Only the weights are
// then out of step: the weights of a whole chunk start `phase` bytes past a 16-byte boundary of w, the same phase
// for every chunk of the row.

template <int VB, bool EARLY>
__device__ __forceinline__ Vec<VB> ld_weight_at(const void* p)
{
    if constexpr (EARLY) return ld_weight_early<VB>(p);
    else return ld_weight<VB>(p);
}

// out.w[k] = the 32-bit word that starts WS words and `sh` bits into the aligned words a[].
template <int NW, int WS>
__device__ __forceinline__ void shift_words(const uint32_t (&a)[NW + 4], uint32_t sh, uint32_t (&out)[NW])
{
#pragma unroll
    for (int k = 0; k < NW; ++k) out[k] = __funnelshift_r(a[k + WS], a[k + WS + 1], sh);
}

// VB bytes of w from address p (a multiple of the element size; `phase` = p modulo 16, the same for every chunk of
// a row).  phase = 0: aligned vectors.  Otherwise the VB / 16 + 1 aligned 16-byte vectors around p, shifted together
// (`whole_span`: all of them lie inside w), or - for the one chunk per row whose last vector would reach past the
// end of w - element by element.  EARLY pins the loads in program order, for a fetch ahead of the row reduction.
template <typename T, int VB, bool EARLY>
__device__ __forceinline__ Vec<VB> ld_weight_ragged(const unsigned char* p, int phase, bool whole_span)
{
    if (phase == 0) return ld_weight_at<VB, EARLY>(p);
    constexpr int NW = VB / 4;
    Vec<VB> v;
    if (!whole_span) {
        if constexpr (sizeof(T) == 4) {
#pragma unroll
            for (int k = 0; k < NW; ++k) v.w[k] = ld_weight_at<4, EARLY>(p + 4 * k).w[0];
        } else {
#pragma unroll
            for (int k = 0; k < NW; ++k)
                v.w[k] = ld_weight_at<2, EARLY>(p + 4 * k).w[0] | (ld_weight_at<2, EARLY>(p + 4 * k + 2).w[0] << 16);
        }
        return v;
    }
    uint32_t a[NW + 4];
#pragma unroll
    for (int q = 0; q < NW / 4 + 1; ++q) {
        const Vec<16> t = ld_weight_at<16, EARLY>(p - phase + 16 * q);
        a[4 * q] = t.w[0]; a[4 * q + 1] = t.w[1]; a[4 * q + 2] = t.w[2]; a[4 * q + 3] = t.w[3];
    }
    const uint32_t sh = (uint32_t)(phase & 3) * 8u;  // 0 or 16 bits inside a word
    switch (phase >> 2) {  // a branch that is uniform over the row keeps every register index static
        case 0: shift_words<NW, 0>(a, sh, v.w); break;
        case 1: shift_words<NW, 1>(a, sh, v.w); break;
        case 2: shift_words<NW, 2>(a, sh, v.w); break;
        default: shift_words<NW, 3>(a, sh, v.w); break;
    }
    return v;
}

// ---- synchronisation helpers --------------------------------------------------------------------

// Barrier over the threads of one row only (named barrier 1 + row); a warp-wide row needs no bar.
__device__ __forceinline__ void row_sync(int row_in_cta, int threads_per_row)
{
    if (threads_per_row == 32) {
        __syncwarp();
    } else {
        asm volatile("bar.sync %0, %1;" ::"r"(row_in_cta + 1), "r"(threads_per_row) : "memory");
    }
}

__device__ __forceinline__ uint32_t cluster_cta_rank()
{
    uint32_t v;
    asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(v));
    return v;
}
__device__ __forceinline__ uint32_t cluster_num_ctas()
{
    uint32_t v;
    asm volatile("mov.u32 %0, %%cluster_nctarank;" : "=r"(v));
    return v;
}
__device__ __forceinline__ void cluster_arrive_relaxed() { asm volatile("barrier.cluster.arrive.relaxed.aligned;" ::: "memory"); }
__device__ __forceinline__ void cluster_arrive_release() { asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory"); }
__device__ __forceinline__ void cluster_wait_acquire() { asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory"); }

__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void st_cluster_f32(const float* local_slot, uint32_t peer_rank, float value)
{
    uint32_t remote;
    asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(remote) : "r"(smem_u32(local_slot)), "r"(peer_rank));
    asm volatile("st.shared::cluster.f32 [%0], %1;" ::"r"(remote), "f"(value) : "memory");
}

__device__ __forceinline__ void mbarrier_init(uint64_t* bar, uint32_t count)
{
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(bar)), "r"(count) : "memory");
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
}
__device__ __forceinline__ void mbarrier_expect_tx(uint64_t* bar, uint32_t bytes)
{
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_u32(bar)), "r"(bytes) : "memory");
}
// One TMA bulk copy global -> this CTA's shared memory; completion is counted on `bar` in bytes.
// Both addresses and the size are multiples of 16 bytes (checked on the host before launch).
__device__ __forceinline__ void tma_bulk_load(void* smem_dst, const void* gmem_src, uint32_t bytes, uint64_t* bar)
{
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                 ::"r"(smem_u32(smem_dst)), "l"(gmem_src), "r"(bytes), "r"(smem_u32(bar)) : "memory");
}
// Bounded wait for phase `parity` of `bar`.  Returns false when the poll limit is reached.
__device__ __forceinline__ bool mbarrier_wait_bounded(uint64_t* bar, uint32_t parity, unsigned poll_limit = kMbarrierPollLimit)
{
    const uint32_t addr = smem_u32(bar);
    const long long t0 = clock64();
    for (unsigned it = 0; it < poll_limit; ++it) {
        uint32_t done;
        asm volatile(
            "{\n\t.reg .pred p;\n\t"
            "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
            "selp.u32 %0, 1, 0, p;\n\t}"
            : "=r"(done) : "r"(addr), "r"(parity) : "memory");
        if (done) return true;
        if ((it & 255u) == 255u && clock64() - t0 > kMbarrierCycleLimit) break;
    }
    return false;
}

// Programmatic dependent launch.  When the kernel is launched with the programmatic-stream-serialization
// attribute, its CTAs may be scheduled while the previous kernel of the stream is still draining; everything above
// this call (index arithmetic) overlaps that kernel's tail, and the call returns once that kernel has completed
// and its writes are visible, so nothing below it can see unfinished data.  Without the attribute it is a no-op.
// The kernels never signal their own dependents early (no griddepcontrol.launch_dependents): measured on B200,
// dependents that start while this kernel still streams only take SM slots from it.
__device__ __forceinline__ void wait_for_previous_kernel()
{
    asm volatile("griddepcontrol.wait;" ::: "memory");
}

// ---- the per-row reduction of the sum of squares ---------------------------------------------

// Every thread of the row passes its partial; every thread of the row receives the row total.
template <int REDUCE>
__device__ __forceinline__ float row_reduce(float partial, int tx, int ty, int tpr, uint32_t crank, uint32_t csize)
{
    __shared__ float warp_part[kMaxRowsPerCta][32];
    float total;
    if constexpr (REDUCE == kReduceSmem) {
        __shared__ float tree[1024];
        float* mine = tree + ty * tpr;
        mine[tx] = partial;
        for (int stride = tpr >> 1; stride >= 1; stride >>= 1) {
            row_sync(ty, tpr);
            if (tx < stride) mine[tx] += mine[tx + stride];
        }
        row_sync(ty, tpr);
        total = mine[0];
    } else {
#pragma unroll
        for (int off = 16; off >= 1; off >>= 1) partial += __shfl_xor_sync(0xffffffffu, partial, off);
        total = partial;
        if (tpr > 32) {
            const int lane = tx & 31, warp_in_row = tx >> 5, n_warps = tpr >> 5;
            if (lane == 0) warp_part[ty][warp_in_row] = partial;
            row_sync(ty, tpr);
            float v = lane < n_warps ? warp_part[ty][lane] : 0.f;
#pragma unroll
            for (int off = 16; off >= 1; off >>= 1) v += __shfl_xor_sync(0xffffffffu, v, off);
            total = v;
        }
    }
    if constexpr (REDUCE == kReduceCluster) {
        // The row is split over the CTAs of a cluster: exchange CTA totals through distributed shared
        // memory.  The first wait pairs with the arrive at kernel entry (all peers are running).
        __shared__ float slot[kMaxRowsPerCta][kMaxClusterSize];
        cluster_wait_acquire();
        if (tx < (int)csize) st_cluster_f32(&slot[ty][crank], (uint32_t)tx, total);
        cluster_arrive_release();
        cluster_wait_acquire();
        float v = 0.f;
        for (uint32_t k = 0; k < csize; ++k) v += slot[ty][k];
        total = v;
    }
    return total;
}

// ---- the kernel ---------------------------------------------------------------------------------

// Shared-memory layout of the fp32 sums (STAGE == kStageSmemLdg): EPV floats of one vector are kept
// as EPV/W chunks of W floats in separate planes, so that consecutive threads write consecutive
// 16-byte (or 8/4-byte) chunks: no bank conflicts.
template <int EPV>
struct SumPlanes {
    static constexpr int W = EPV >= 4 ? 4 : EPV;
    static constexpr int PLANES = EPV / W;
    static __device__ __forceinline__ void store(float* row_base, int slice_cap, int v, const float (&s)[EPV])
    {
#pragma unroll
        for (int p = 0; p < PLANES; ++p) {
            float* dst = row_base + ((size_t)p * slice_cap + v) * W;
            if constexpr (W == 4) *reinterpret_cast<float4*>(dst) = make_float4(s[4 * p], s[4 * p + 1], s[4 * p + 2], s[4 * p + 3]);
            else if constexpr (W == 2) *reinterpret_cast<float2*>(dst) = make_float2(s[0], s[1]);
            else dst[0] = s[0];
        }
    }
    static __device__ __forceinline__ void load(const float* row_base, int slice_cap, int v, float (&s)[EPV])
    {
#pragma unroll
        for (int p = 0; p < PLANES; ++p) {
            const float* src = row_base + ((size_t)p * slice_cap + v) * W;
            if constexpr (W == 4) {
                const float4 q = *reinterpret_cast<const float4*>(src);
                s[4 * p] = q.x; s[4 * p + 1] = q.y; s[4 * p + 2] = q.z; s[4 * p + 3] = q.w;
            } else if constexpr (W == 2) {
                const float2 q = *reinterpret_cast<const float2*>(src);
                s[0] = q.x; s[1] = q.y;
            } else {
                s[0] = src[0];
            }
        }
    }
};

template <typename T, int VB, int STAGE, int REDUCE, int U, int CAP, bool TRACE = false>
__global__ void add_rmsnorm_kernel(const KernelArgs a)
{
    PhaseTrace<TRACE> trace;
    trace.begin();
    using C = Codec<T, VB>;
    constexpr int EPV = C::EPV;
    static_assert((STAGE != kStageReg && STAGE != kStageRegRealign) || CAP % U == 0, "the unroll depth divides the per-thread vector count");
    extern __shared__ __align__(128) unsigned char dyn_smem[];

    const int tx = threadIdx.x, ty = threadIdx.y, tpr = blockDim.x;
    uint32_t crank = 0, csize = 1;
    long long row_block = blockIdx.x;
    if constexpr (REDUCE == kReduceCluster) {
        cluster_arrive_relaxed();  // matched by the first wait inside row_reduce
        crank = cluster_cta_rank();
        csize = cluster_num_ctas();
        row_block = blockIdx.x / csize;
    }
    const long long row = row_block * blockDim.y + ty;
    const int v_begin = (int)crank * a.slice_nvec;
    int n = a.nvec - v_begin;              // vectors of this row owned by this CTA
    if (n > a.slice_nvec) n = a.slice_nvec;
    if (n < 0 || row >= a.n_tokens) n = 0;  // rows past the end and empty slices still reach every barrier

    const size_t row_off = ((size_t)(row < a.n_tokens ? row : 0) * (size_t)a.nvec + (size_t)v_begin) * VB;
    const unsigned char* xrow = reinterpret_cast<const unsigned char*>(a.x) + row_off;
    const unsigned char* rrow = reinterpret_cast<const unsigned char*>(a.r) + row_off;
    const unsigned char* wrow = reinterpret_cast<const unsigned char*>(a.w) + (size_t)v_begin * VB;
    unsigned char* yrow = reinterpret_cast<unsigned char*>(a.y) + row_off;
    unsigned char* orow = reinterpret_cast<unsigned char*>(a.r_out) + row_off;

    wait_for_previous_kernel();
    trace.mark(kTraceReleased);
    float ss = 0.f;

    if constexpr (STAGE == kStageReg) {
        float s[CAP][EPV];
        // A thread that owns at most two vectors (the latency-bound shapes) fetches its weights ahead of the
        // reduction: a few registers buy the overlap of that fetch with the barrier.  With a single vector it
        // fetches them first of all, so that the fetch also overlaps the loads of x and r (with two vectors that
        // order costs four registers and, at 256 threads, a resident CTA on the bandwidth-bound shapes).  Threads that
        // own more fetch them after the reduction, where other CTAs' traffic hides the latency and registers are scarce.
        constexpr bool kEarlyWeight = CAP <= 2;
        constexpr bool kWeightFirst = CAP == 1;
        Vec<VB> wv[kEarlyWeight ? CAP : 1];
        if constexpr (kWeightFirst) {
            if (tx < n) wv[0] = ld_weight_early<VB>(wrow + (size_t)tx * VB);
        }
#pragma unroll
        for (int i0 = 0; i0 < CAP; i0 += U) {
            Vec<VB> xv[U], rv[U];
#pragma unroll
            for (int u = 0; u < U; ++u) {
                const int v = tx + (i0 + u) * tpr;
                if (v < n) xv[u] = ld_stream<VB>(xrow + (size_t)v * VB);
            }
#pragma unroll
            for (int u = 0; u < U; ++u) {
                const int v = tx + (i0 + u) * tpr;
                if (v < n) rv[u] = ld_stream<VB>(rrow + (size_t)v * VB);
            }
#pragma unroll
            for (int u = 0; u < U; ++u) {
                const int v = tx + (i0 + u) * tpr;
                if (v < n) {
                    float xf[EPV], rf[EPV];
                    C::unpack(xv[u], xf);
                    C::unpack(rv[u], rf);
                    float sv = 0.f;  // this vector's sum of squares: the thread's running sum takes one addition per vector
#pragma unroll
                    for (int e = 0; e < EPV; ++e) {
                        s[i0 + u][e] = xf[e] + rf[e];
                        sv = fmaf(s[i0 + u][e], s[i0 + u][e], sv);
                    }
                    ss += sv;
                    st_stream<VB, true>(orow + (size_t)v * VB, C::pack(s[i0 + u]));
                }
            }
        }
        if constexpr (kEarlyWeight && !kWeightFirst) {
#pragma unroll
            for (int i = 0; i < CAP; ++i) {
                const int v = tx + i * tpr;
                if (v < n) wv[i] = ld_weight_early<VB>(wrow + (size_t)v * VB);
            }
        }
        trace.mark(kTraceLoaded);
        const float total = row_reduce<REDUCE>(ss, tx, ty, tpr, crank, csize);
        const float rho = __frsqrt_rn(total / (float)a.hidden + a.eps);
        trace.mark(kTraceReduced);
#pragma unroll
        for (int i = 0; i < CAP; ++i) {
            const int v = tx + i * tpr;
            if (v < n) {
                float wf[EPV], yf[EPV];
                if constexpr (kEarlyWeight) C::unpack(wv[i], wf);
                else C::unpack(ld_weight<VB>(wrow + (size_t)v * VB), wf);
#pragma unroll
                for (int e = 0; e < EPV; ++e) yf[e] = s[i][e] * rho * wf[e];
                st_stream<VB, true>(yrow + (size_t)v * VB, C::pack(yf));
            }
        }
    } else if constexpr (STAGE == kStageRegRealign) {
        static_assert((VB == 16 || VB == 32) && REDUCE != kReduceCluster, "ragged rows: 16- or 32-byte chunks, one CTA per row");
        constexpr int EB = (int)sizeof(T);
        using C1 = Codec<T, EB>;  // one element
        const bool live = row < a.n_tokens;
        const size_t row_byte = (size_t)(live ? row : 0) * (size_t)a.hidden * EB;
        int head = (int)(((unsigned)VB - (unsigned)(row_byte & (VB - 1))) & (VB - 1)) / EB;  // elements before the first boundary
        if (head > a.hidden) head = a.hidden;
        const int n_whole = live ? (a.hidden - head) / EPV : 0;            // aligned chunks wholly inside the row
        const int tail = a.hidden - head - n_whole * EPV;                  // elements after the last of them
        const int n_edge = live ? head + tail : 0;                         // < 2 * EPV <= 32: one thread each
        const int edge_col = tx < head ? tx : head + n_whole * EPV + (tx - head);
        const int phase = (head * EB) & 15;                                // address of a chunk's weights, modulo 16
        const size_t chunk_off = row_byte + (size_t)head * EB;
        const unsigned char* xc = reinterpret_cast<const unsigned char*>(a.x) + chunk_off;
        const unsigned char* rc = reinterpret_cast<const unsigned char*>(a.r) + chunk_off;
        const unsigned char* wc = reinterpret_cast<const unsigned char*>(a.w) + (size_t)head * EB;
        unsigned char* yc = reinterpret_cast<unsigned char*>(a.y) + chunk_off;
        unsigned char* oc = reinterpret_cast<unsigned char*>(a.r_out) + chunk_off;
        const size_t edge_off = row_byte + (size_t)edge_col * EB;
        // the chunk whose last aligned weight vector would end past w is read element by element
        const int v_unsafe = (phase != 0 && tail * EB < 16 - phase) ? n_whole - 1 : -1;
        float s[CAP][EPV];
        float s_edge = 0.f;
#pragma unroll
        for (int i0 = 0; i0 < CAP; i0 += U) {
            Vec<VB> xv[U], rv[U];
#pragma unroll
            for (int u = 0; u < U; ++u) {
                const int v = tx + (i0 + u) * tpr;
                if (v < n_whole) xv[u] = ld_stream<VB>(xc + (size_t)v * VB);
            }
#pragma unroll
            for (int u = 0; u < U; ++u) {
                const int v = tx + (i0 + u) * tpr;
                if (v < n_whole) rv[u] = ld_stream<VB>(rc + (size_t)v * VB);
            }
#pragma unroll
            for (int u = 0; u < U; ++u) {
                const int v = tx + (i0 + u) * tpr;
                if (v < n_whole) {
                    float xf[EPV], rf[EPV];
                    C::unpack(xv[u], xf);
                    C::unpack(rv[u], rf);
                    float sv = 0.f;  // this vector's sum of squares: the thread's running sum takes one addition per vector
#pragma unroll
                    for (int e = 0; e < EPV; ++e) {
                        s[i0 + u][e] = xf[e] + rf[e];
                        sv = fmaf(s[i0 + u][e], s[i0 + u][e], sv);
                    }
                    ss += sv;
                    st_stream<VB, true>(oc + (size_t)v * VB, C::pack(s[i0 + u]));
                }
            }
        }
        if (tx < n_edge) {
            float xf[1], rf[1], sf[1];
            C1::unpack(ld_stream<EB>(reinterpret_cast<const unsigned char*>(a.x) + edge_off), xf);
            C1::unpack(ld_stream<EB>(reinterpret_cast<const unsigned char*>(a.r) + edge_off), rf);
            sf[0] = s_edge = xf[0] + rf[0];
            ss = fmaf(s_edge, s_edge, ss);
            st_stream<EB>(reinterpret_cast<unsigned char*>(a.r_out) + edge_off, C1::pack(sf));
        }
        // As in the register stage, a thread that owns at most 32 bytes of the row fetches its weights ahead of the
        // reduction; the one weight of a head or tail element always is.
        constexpr bool kEarlyWeight = CAP * VB <= 32;
        Vec<VB> wv[kEarlyWeight ? CAP : 1];
        Vec<EB> w_edge;
        if constexpr (kEarlyWeight) {
#pragma unroll
            for (int k = 0; k < CAP; ++k) {
                const int v = tx + k * tpr;
                if (v < n_whole) wv[k] = ld_weight_ragged<T, VB, true>(wc + (size_t)v * VB, phase, v != v_unsafe);
            }
        }
        if (tx < n_edge) w_edge = ld_weight_early<EB>(reinterpret_cast<const unsigned char*>(a.w) + (size_t)edge_col * EB);
        trace.mark(kTraceLoaded);
        const float total = row_reduce<REDUCE>(ss, tx, ty, tpr, crank, csize);
        const float rho = __frsqrt_rn(total / (float)a.hidden + a.eps);
        trace.mark(kTraceReduced);
#pragma unroll
        for (int k = 0; k < CAP; ++k) {
            const int v = tx + k * tpr;
            if (v < n_whole) {
                float wf[EPV], yf[EPV];
                if constexpr (kEarlyWeight) C::unpack(wv[k], wf);
                else C::unpack(ld_weight_ragged<T, VB, false>(wc + (size_t)v * VB, phase, v != v_unsafe), wf);
#pragma unroll
                for (int e = 0; e < EPV; ++e) yf[e] = s[k][e] * rho * wf[e];
                st_stream<VB, true>(yc + (size_t)v * VB, C::pack(yf));
            }
        }
        if (tx < n_edge) {
            float wf[1], yf[1];
            C1::unpack(w_edge, wf);
            yf[0] = s_edge * rho * wf[0];
            st_stream<EB>(reinterpret_cast<unsigned char*>(a.y) + edge_off, C1::pack(yf));
        }
    } else if constexpr (STAGE == kStageSmemLdg) {
        using P = SumPlanes<EPV>;
        float* srow = reinterpret_cast<float*>(dyn_smem) + (size_t)ty * a.slice_nvec * EPV;
        for (int v0 = tx; v0 < n; v0 += U * tpr) {
            Vec<VB> xv[U], rv[U];
#pragma unroll
            for (int u = 0; u < U; ++u) {
                const int v = v0 + u * tpr;
                if (v < n) xv[u] = ld_stream<VB>(xrow + (size_t)v * VB);
            }
#pragma unroll
            for (int u = 0; u < U; ++u) {
                const int v = v0 + u * tpr;
                if (v < n) rv[u] = ld_stream<VB>(rrow + (size_t)v * VB);
            }
#pragma unroll
            for (int u = 0; u < U; ++u) {
                const int v = v0 + u * tpr;
                if (v < n) {
                    float xf[EPV], rf[EPV], s[EPV];
                    C::unpack(xv[u], xf);
                    C::unpack(rv[u], rf);
                    float sv = 0.f;
#pragma unroll
                    for (int e = 0; e < EPV; ++e) {
                        s[e] = xf[e] + rf[e];
                        sv = fmaf(s[e], s[e], sv);
                    }
                    ss += sv;
                    st_stream<VB, true>(orow + (size_t)v * VB, C::pack(s));
                    P::store(srow, a.slice_nvec, v, s);  // read back by this same thread only
                }
            }
        }
        trace.mark(kTraceLoaded);
        const float total = row_reduce<REDUCE>(ss, tx, ty, tpr, crank, csize);
        const float rho = __frsqrt_rn(total / (float)a.hidden + a.eps);
        trace.mark(kTraceReduced);
        for (int v0 = tx; v0 < n; v0 += U * tpr) {
            Vec<VB> wv[U];
#pragma unroll
            for (int u = 0; u < U; ++u) {
                const int v = v0 + u * tpr;
                if (v < n) wv[u] = ld_weight<VB>(wrow + (size_t)v * VB);
            }
#pragma unroll
            for (int u = 0; u < U; ++u) {
                const int v = v0 + u * tpr;
                if (v < n) {
                    float s[EPV], wf[EPV], yf[EPV];
                    P::load(srow, a.slice_nvec, v, s);
                    C::unpack(wv[u], wf);
#pragma unroll
                    for (int e = 0; e < EPV; ++e) yf[e] = s[e] * rho * wf[e];
                    st_stream<VB, true>(yrow + (size_t)v * VB, C::pack(yf));
                }
            }
        }
    } else if constexpr (STAGE == kStageSmemTma) {
        // TMA: one thread per row posts two bulk copies (x slice, r slice) that complete on the row's
        // mbarrier; the row's threads then work out of shared memory.
        __shared__ __align__(8) uint64_t bars[kMaxRowsPerCta];
        const size_t slice_bytes = (size_t)a.slice_nvec * VB;
        unsigned char* xs = dyn_smem + (size_t)ty * 2 * slice_bytes;
        unsigned char* rs = xs + slice_bytes;
        if (tx == 0) {
            mbarrier_init(&bars[ty], 1);
            if (n > 0 && !a.drop_copies) {
                const uint32_t bytes = (uint32_t)n * VB;
                mbarrier_expect_tx(&bars[ty], 2 * bytes);
                tma_bulk_load(xs, xrow, bytes, &bars[ty]);
                tma_bulk_load(rs, rrow, bytes, &bars[ty]);
            }
        }
        row_sync(ty, tpr);  // the barrier is initialised before anyone polls it
        if (n > 0) {
            bool landed = mbarrier_wait_bounded(&bars[ty], 0, a.wait_polls);
            if (!landed) {
                atomicExch(a.status, kDeviceTimeoutCode);
                landed = mbarrier_wait_bounded(&bars[ty], 0, a.wait_polls);  // do not leave while the copies may still land
            }
        }
        for (int v0 = tx; v0 < n; v0 += U * tpr) {
#pragma unroll
            for (int u = 0; u < U; ++u) {
                const int v = v0 + u * tpr;
                if (v < n) {
                    float xf[EPV], rf[EPV], s[EPV];
                    C::unpack(ld_shared<VB>(xs + (size_t)v * VB), xf);
                    C::unpack(ld_shared<VB>(rs + (size_t)v * VB), rf);
                    float sv = 0.f;
#pragma unroll
                    for (int e = 0; e < EPV; ++e) {
                        s[e] = xf[e] + rf[e];
                        sv = fmaf(s[e], s[e], sv);
                    }
                    ss += sv;
                    st_stream<VB>(orow + (size_t)v * VB, C::pack(s));
                }
            }
        }
        trace.mark(kTraceLoaded);
        const float total = row_reduce<REDUCE>(ss, tx, ty, tpr, crank, csize);
        const float rho = __frsqrt_rn(total / (float)a.hidden + a.eps);
        trace.mark(kTraceReduced);
        for (int v0 = tx; v0 < n; v0 += U * tpr) {
            Vec<VB> wv[U];
#pragma unroll
            for (int u = 0; u < U; ++u) {
                const int v = v0 + u * tpr;
                if (v < n) wv[u] = ld_weight<VB>(wrow + (size_t)v * VB);
            }
#pragma unroll
            for (int u = 0; u < U; ++u) {
                const int v = v0 + u * tpr;
                if (v < n) {
                    float xf[EPV], rf[EPV], wf[EPV], yf[EPV];
                    C::unpack(ld_shared<VB>(xs + (size_t)v * VB), xf);
                    C::unpack(ld_shared<VB>(rs + (size_t)v * VB), rf);
                    C::unpack(wv[u], wf);
#pragma unroll
                    for (int e = 0; e < EPV; ++e) yf[e] = (xf[e] + rf[e]) * rho * wf[e];  // same binary32 sum as pass 1
                    st_stream<VB>(yrow + (size_t)v * VB, C::pack(yf));
                }
            }
        }
    } else {
        // Persistent pipeline: the grid holds as many CTAs as stay resident; CTA b handles row blocks b, b + grid,
        // b + 2 grid, ...  Every row slot of the CTA owns a ring of U shared-memory stages, each with its own
        // mbarrier.  The slot's first thread posts the bulk copies of block i + U into a stage as soon as the slot's
        // threads have finished with block i in it, so up to U - 1 blocks are on their way while one is reduced and
        // stored.  Stage i % U is filled for the (i / U)-th time by block i: its mbarrier phase is (i / U) & 1.
        static_assert(REDUCE != kReduceCluster, "the pipeline stage keeps a row inside one CTA");
        static_assert(U <= kMaxPipelineDepth, "ring deeper than the barrier array");
        constexpr int IU = 2;  // vectors per thread and batch in the two passes over a stage
        __shared__ __align__(8) uint64_t bars[kMaxPipelineDepth][kMaxRowsPerCta];
        const size_t row_bytes = (size_t)a.nvec * VB;
        const size_t stage_bytes = (size_t)blockDim.y * 2 * row_bytes;  // one stage: x and r of every row slot
        const long long n_blocks = (a.n_tokens + blockDim.y - 1) / blockDim.y;
        const long long stride = gridDim.x;
        const unsigned char* xbase = reinterpret_cast<const unsigned char*>(a.x);
        const unsigned char* rbase = reinterpret_cast<const unsigned char*>(a.r);
        const unsigned char* wbase = reinterpret_cast<const unsigned char*>(a.w);
        auto post = [&](long long block, int stage) {  // called by the slot's first thread only
            const long long rw = block * blockDim.y + ty;
            if (block >= n_blocks || rw >= a.n_tokens || a.drop_copies) return;
            unsigned char* xs = dyn_smem + (size_t)stage * stage_bytes + (size_t)ty * 2 * row_bytes;
            const size_t off = (size_t)rw * row_bytes;
            mbarrier_expect_tx(&bars[stage][ty], 2 * (uint32_t)row_bytes);
            tma_bulk_load(xs, xbase + off, (uint32_t)row_bytes, &bars[stage][ty]);
            tma_bulk_load(xs + row_bytes, rbase + off, (uint32_t)row_bytes, &bars[stage][ty]);
        };
        if (tx == 0) {
#pragma unroll
            for (int st = 0; st < U; ++st) mbarrier_init(&bars[st][ty], 1);
#pragma unroll
            for (int st = 0; st < U; ++st) post((long long)blockIdx.x + st * stride, st);
        }
        row_sync(ty, tpr);  // the barriers are initialised before anyone polls them
        int it = 0;
        for (long long block = blockIdx.x; block < n_blocks; block += stride, ++it) {
            const int stage = it % U;
            const uint32_t parity = (uint32_t)(it / U) & 1u;
            const long long rw = block * blockDim.y + ty;
            const int nv = rw < a.n_tokens ? a.nvec : 0;
            const unsigned char* xs = dyn_smem + (size_t)stage * stage_bytes + (size_t)ty * 2 * row_bytes;
            const unsigned char* rs = xs + row_bytes;
            unsigned char* yr = reinterpret_cast<unsigned char*>(a.y) + (size_t)(nv ? rw : 0) * row_bytes;
            unsigned char* orw = reinterpret_cast<unsigned char*>(a.r_out) + (size_t)(nv ? rw : 0) * row_bytes;
            if (nv > 0) {
                bool landed = mbarrier_wait_bounded(&bars[stage][ty], parity, a.wait_polls);
                if (!landed) {
                    atomicExch(a.status, kDeviceTimeoutCode);
                    landed = mbarrier_wait_bounded(&bars[stage][ty], parity, a.wait_polls);
                }
            }
            float ssb = 0.f;
            for (int v0 = tx; v0 < nv; v0 += IU * tpr) {
#pragma unroll
                for (int u = 0; u < IU; ++u) {
                    const int v = v0 + u * tpr;
                    if (v < nv) {
                        float xf[EPV], rf[EPV], sum[EPV];
                        C::unpack(ld_shared<VB>(xs + (size_t)v * VB), xf);
                        C::unpack(ld_shared<VB>(rs + (size_t)v * VB), rf);
                        float sv = 0.f;
#pragma unroll
                        for (int e = 0; e < EPV; ++e) {
                            sum[e] = xf[e] + rf[e];
                            sv = fmaf(sum[e], sum[e], sv);
                        }
                        ssb += sv;
                        st_stream<VB>(orw + (size_t)v * VB, C::pack(sum));
                    }
                }
            }
            const float total = row_reduce<REDUCE>(ssb, tx, ty, tpr, 0u, 1u);
            const float rho = __frsqrt_rn(total / (float)a.hidden + a.eps);
            for (int v0 = tx; v0 < nv; v0 += IU * tpr) {
                Vec<VB> wv[IU];
#pragma unroll
                for (int u = 0; u < IU; ++u) {
                    const int v = v0 + u * tpr;
                    if (v < nv) wv[u] = ld_weight<VB>(wbase + (size_t)v * VB);
                }
#pragma unroll
                for (int u = 0; u < IU; ++u) {
                    const int v = v0 + u * tpr;
                    if (v < nv) {
                        float xf[EPV], rf[EPV], wf[EPV], yf[EPV];
                        C::unpack(ld_shared<VB>(xs + (size_t)v * VB), xf);
                        C::unpack(ld_shared<VB>(rs + (size_t)v * VB), rf);
                        C::unpack(wv[u], wf);
#pragma unroll
                        for (int e = 0; e < EPV; ++e) yf[e] = (xf[e] + rf[e]) * rho * wf[e];  // same binary32 sum as pass 1
                        st_stream<VB>(yr + (size_t)v * VB, C::pack(yf));
                    }
                }
            }
            row_sync(ty, tpr);  // every thread of the slot has read the stage for the last time
            if (tx == 0) post(block + (long long)U * stride, stage);
        }
    }
    trace.mark(kTraceStored);
    trace.flush(a);
}

}  // namespace rt
