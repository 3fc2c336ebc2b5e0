// silu_and_mul as a parameterised kernel template (sm_100a): the second of the paper's three tuned
// kernels ("Kernels", Experimental Setup), put through the same deriver and search as the norm kernel.
//
//   x: [n_tokens, 2*d], out: [n_tokens, d];  out[t,j] = rn( silu(x[t,j]) * x[t,d+j] ),  silu(g) = g/(1+e^-g)
//
// Axes: threads per row and rows per CTA (run-time block shape), VB bytes per ld/st, U independent loads
// in flight, STAGE = registers (ld.global straight into registers) or TMA bulk (the whole input row of one
// token - gate and value are contiguous - lands in shared memory with one cp.async.bulk).
#pragma once

#include "add_rmsnorm_kernel.cuh"

namespace rt {

struct SiluArgs {
    const void* x;
    void* out;
    long long n_tokens;
    int nvec;     // vectors of VB bytes in one output row (= in each half of an input row)
    int* status;  // device status word
};

// silu(g) * u in fp32: e^-g through ex2.approx, the quotient through rcp.approx.  For g below about -87
// the quotient underflows to -0 (the exact value is below 1e-36 in magnitude).
__device__ __forceinline__ float silu_mul(float g, float u)
{
    const float e = exp2f(-g * 1.4426950408889634f);
    return __fdividef(g, 1.0f + e) * u;
}

template <typename T, int VB, int STAGE, int U>
__global__ void silu_and_mul_kernel(const SiluArgs a)
{
    using C = Codec<T, VB>;
    constexpr int EPV = C::EPV;
    extern __shared__ __align__(128) unsigned char dyn_smem[];
    const int tx = threadIdx.x, ty = threadIdx.y, tpr = blockDim.x;
    const long long row = (long long)blockIdx.x * blockDim.y + ty;
    const int n = row < a.n_tokens ? a.nvec : 0;
    const size_t half_bytes = (size_t)a.nvec * VB;
    const size_t safe_row = (size_t)(row < a.n_tokens ? row : 0);
    const unsigned char* gate = reinterpret_cast<const unsigned char*>(a.x) + safe_row * 2 * half_bytes;
    const unsigned char* value = gate + half_bytes;
    unsigned char* out = reinterpret_cast<unsigned char*>(a.out) + safe_row * half_bytes;
    wait_for_previous_kernel();

    if constexpr (STAGE == kStageSmemTma) {
        __shared__ __align__(8) uint64_t bars[kMaxRowsPerCta];
        unsigned char* srow = dyn_smem + (size_t)ty * 2 * half_bytes;
        if (tx == 0) {
            mbarrier_init(&bars[ty], 1);
            if (n > 0) {
                mbarrier_expect_tx(&bars[ty], (uint32_t)(2 * half_bytes));
                tma_bulk_load(srow, gate, (uint32_t)(2 * half_bytes), &bars[ty]);
            }
        }
        row_sync(ty, tpr);
        if (n > 0) {
            bool landed = mbarrier_wait_bounded(&bars[ty], 0);
            if (!landed) {
                atomicExch(a.status, kDeviceTimeoutCode);
                landed = mbarrier_wait_bounded(&bars[ty], 0);
            }
        }
        gate = srow;
        value = srow + half_bytes;
    }

    for (int v0 = tx; v0 < n; v0 += U * tpr) {
        Vec<VB> gv[U], uv[U];
#pragma unroll
        for (int u = 0; u < U; ++u) {
            const int v = v0 + u * tpr;
            if (v < n) {
                if constexpr (STAGE == kStageSmemTma) gv[u] = ld_shared<VB>(gate + (size_t)v * VB);
                else gv[u] = ld_stream<VB>(gate + (size_t)v * VB);
            }
        }
#pragma unroll
        for (int u = 0; u < U; ++u) {
            const int v = v0 + u * tpr;
            if (v < n) {
                if constexpr (STAGE == kStageSmemTma) uv[u] = ld_shared<VB>(value + (size_t)v * VB);
                else uv[u] = ld_stream<VB>(value + (size_t)v * VB);
            }
        }
#pragma unroll
        for (int u = 0; u < U; ++u) {
            const int v = v0 + u * tpr;
            if (v < n) {
                float gf[EPV], uf[EPV], of[EPV];
                C::unpack(gv[u], gf);
                C::unpack(uv[u], uf);
#pragma unroll
                for (int e = 0; e < EPV; ++e) of[e] = silu_mul(gf[e], uf[e]);
                st_stream<VB, STAGE == kStageReg>(out + (size_t)v * VB, C::pack(of));
            }
        }
    }
}

}  // namespace rt
