// merge_attn_states as a parameterised kernel template (sm_100a): the third of the paper's three tuned
// kernels ("Kernels", Experimental Setup, shapes (n, h, d)), put through the same deriver and search.
//
//   v_a, v_b: [n, h, d] (dtype), s_a, s_b: [n, h] (binary32 log-sum-exp);  m = max(s_a, s_b),
//   w_a = e^(s_a - m), w_b = e^(s_b - m), D = w_a + w_b;
//   v_out = rn((w_a v_a + w_b v_b) / D),  s_out = m + ln D;   both parts empty (m = -inf): v_out = 0, s_out = -inf.
//
// One row of the template is one token: h * d contiguous elements.  A vector of VB bytes lies inside one
// head (checked on the host), so a thread finds its head as vector index / vectors per head and reads that
// head's two log-sum-exps through the read-only path.  Axes: threads per row, rows per CTA, VB, U loads in
// flight, STAGE = registers or TMA bulk (the token's v_a row and v_b row land in shared memory).
#pragma once

#include "add_rmsnorm_kernel.cuh"

namespace rt {

struct MergeArgs {
    const void* v_a;
    const void* v_b;
    const float* s_a;
    const float* s_b;
    void* v_out;
    float* s_out;
    long long n_tokens;
    int nvec;           // vectors of VB bytes in one token row (h * d elements)
    int vec_per_head;   // vectors in one head (d elements)
    int heads;
    int* status;        // device status word
};

// Normalised weights of the two parts and the merged log-sum-exp of one (token, head).
__device__ __forceinline__ void merge_weights(float sa, float sb, float& wa, float& wb, float& s)
{
    const float m = fmaxf(sa, sb);
    if (m == -INFINITY) {  // both parts empty
        wa = 0.f;
        wb = 0.f;
        s = -INFINITY;
        return;
    }
    const float ea = expf(sa - m), eb = expf(sb - m);
    const float d = ea + eb;  // in [1, 2]
    wa = ea / d;
    wb = eb / d;
    s = m + logf(d);
}

template <typename T, int VB, int STAGE, int U>
__global__ void merge_attn_states_kernel(const MergeArgs a)
{
    using C = Codec<T, VB>;
    constexpr int EPV = C::EPV;
    extern __shared__ __align__(128) unsigned char dyn_smem[];
    const int tx = threadIdx.x, ty = threadIdx.y, tpr = blockDim.x;
    const long long row = (long long)blockIdx.x * blockDim.y + ty;
    const int n = row < a.n_tokens ? a.nvec : 0;
    const size_t row_bytes = (size_t)a.nvec * VB;
    const size_t safe_row = (size_t)(row < a.n_tokens ? row : 0);
    const unsigned char* pa = reinterpret_cast<const unsigned char*>(a.v_a) + safe_row * row_bytes;
    const unsigned char* pb = reinterpret_cast<const unsigned char*>(a.v_b) + safe_row * row_bytes;
    unsigned char* po = reinterpret_cast<unsigned char*>(a.v_out) + safe_row * row_bytes;
    const float* sa = a.s_a + safe_row * a.heads;
    const float* sb = a.s_b + safe_row * a.heads;
    float* so = a.s_out + safe_row * a.heads;

    if constexpr (STAGE == kStageSmemTma) {
        __shared__ __align__(8) uint64_t bars[kMaxRowsPerCta];
        unsigned char* xs = dyn_smem + (size_t)ty * 2 * row_bytes;
        unsigned char* ys = xs + row_bytes;
        if (tx == 0) {
            mbarrier_init(&bars[ty], 1);
            if (n > 0) {
                mbarrier_expect_tx(&bars[ty], (uint32_t)(2 * row_bytes));
                tma_bulk_load(xs, pa, (uint32_t)row_bytes, &bars[ty]);
                tma_bulk_load(ys, pb, (uint32_t)row_bytes, &bars[ty]);
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
        pa = xs;
        pb = ys;
    }

    for (int v0 = tx; v0 < n; v0 += U * tpr) {
        Vec<VB> av[U], bv[U];
        float fa[U], fb[U];
#pragma unroll
        for (int u = 0; u < U; ++u) {
            const int v = v0 + u * tpr;
            if (v < n) {
                if constexpr (STAGE == kStageSmemTma) av[u] = ld_shared<VB>(pa + (size_t)v * VB);
                else av[u] = ld_stream<VB>(pa + (size_t)v * VB);
            }
        }
#pragma unroll
        for (int u = 0; u < U; ++u) {
            const int v = v0 + u * tpr;
            if (v < n) {
                if constexpr (STAGE == kStageSmemTma) bv[u] = ld_shared<VB>(pb + (size_t)v * VB);
                else bv[u] = ld_stream<VB>(pb + (size_t)v * VB);
            }
        }
#pragma unroll
        for (int u = 0; u < U; ++u) {
            const int v = v0 + u * tpr;
            if (v < n) {
                const int head = v / a.vec_per_head;
                fa[u] = __ldg(sa + head);
                fb[u] = __ldg(sb + head);
            }
        }
#pragma unroll
        for (int u = 0; u < U; ++u) {
            const int v = v0 + u * tpr;
            if (v < n) {
                float wa, wb, s;
                merge_weights(fa[u], fb[u], wa, wb, s);
                const int head = v / a.vec_per_head;
                if (v - head * a.vec_per_head == 0) so[head] = s;  // the head's first vector writes s_out
                float xf[EPV], yf[EPV], of[EPV];
                C::unpack(av[u], xf);
                C::unpack(bv[u], yf);
#pragma unroll
                for (int e = 0; e < EPV; ++e) of[e] = fmaf(wa, xf[e], wb * yf[e]);
                st_stream<VB>(po + (size_t)v * VB, C::pack(of));
            }
        }
    }
}

}  // namespace rt
