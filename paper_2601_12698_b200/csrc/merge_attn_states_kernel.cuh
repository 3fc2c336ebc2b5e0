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
    int head_shift;     // log2(vec_per_head) when it is a power of two, else -1
    int* status;        // device status word
};

// Normalised weights of the two parts of one (token, head), and D = w_a + w_b before normalisation.
// e^x through ex2.approx, 1/D through rcp.approx: the weights carry a relative error of about 1e-6, far
// inside the output tolerance; e^0 = 1, e^-inf = 0 and 1/1 = 1 come out exactly, so an empty part returns the
// other part bit for bit.  Both parts empty (m = -inf): both weights are zero.
__device__ __forceinline__ void merge_weights(float sa, float sb, float& wa, float& wb, float& m, float& d)
{
    m = fmaxf(sa, sb);
    if (m == -INFINITY) {
        wa = 0.f;
        wb = 0.f;
        d = 0.f;
        return;
    }
    const float ea = exp2f((sa - m) * 1.4426950408889634f), eb = exp2f((sb - m) * 1.4426950408889634f);
    d = ea + eb;  // in [1, 2]
    const float inv = __fdividef(1.0f, d);
    wa = ea * inv;
    wb = eb * inv;
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
    wait_for_previous_kernel();

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
                const int head = a.head_shift >= 0 ? (v >> a.head_shift) : (v / a.vec_per_head);
                fa[u] = __ldg(sa + head);
                fb[u] = __ldg(sb + head);
            }
        }
#pragma unroll
        for (int u = 0; u < U; ++u) {
            const int v = v0 + u * tpr;
            if (v < n) {
                float wa, wb, m, d;
                merge_weights(fa[u], fb[u], wa, wb, m, d);
                const int head = a.head_shift >= 0 ? (v >> a.head_shift) : (v / a.vec_per_head);
                if (v - head * a.vec_per_head == 0)  // the head's first vector writes the merged log-sum-exp
                    so[head] = d > 0.f ? m + logf(d) : -INFINITY;
                float xf[EPV], yf[EPV], of[EPV];
                C::unpack(av[u], xf);
                C::unpack(bv[u], yf);
#pragma unroll
                for (int e = 0; e < EPV; ++e) of[e] = fmaf(wa, xf[e], wb * yf[e]);
                st_stream<VB, STAGE == kStageReg>(po + (size_t)v * VB, C::pack(of));
            }
        }
    }
}

}  // namespace rt
