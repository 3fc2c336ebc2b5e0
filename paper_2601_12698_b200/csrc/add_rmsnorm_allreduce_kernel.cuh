// Fused all-reduce + residual-add + RMSNorm: the norm template's variant for tensor-parallel serving, where the
// x of the operator is the sum over the ranks of a group of each rank's partial result.  One launch handles a
// block of rows: it reads the rows of every rank's partial (plain loads; a peer's memory over NVLink is read the
// same way as this GPU's own), sums them in rank order in binary32, adds the residual, normalises, and writes
// y for those rows into every y destination it is given (this GPU's and, for the gather half of the all-reduce,
// each peer's) and r_out into every r_out destination (usually this GPU's only: the next norm of the same rank
// needs the residual of its own rows only).  With each rank launching it on its own block of rows, every rank
// ends with the full y: reduce-scatter, the operator and all-gather in one kernel, with no wait inside the
// kernel - the ranks meet on the host (or in stream order) before and after the launch.
//
// Per row:  a = fp32(x^(0));  a += fp32(x^(k)) for k = 1..NP-1 in this order;  s = a + fp32(r);
//           r_out = rn(s);  y = rn(s * rsqrt(mean(s^2) + eps) * w).
// Register stage, 16-byte vectors, shuffle reduction; axes: threads per row, rows per CTA, unroll U (vectors
// per part in flight: U * NP loads of x are issued together), CAP row vectors kept per thread.
#pragma once

#include "add_rmsnorm_kernel.cuh"

namespace rt {

constexpr int kMaxParts = 8;

struct AllreduceArgs {
    const void* x_parts[kMaxParts];  // part k: [*, hidden] rows, indexed by absolute row
    const void* r;
    const void* w;
    void* y_outs[kMaxParts];         // destinations 0..n_y_outs-1 receive the rows of y of this launch
    void* r_outs[kMaxParts];         // destinations 0..n_r_outs-1 the rows of r_out
    int n_y_outs, n_r_outs;
    long long row_begin, row_end;    // absolute rows handled by this launch
    int hidden;
    int nvec;                        // vectors (16 or 32 bytes) in one row
    float eps;
};

template <typename T, int VB, int NP, int U, int CAP>
__global__ void add_rmsnorm_allreduce_kernel(const AllreduceArgs a)
{
    static_assert(VB == 16 || VB == 32, "16- or 32-byte vectors");
    using C = Codec<T, VB>;
    constexpr int EPV = C::EPV;
    static_assert(NP >= 2 && NP <= kMaxParts, "2..8 parts");
    static_assert(CAP % U == 0, "the unroll depth divides the per-thread vector count");

    const int tx = threadIdx.x, ty = threadIdx.y, tpr = blockDim.x;
    const long long row = a.row_begin + (long long)blockIdx.x * blockDim.y + ty;
    const int n = row < a.row_end ? a.nvec : 0;  // rows past the end still reach the barrier
    const size_t row_off = (size_t)(row < a.row_end ? row : a.row_begin) * (size_t)a.nvec * VB;
    const unsigned char* rrow = reinterpret_cast<const unsigned char*>(a.r) + row_off;
    const unsigned char* wrow = reinterpret_cast<const unsigned char*>(a.w);
    wait_for_previous_kernel();

    // the same vector to every destination; the destination count is uniform over the grid
    auto store_all = [&](void* const (&dst)[kMaxParts], int n_dst, size_t off, const Vec<VB>& v) {
#pragma unroll
        for (int d = 0; d < kMaxParts; ++d)
            if (d < n_dst) st_stream<VB, true>(reinterpret_cast<unsigned char*>(dst[d]) + off, v);
    };

    float ss = 0.f;
    float s[CAP][EPV];
#pragma unroll
    for (int i0 = 0; i0 < CAP; i0 += U) {
        Vec<VB> xv[NP][U], rv[U];
#pragma unroll
        for (int k = 0; k < NP; ++k) {
            const unsigned char* xrow = reinterpret_cast<const unsigned char*>(a.x_parts[k]) + row_off;
#pragma unroll
            for (int u = 0; u < U; ++u) {
                const int v = tx + (i0 + u) * tpr;
                if (v < n) xv[k][u] = ld_stream<VB>(xrow + (size_t)v * VB);
            }
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
                float acc[EPV], pf[EPV];
                C::unpack(xv[0][u], acc);
#pragma unroll
                for (int k = 1; k < NP; ++k) {
                    C::unpack(xv[k][u], pf);
#pragma unroll
                    for (int e = 0; e < EPV; ++e) acc[e] = __fadd_rn(acc[e], pf[e]);  // rank order, never contracted
                }
                C::unpack(rv[u], pf);
#pragma unroll
                for (int e = 0; e < EPV; ++e) {
                    s[i0 + u][e] = __fadd_rn(acc[e], pf[e]);
                    ss = fmaf(s[i0 + u][e], s[i0 + u][e], ss);
                }
                store_all(a.r_outs, a.n_r_outs, row_off + (size_t)v * VB, C::pack(s[i0 + u]));
            }
        }
    }
    const float total = row_reduce<kReduceShfl>(ss, tx, ty, tpr, 0u, 1u);
    const float rho = __frsqrt_rn(total / (float)a.hidden + a.eps);
#pragma unroll
    for (int i = 0; i < CAP; ++i) {
        const int v = tx + i * tpr;
        if (v < n) {
            float wf[EPV], yf[EPV];
            C::unpack(ld_weight<VB>(wrow + (size_t)v * VB), wf);
#pragma unroll
            for (int e = 0; e < EPV; ++e) yf[e] = s[i][e] * rho * wf[e];
            store_all(a.y_outs, a.n_y_outs, row_off + (size_t)v * VB, C::pack(yf));
        }
    }
}

}  // namespace rt
