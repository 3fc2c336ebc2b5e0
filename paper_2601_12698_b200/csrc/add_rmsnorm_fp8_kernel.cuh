// Fused residual-add + RMSNorm with a per-token fp8 (e4m3) quantised output: the norm template's variant
// for a following fp8 GEMM.  Same row mapping and stages as add_rmsnorm_kernel (registers or TMA bulk),
// 16- or 32-byte vectors of a 16-bit element type, shuffle reduction.
//
// Per row:  s = fp32(x) + fp32(r);  r_out = rn(s);  y = s * rsqrt(mean(s^2) + eps) * w   (not rounded);
//           scale = max(max_j |y_j|, 1e-12) / 448;   q_j = rn_e4m3_satfinite(y_j / scale).
// The row maximum of |s_j w_j| travels through the same reduction as the sum of squares (one barrier),
// since max_j |y_j| = rho * max_j |s_j w_j|.
#pragma once

#include "add_rmsnorm_kernel.cuh"

namespace rt {

struct Fp8Args {
    const void* x;
    const void* r;
    const void* w;
    void* q;        // [n_tokens, hidden] bytes
    float* scale;   // [n_tokens]
    void* r_out;
    long long n_tokens;
    int hidden;
    int nvec;       // vectors (16 or 32 bytes) in one row
    float eps;
    int* status;
};

constexpr float kE4m3Max = 448.0f;
constexpr float kScaleFloor = 1e-12f;

// Two binary32 values -> two e4m3 bytes (round to nearest even, saturating to +-448); `lo` lands in the low byte.
__device__ __forceinline__ uint32_t pack_e4m3x2(float lo, float hi)
{
    unsigned short d;
    asm("cvt.rn.satfinite.e4m3x2.f32 %0, %1, %2;" : "=h"(d) : "f"(hi), "f"(lo));
    return d;
}

// Row-wide sum and maximum in one pass: warp shuffles, one shared-memory hop across the row's warps.
__device__ __forceinline__ void row_reduce_sum_max(float& sum, float& mx, int tx, int ty, int tpr)
{
    __shared__ float part_sum[kMaxRowsPerCta][32];
    __shared__ float part_max[kMaxRowsPerCta][32];
#pragma unroll
    for (int off = 16; off >= 1; off >>= 1) {
        sum += __shfl_xor_sync(0xffffffffu, sum, off);
        mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, off));
    }
    if (tpr > 32) {
        const int lane = tx & 31, warp_in_row = tx >> 5, n_warps = tpr >> 5;
        if (lane == 0) {
            part_sum[ty][warp_in_row] = sum;
            part_max[ty][warp_in_row] = mx;
        }
        row_sync(ty, tpr);
        sum = lane < n_warps ? part_sum[ty][lane] : 0.f;
        mx = lane < n_warps ? part_max[ty][lane] : 0.f;
#pragma unroll
        for (int off = 16; off >= 1; off >>= 1) {
            sum += __shfl_xor_sync(0xffffffffu, sum, off);
            mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, off));
        }
    }
}

template <typename T, int VB, int STAGE, int U, int CAP>
__global__ void add_rmsnorm_fp8_kernel(const Fp8Args a)
{
    static_assert(VB == 16 || VB == 32, "16- or 32-byte vectors of x and r; q leaves as 8 or 16 bytes");
    using C = Codec<T, VB>;
    constexpr int EPV = C::EPV;  // 8 or 16
    static_assert(sizeof(T) == 2, "the fp8-output variant takes 16-bit inputs");
    static_assert(STAGE != kStageReg || CAP % U == 0, "the unroll depth divides the per-thread vector count");
    extern __shared__ __align__(128) unsigned char dyn_smem[];

    const int tx = threadIdx.x, ty = threadIdx.y, tpr = blockDim.x;
    const long long row = (long long)blockIdx.x * blockDim.y + ty;
    const int n = row < a.n_tokens ? a.nvec : 0;
    const size_t safe_row = (size_t)(row < a.n_tokens ? row : 0);
    const size_t row_off = safe_row * (size_t)a.nvec * VB;
    const unsigned char* xrow = reinterpret_cast<const unsigned char*>(a.x) + row_off;
    const unsigned char* rrow = reinterpret_cast<const unsigned char*>(a.r) + row_off;
    const unsigned char* wrow = reinterpret_cast<const unsigned char*>(a.w);
    unsigned char* orow = reinterpret_cast<unsigned char*>(a.r_out) + row_off;
    unsigned char* qrow = reinterpret_cast<unsigned char*>(a.q) + row_off / 2;  // one byte per element
    wait_for_previous_kernel();

    float ss = 0.f, amax = 0.f;

    // y_j * inv_scale -> one byte per element: 8 or 16 bytes per vector
    auto quantise_store = [&](int v, const float (&s)[EPV], const float (&wf)[EPV], float rho, float inv_scale) {
        float t[EPV];
#pragma unroll
        for (int e = 0; e < EPV; ++e) t[e] = s[e] * rho * wf[e] * inv_scale;
        Vec<EPV> out;
#pragma unroll
        for (int k = 0; k < EPV / 4; ++k)
            out.w[k] = pack_e4m3x2(t[4 * k], t[4 * k + 1]) | (pack_e4m3x2(t[4 * k + 2], t[4 * k + 3]) << 16);
        st_stream<EPV, STAGE == kStageReg>(qrow + (size_t)v * EPV, out);
    };
    auto finish_row = [&](float& rho, float& inv_scale) {
        row_reduce_sum_max(ss, amax, tx, ty, tpr);
        rho = __frsqrt_rn(ss / (float)a.hidden + a.eps);
        const float amax_y = fmaxf(amax * rho, kScaleFloor);
        const float scale = amax_y / kE4m3Max;
        inv_scale = 1.0f / scale;
        if (tx == 0 && n > 0) a.scale[row] = scale;
    };

    if constexpr (STAGE == kStageReg) {
        float s[CAP][EPV];
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
                    float xf[EPV], rf[EPV], wf[EPV];
                    C::unpack(xv[u], xf);
                    C::unpack(rv[u], rf);
                    C::unpack(ld_weight<VB>(wrow + (size_t)v * VB), wf);
#pragma unroll
                    for (int e = 0; e < EPV; ++e) {
                        s[i0 + u][e] = xf[e] + rf[e];
                        ss = fmaf(s[i0 + u][e], s[i0 + u][e], ss);
                        amax = fmaxf(amax, fabsf(s[i0 + u][e] * wf[e]));
                    }
                    st_stream<VB, STAGE == kStageReg>(orow + (size_t)v * VB, C::pack(s[i0 + u]));
                }
            }
        }
        float rho, inv_scale;
        finish_row(rho, inv_scale);
#pragma unroll
        for (int i = 0; i < CAP; ++i) {
            const int v = tx + i * tpr;
            if (v < n) {
                float wf[EPV];
                C::unpack(ld_weight<VB>(wrow + (size_t)v * VB), wf);  // L1 hit: read in pass 1 already
                quantise_store(v, s[i], wf, rho, inv_scale);
            }
        }
    } else {
        __shared__ __align__(8) uint64_t bars[kMaxRowsPerCta];
        const size_t row_bytes = (size_t)a.nvec * VB;
        unsigned char* xs = dyn_smem + (size_t)ty * 2 * row_bytes;
        unsigned char* rs = xs + row_bytes;
        if (tx == 0) {
            mbarrier_init(&bars[ty], 1);
            if (n > 0) {
                mbarrier_expect_tx(&bars[ty], (uint32_t)(2 * row_bytes));
                tma_bulk_load(xs, xrow, (uint32_t)row_bytes, &bars[ty]);
                tma_bulk_load(rs, rrow, (uint32_t)row_bytes, &bars[ty]);
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
        for (int v0 = tx; v0 < n; v0 += U * tpr) {
#pragma unroll
            for (int u = 0; u < U; ++u) {
                const int v = v0 + u * tpr;
                if (v < n) {
                    float xf[EPV], rf[EPV], wf[EPV], s[EPV];
                    C::unpack(ld_shared<VB>(xs + (size_t)v * VB), xf);
                    C::unpack(ld_shared<VB>(rs + (size_t)v * VB), rf);
                    C::unpack(ld_weight<VB>(wrow + (size_t)v * VB), wf);
#pragma unroll
                    for (int e = 0; e < EPV; ++e) {
                        s[e] = xf[e] + rf[e];
                        ss = fmaf(s[e], s[e], ss);
                        amax = fmaxf(amax, fabsf(s[e] * wf[e]));
                    }
                    st_stream<VB, STAGE == kStageReg>(orow + (size_t)v * VB, C::pack(s));
                }
            }
        }
        float rho, inv_scale;
        finish_row(rho, inv_scale);
        for (int v0 = tx; v0 < n; v0 += U * tpr) {
#pragma unroll
            for (int u = 0; u < U; ++u) {
                const int v = v0 + u * tpr;
                if (v < n) {
                    float xf[EPV], rf[EPV], wf[EPV], s[EPV];
                    C::unpack(ld_shared<VB>(xs + (size_t)v * VB), xf);
                    C::unpack(ld_shared<VB>(rs + (size_t)v * VB), rf);
                    C::unpack(ld_weight<VB>(wrow + (size_t)v * VB), wf);
#pragma unroll
                    for (int e = 0; e < EPV; ++e) s[e] = xf[e] + rf[e];  // the same binary32 sum as pass 1
                    quantise_store(v, s, wf, rho, inv_scale);
                }
            }
        }
    }
}

}  // namespace rt
