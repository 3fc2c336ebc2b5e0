/*
 * CPU oracle for fused residual-add + RMSNorm with a per-token fp8 (e4m3) quantised output: the norm
 * kernel's variant that feeds an fp8 GEMM ("fused output quantisation" is one of the execution-strategy
 * variants the paper's template axes - "organization of shared memory and registers", Section "Tuning
 * parameter selection and search space derivation" - leave room for; the paper prints no formula).
 *
 * TEST INFRASTRUCTURE ONLY; shares nothing with the CUDA path.
 *
 * Per token row t:
 *   s_j     = fl32(x_j) + fl32(r_j);   r'_j = RNE_dtype(s_j)            (as in add_rmsnorm_oracle.c)
 *   y_j     = s_j w_j / sqrt(mean_j s_j^2 + eps)                         (fp64, not rounded)
 *   amax    = max_j |y_j|;   scale_t = max(amax, 1e-12) / 448            (448 = largest finite e4m3 value)
 *   q_j     = RNE_e4m3(y_j / scale_t), saturating at +-448               (one byte per element)
 *   outputs: r' [T,H] (dtype), q [T,H] (bytes), scale [T] (binary32 = RNE of scale_t).
 *
 * e4m3 here is the 8-bit format with 4 exponent bits (bias 7), 3 significand bits, subnormals, no
 * infinities, and the single NaN magnitude pattern 0x7F; its finite range ends at 0x7E = 448.
 *
 * Pins (tests/test_oracle_fp8.py): all 256 patterns against a library decode; every midpoint between
 * adjacent values rounds to even; saturation; constant and one-hot rows (the largest element always maps
 * to +-448); q * scale reproduces the un-quantised oracle's y within half an e4m3 step.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>

#include "number_formats.h"

static double decode_e4m3(uint8_t b)
{
    const int sign = b >> 7, e = (b >> 3) & 0xF, m = b & 0x7;
    double v;
    if (e == 0xF && m == 0x7)
        v = NAN;
    else if (e == 0)
        v = ldexp((double)m, 1 - 7 - 3);
    else
        v = ldexp((double)(m | 0x8), e - 7 - 3);
    return sign ? -v : v;
}

/* Nearest e4m3 value, ties to even, saturating to +-448; NaN stays NaN. */
static uint8_t encode_e4m3(double d)
{
    const uint8_t sign = signbit(d) ? 0x80u : 0u;
    if (isnan(d)) return (uint8_t)(sign | 0x7Fu);
    double a = fabs(d);
    if (a == 0.0) return sign;
    if (a >= 448.0) return (uint8_t)(sign | 0x7Eu);
    int e2;
    (void)frexp(a, &e2);
    const int E = e2 - 1;
    const int emin = 1 - 7;
    const int q = (E < emin ? emin : E) - 3;
    const double scaled = ldexp(a, -q);
    const double lo = floor(scaled);
    const double rem = scaled - lo;
    uint64_t n = (uint64_t)lo;
    if (rem > 0.5 || (rem == 0.5 && (n & 1u))) n += 1;
    uint32_t bits = E < emin ? (uint32_t)n : ((uint32_t)(E + 7) << 3) + (uint32_t)(n - 8);
    /* a < 448 = 14 * 2^5 gives n <= 14 at the top exponent: the result cannot pass 0x7E */
    return (uint8_t)(sign | bits);
}

void oracle_decode_e4m3(const uint8_t* bits, double* out, int64_t n)
{
    for (int64_t i = 0; i < n; ++i) out[i] = decode_e4m3(bits[i]);
}

void oracle_encode_e4m3(const double* v, uint8_t* out, int64_t n)
{
    for (int64_t i = 0; i < n; ++i) out[i] = encode_e4m3(v[i]);
}

static float load32(const void* p, int64_t i, int dtype)
{
    if (dtype == ORACLE_FP32) return ((const float*)p)[i];
    return (float)decode16(((const uint16_t*)p)[i], dtype == ORACLE_BF16 ? FMT_BF16 : FMT_FP16);
}

/* x, r, r_out: [n_tokens, hidden] of `dtype`; w: [hidden]; q: [n_tokens, hidden] bytes; scale: [n_tokens].
 * Returns 0, 1 for a bad argument, 2 for an allocation failure. */
int oracle_add_rmsnorm_fp8(const void* x, const void* r, const void* w, uint8_t* q, float* scale, void* r_out,
                           int64_t n_tokens, int64_t hidden, float eps, int dtype)
{
    if (n_tokens < 0 || hidden <= 0 || dtype < 0 || dtype > 2) return 1;
    if (n_tokens == 0) return 0;
    if (!x || !r || !w || !q || !scale || !r_out) return 1;
    double* y = (double*)malloc((size_t)hidden * sizeof(double));
    if (!y) return 2;
    for (int64_t t = 0; t < n_tokens; ++t) {
        const int64_t base = t * hidden;
        double acc = 0.0;
        for (int64_t j = 0; j < hidden; ++j) {
            const float s32 = load32(x, base + j, dtype) + load32(r, base + j, dtype);
            if (dtype == ORACLE_FP32)
                ((float*)r_out)[base + j] = s32;
            else
                ((uint16_t*)r_out)[base + j] = encode16((double)s32, dtype == ORACLE_BF16 ? FMT_BF16 : FMT_FP16);
            y[j] = (double)s32;
            acc += (double)s32 * (double)s32;
        }
        const double denom = sqrt(acc / (double)hidden + (double)eps);
        double amax = 0.0;
        for (int64_t j = 0; j < hidden; ++j) {
            y[j] = y[j] * (double)load32(w, j, dtype) / denom;
            if (fabs(y[j]) > amax) amax = fabs(y[j]);
        }
        const double sc = (amax > 1e-12 ? amax : 1e-12) / 448.0;
        scale[t] = (float)sc;
        for (int64_t j = 0; j < hidden; ++j) q[base + j] = encode_e4m3(y[j] / sc);
    }
    free(y);
    return 0;
}

/* Distance between two arrays of e4m3 codes on the format's value lattice (+0 == -0, NaN matches NaN):
 * the largest distance in code steps and the number of elements beyond tol_steps. */
void oracle_e4m3_compare(const uint8_t* got, const uint8_t* ref, int64_t n, int32_t tol_steps, int32_t* max_steps,
                         int64_t* n_bad)
{
    int32_t worst = 0;
    int64_t bad = 0;
    for (int64_t i = 0; i < n; ++i) {
        const int gn = (got[i] & 0x7F) == 0x7F, rn = (ref[i] & 0x7F) == 0x7F;
        int32_t d;
        if (gn || rn) {
            d = (gn && rn) ? 0 : 255;
        } else {
            int32_t gi = got[i] & 0x7F, ri = ref[i] & 0x7F;
            if (got[i] & 0x80) gi = -gi;
            if (ref[i] & 0x80) ri = -ri;
            d = gi > ri ? gi - ri : ri - gi;
        }
        if (d > worst) worst = d;
        if (d > tol_steps) ++bad;
    }
    *max_steps = worst;
    *n_bad = bad;
}
