/*
 * CPU oracle for `merge_attn_states` (the third of the serving kernels the paper tunes, named in
 * "Kernels", Experimental Setup, with shapes (n, h, d); the paper prints no formula).
 *
 * TEST INFRASTRUCTURE ONLY; shares nothing with the CUDA path.
 *
 * Two partial attention results over disjoint key sets, each a normalised output and the natural
 * logarithm of its softmax denominator, are merged into the result over the union of the key sets:
 *
 *   inputs   v_a, v_b : [n, h, d]  (dtype)        s_a, s_b : [n, h]  (binary32, log-sum-exp)
 *   m      = max(s_a, s_b)
 *   w_a    = exp(s_a - m),  w_b = exp(s_b - m),  D = w_a + w_b
 *   v_out  = RNE_dtype( (w_a v_a + w_b v_b) / D )         [n, h, d]
 *   s_out  = RNE_binary32( m + ln D )                      [n, h]
 *   if m = -inf (both parts empty): v_out = 0, s_out = -inf.
 *
 * Evaluated in fp64 on exactly decoded inputs, one rounding per output at the end.
 *
 * Pins (tests/test_oracle_merge.py): equal weights give the mean and s + ln 2; an empty part returns the
 * other part unchanged; s_a - s_b = ln 3 gives weights 3/4 and 1/4; a <-> b symmetry; a common shift
 * of s_a and s_b moves only s_out; and the defining property - attention over two key blocks,
 * merged, equals attention over their concatenation (float64 library softmax).
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>

#include "number_formats.h"

static double load_value(const void* p, int64_t i, int dtype)
{
    if (dtype == ORACLE_FP32) return (double)((const float*)p)[i];
    return decode16(((const uint16_t*)p)[i], dtype == ORACLE_BF16 ? FMT_BF16 : FMT_FP16);
}

static void store_value(void* p, int64_t i, int dtype, double v)
{
    if (dtype == ORACLE_FP32)
        ((float*)p)[i] = (float)v;
    else
        ((uint16_t*)p)[i] = encode16(v, dtype == ORACLE_BF16 ? FMT_BF16 : FMT_FP16);
}

/* All buffers are host memory.  Returns 0, or 1 for a bad argument. */
int oracle_merge_attn_states(const void* v_a, const float* s_a, const void* v_b, const float* s_b, void* v_out,
                             float* s_out, int64_t n_tokens, int64_t heads, int64_t head_dim, int dtype)
{
    if (n_tokens < 0 || heads <= 0 || head_dim <= 0 || dtype < 0 || dtype > 2) return 1;
    if (n_tokens == 0) return 0;
    if (!v_a || !s_a || !v_b || !s_b || !v_out || !s_out) return 1;
    for (int64_t t = 0; t < n_tokens; ++t) {
        for (int64_t k = 0; k < heads; ++k) {
            const int64_t row = t * heads + k;
            const double sa = (double)s_a[row], sb = (double)s_b[row];
            const double m = sa > sb ? sa : sb;
            if (isinf(m) && m < 0) {
                for (int64_t j = 0; j < head_dim; ++j) store_value(v_out, row * head_dim + j, dtype, 0.0);
                s_out[row] = -INFINITY;
                continue;
            }
            const double wa = exp(sa - m), wb = exp(sb - m), D = wa + wb;
            for (int64_t j = 0; j < head_dim; ++j) {
                const double a = load_value(v_a, row * head_dim + j, dtype);
                const double b = load_value(v_b, row * head_dim + j, dtype);
                store_value(v_out, row * head_dim + j, dtype, (wa * a + wb * b) / D);
            }
            s_out[row] = (float)(m + log(D));
        }
    }
    return 0;
}

/*
 * Mixed tolerance for outputs that may cancel: an element passes if it is within tol_ulp units in the
 * last place of the reference (16-bit types) or tol_rel * |ref| (binary32), OR within tol_abs
 * absolutely.  Writes the count of failing elements and the largest absolute difference.
 */
void oracle_mixed_compare(const void* got, const void* ref, int64_t n, int dtype, double tol_ulp_or_rel, double tol_abs,
                          double* max_abs, int64_t* n_bad)
{
    double worst = 0.0;
    int64_t bad = 0;
    for (int64_t i = 0; i < n; ++i) {
        const double g = load_value(got, i, dtype), q = load_value(ref, i, dtype);
        int ok;
        double diff;
        if (isnan(g) || isnan(q)) {
            ok = isnan(g) && isnan(q);
            diff = ok ? 0.0 : INFINITY;
        } else if (g == q) {
            ok = 1;
            diff = 0.0;
        } else {
            diff = fabs(g - q);
            if (dtype == ORACLE_FP32) {
                ok = !isinf(g) && !isinf(q) && (diff <= tol_ulp_or_rel * fabs(q) || diff <= tol_abs);
            } else {
                const uint16_t gb = ((const uint16_t*)got)[i], qb = ((const uint16_t*)ref)[i];
                int32_t gi = gb & 0x7FFF, qi = qb & 0x7FFF;
                if (gb & 0x8000u) gi = -gi;
                if (qb & 0x8000u) qi = -qi;
                const double ulps = fabs((double)gi - (double)qi);
                /* g != q here: an infinity on either side is no neighbour of any finite value */
                ok = !isinf(g) && !isinf(q) && (ulps <= tol_ulp_or_rel || diff <= tol_abs);
            }
        }
        if (!ok) ++bad;
        if (diff > worst) worst = diff;
    }
    *max_abs = worst;
    *n_bad = bad;
}
