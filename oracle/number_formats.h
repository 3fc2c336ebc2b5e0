/*
 * Number formats of the CPU oracle: exact decoding of bf16 / fp16 patterns and rounding of a double to
 * those formats (nearest, ties to even, gradual underflow, overflow to infinity), by integer arithmetic
 * on an exactly scaled value.  TEST INFRASTRUCTURE ONLY; included by the oracle's C files and by nothing
 * else.  Pinned by tests/test_oracle_codec.py (every 16-bit pattern, every tie, a library conversion,
 * exact-fraction bracket search).
 */
#ifndef ORACLE_NUMBER_FORMATS_H_
#define ORACLE_NUMBER_FORMATS_H_

#include <math.h>
#include <stdint.h>

enum { ORACLE_BF16 = 0, ORACLE_FP16 = 1, ORACLE_FP32 = 2 };

typedef struct {
    int ebits; /* exponent field width */
    int mbits; /* stored significand bits */
} fmt16;

static const fmt16 FMT_BF16 = {8, 7};
static const fmt16 FMT_FP16 = {5, 10};

/* Exact value of a 16-bit floating-point pattern, as a double. */
static double decode16(uint16_t bits, fmt16 f)
{
    const int emax_field = (1 << f.ebits) - 1;
    const int bias = (1 << (f.ebits - 1)) - 1;
    const int sign = bits >> 15;
    const int e = (bits >> f.mbits) & emax_field;
    const int m = bits & ((1 << f.mbits) - 1);
    double v;
    if (e == emax_field)
        v = m ? NAN : INFINITY;
    else if (e == 0)
        v = ldexp((double)m, 1 - bias - f.mbits); /* zero and subnormals */
    else
        v = ldexp((double)(m | (1 << f.mbits)), e - bias - f.mbits);
    return sign ? -v : v;
}

/*
 * Round a double to the nearest value of a 16-bit format, ties to even, with
 * gradual underflow and overflow to infinity.  One rounding, done on integers:
 * the value is scaled by an exact power of two so that one unit of the target
 * format's last place becomes 1, then rounded to an integer.
 */
static uint16_t encode16(double d, fmt16 f)
{
    const int emax_field = (1 << f.ebits) - 1;
    const int bias = (1 << (f.ebits - 1)) - 1;
    const uint32_t inf_bits = (uint32_t)emax_field << f.mbits;
    const uint16_t sign = signbit(d) ? 0x8000u : 0u;
    if (isnan(d))
        return (uint16_t)(sign | inf_bits | (1u << (f.mbits - 1)));
    double a = fabs(d);
    if (isinf(a))
        return (uint16_t)(sign | inf_bits);
    if (a == 0.0)
        return sign;

    int e2;
    (void)frexp(a, &e2);       /* a = m * 2^e2 with m in [0.5, 1) */
    const int E = e2 - 1;      /* a in [2^E, 2^(E+1)) */
    const int emin = 1 - bias; /* smallest normal exponent */
    const int q = (E < emin ? emin : E) - f.mbits; /* exponent of one ulp */
    const double scaled = ldexp(a, -q);            /* exact */
    const double lo = floor(scaled);
    const double rem = scaled - lo; /* exact, in [0, 1) */
    uint64_t n = (uint64_t)lo;
    if (rem > 0.5 || (rem == 0.5 && (n & 1u)))
        n += 1;

    uint32_t bits;
    if (E < emin)
        bits = (uint32_t)n; /* subnormal; n == 2^mbits is the smallest normal */
    else if (E + bias >= emax_field)
        bits = inf_bits;
    else
        bits = ((uint32_t)(E + bias) << f.mbits) + (uint32_t)(n - (1ull << f.mbits));
    if (bits > inf_bits)
        bits = inf_bits;
    return (uint16_t)(sign | bits);
}


#endif /* ORACLE_NUMBER_FORMATS_H_ */
