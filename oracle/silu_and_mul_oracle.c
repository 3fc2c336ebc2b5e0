/*
 * CPU oracle for the gated activation `silu_and_mul` (the second of the three serving kernels the
 * paper tunes, named in "Kernels", Experimental Setup; the paper prints no formula).
 *
 * TEST INFRASTRUCTURE ONLY; shares nothing with the CUDA path.
 *
 * Input x is [n_tokens, 2*d] row-major: the first d columns of a row are the gate g, the last d the
 * value u.  Output is [n_tokens, d]:
 *
 *     out[t, j] = RNE_dtype( silu(g) * u ),   silu(g) = g / (1 + exp(-g)),
 *     g = x[t, j],  u = x[t, d + j]
 *
 * evaluated in fp64 on the exactly decoded inputs, with ONE rounding to the output type at the end
 * (directly from fp64, gradual underflow, overflow to infinity).
 *
 * Pins (tests/test_oracle_silu.py): silu(0) = 0; silu(g) - silu(-g) = g; silu(ln 3) = 0.75 ln 3;
 * silu(g) = g for g >= 40 in fp64; which half of the row is the gate; zero gate or zero value gives
 * zero; an 80-digit decimal evaluation on tiny shapes; a float64 library evaluation
 * (torch.nn.functional.silu) at real sizes.
 */
#include <math.h>
#include <pthread.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

#include "number_formats.h"

typedef struct {
    const void* x;
    void* out;
    int64_t row_begin, row_end, d;
    int dtype;
} silu_job;

static double load_elem(const void* p, int64_t i, int dtype)
{
    if (dtype == ORACLE_FP32) return (double)((const float*)p)[i];
    return decode16(((const uint16_t*)p)[i], dtype == ORACLE_BF16 ? FMT_BF16 : FMT_FP16);
}

static void* silu_rows(void* arg)
{
    silu_job* job = (silu_job*)arg;
    const int64_t d = job->d;
    for (int64_t t = job->row_begin; t < job->row_end; ++t) {
        for (int64_t j = 0; j < d; ++j) {
            const double g = load_elem(job->x, t * 2 * d + j, job->dtype);
            const double u = load_elem(job->x, t * 2 * d + d + j, job->dtype);
            const double v = g / (1.0 + exp(-g)) * u;
            if (job->dtype == ORACLE_FP32)
                ((float*)job->out)[t * d + j] = (float)v;
            else
                ((uint16_t*)job->out)[t * d + j] = encode16(v, job->dtype == ORACLE_BF16 ? FMT_BF16 : FMT_FP16);
        }
    }
    return NULL;
}

/* x: [n_tokens, 2*d], out: [n_tokens, d], host memory of element type `dtype`.  Returns 0, or 1 for a
 * bad argument, 2 for an allocation failure. */
int oracle_silu_and_mul(const void* x, void* out, int64_t n_tokens, int64_t d, int dtype, int n_threads)
{
    if (n_tokens < 0 || d <= 0 || dtype < 0 || dtype > 2) return 1;
    if (n_tokens == 0) return 0;
    if (!x || !out) return 1;
    if (n_threads < 1) n_threads = 1;
    if ((int64_t)n_threads > n_tokens) n_threads = (int)n_tokens;
    silu_job* jobs = (silu_job*)malloc((size_t)n_threads * sizeof(silu_job));
    pthread_t* tids = (pthread_t*)malloc((size_t)n_threads * sizeof(pthread_t));
    if (!jobs || !tids) {
        free(jobs);
        free(tids);
        return 2;
    }
    for (int k = 0; k < n_threads; ++k) {
        jobs[k].x = x;
        jobs[k].out = out;
        jobs[k].d = d;
        jobs[k].dtype = dtype;
        jobs[k].row_begin = n_tokens * k / n_threads;
        jobs[k].row_end = n_tokens * (k + 1) / n_threads;
        if (n_threads == 1 || pthread_create(&tids[k], NULL, silu_rows, &jobs[k]) != 0) {
            silu_rows(&jobs[k]);
            tids[k] = 0;
        }
    }
    for (int k = 0; k < n_threads; ++k)
        if (tids[k]) pthread_join(tids[k], NULL);
    free(jobs);
    free(tids);
    return 0;
}
