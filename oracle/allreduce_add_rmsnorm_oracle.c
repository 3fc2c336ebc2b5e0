/*
 * CPU oracle for the tensor-parallel form of the fused residual-add + RMSNorm:
 * the input x arrives as N partial results (one per rank of a tensor-parallel
 * group, the outputs of a row-parallel matrix product) whose element-wise sum
 * is the x of the plain operator.
 *
 * TEST INFRASTRUCTURE ONLY.  Used by the tests, the smoke check and the
 * CPU-baseline leg of the benchmark; the CUDA library never links, imports or
 * calls it and shares no code with it.
 *
 * What is computed, per token row (rows are independent), for parts
 * x^(0) .. x^(N-1) given in rank order:
 *
 *   a_j   = fl32(x^(0)_j)
 *   a_j   = a_j + fl32(x^(k)_j)   for k = 1 .. N-1, each one IEEE binary32 addition (RNE), in this order
 *   s_j   = a_j + fl32(r_j)       one more binary32 addition: the residual joins last
 *   r'_j  = RNE_dtype(s_j)        bit-exact contract
 *   ms    = (1/H) * sum_j s_j^2   fp64, plain left-to-right
 *   y_j   = RNE_dtype( s_j * w_j / sqrt(ms + eps) )     fp64, one final rounding
 *
 * The paper names the operator only ("Kernels" paragraph: `fused_add_rmsnorm`)
 * and runs on one GPU; this form is the same operator with the all-reduce that
 * precedes it in tensor-parallel serving folded into its load.  Readings taken:
 *   - the sum over ranks is carried in binary32 (one rounding per addition, none
 *     to the storage type in between), strictly in rank order 0, 1, .., N-1, so
 *     that every rank that evaluates a row obtains the same bits;
 *   - the residual is added after the last part;
 *   - with N = 1 the operator is exactly the plain fused add + RMSNorm.
 *
 * Pins (tests/test_oracle_allreduce.py): N = 1 against the plain operator's
 * oracle; exact rational arithmetic with a hand-written round-to-binary32 on
 * tiny shapes; a float32 library evaluation of the same chain; closed forms
 * where binary32 rounding makes the order visible (2^24 + 1 - 2^24); planted
 * mistakes (reversed order, fp64 accumulation, a dropped part, the residual
 * first) each caught by one of them.  No function here is "parity unpinned".
 */
#include <math.h>
#include <pthread.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

#include "number_formats.h"

typedef struct {
    const void* x_parts; /* [n_parts][n_tokens, hidden] */
    const void *r, *w;
    void *y, *r_out;
    int64_t n_tokens, row_begin, row_end, hidden;
    int n_parts, dtype;
    double eps;
    int status;
} ar_job;

static float load32(const void* base, int64_t index, int dtype)
{
    if (dtype == ORACLE_FP32) return ((const float*)base)[index];
    const fmt16 f = dtype == ORACLE_BF16 ? FMT_BF16 : FMT_FP16;
    return (float)decode16(((const uint16_t*)base)[index], f); /* exact: every 16-bit value is a binary32 value */
}

static void ar_rows(ar_job* job)
{
    const int64_t H = job->hidden;
    const int64_t part_stride = job->n_tokens * H;
    double* s = (double*)malloc((size_t)H * sizeof(double));
    if (!s) {
        job->status = 2;
        return;
    }
    for (int64_t t = job->row_begin; t < job->row_end; ++t) {
        const int64_t base = t * H;
        double acc = 0.0;
        for (int64_t j = 0; j < H; ++j) {
            float a = load32(job->x_parts, base + j, job->dtype);
            for (int k = 1; k < job->n_parts; ++k) {
                const float part = load32(job->x_parts, (int64_t)k * part_stride + base + j, job->dtype);
                a = a + part; /* binary32, RNE, rank order */
            }
            const float s32 = a + load32(job->r, base + j, job->dtype);
            if (job->dtype == ORACLE_FP32) {
                ((float*)job->r_out)[base + j] = s32;
            } else {
                const fmt16 f = job->dtype == ORACLE_BF16 ? FMT_BF16 : FMT_FP16;
                ((uint16_t*)job->r_out)[base + j] = encode16((double)s32, f);
            }
            s[j] = (double)s32;
            acc += s[j] * s[j];
        }
        const double denom = sqrt(acc / (double)H + job->eps);
        for (int64_t j = 0; j < H; ++j) {
            const double y64 = s[j] * (double)load32(job->w, j, job->dtype) / denom;
            if (job->dtype == ORACLE_FP32) {
                ((float*)job->y)[base + j] = (float)y64;
            } else {
                const fmt16 f = job->dtype == ORACLE_BF16 ? FMT_BF16 : FMT_FP16;
                ((uint16_t*)job->y)[base + j] = encode16(y64, f);
            }
        }
    }
    free(s);
    job->status = 0;
}

static void* ar_thread(void* arg)
{
    ar_rows((ar_job*)arg);
    return NULL;
}

/*
 * x_parts: [n_parts, n_tokens, hidden] contiguous (part k at offset k * n_tokens * hidden);
 * r, y, r_out: [n_tokens, hidden]; w: [hidden]; all host memory of element type `dtype`.
 * Rows are split over n_threads threads.  Returns 0, 1 for a bad argument, 2 for an allocation failure.
 */
int oracle_allreduce_add_rmsnorm(const void* x_parts, int n_parts, const void* r, const void* w, void* y, void* r_out,
                                 int64_t n_tokens, int64_t hidden, float eps, int dtype, int n_threads)
{
    if (n_tokens < 0 || hidden <= 0 || dtype < 0 || dtype > 2 || n_parts < 1) return 1;
    if (n_tokens == 0) return 0;
    if (!x_parts || !r || !w || !y || !r_out) return 1;
    if (n_threads < 1) n_threads = 1;
    if ((int64_t)n_threads > n_tokens) n_threads = (int)n_tokens;

    ar_job proto;
    memset(&proto, 0, sizeof(proto));
    proto.x_parts = x_parts; proto.n_parts = n_parts;
    proto.r = r; proto.w = w; proto.y = y; proto.r_out = r_out;
    proto.n_tokens = n_tokens; proto.hidden = hidden;
    proto.eps = (double)eps;
    proto.dtype = dtype;
    if (n_threads == 1) {
        proto.row_begin = 0;
        proto.row_end = n_tokens;
        ar_rows(&proto);
        return proto.status;
    }
    ar_job* jobs = (ar_job*)malloc((size_t)n_threads * sizeof(ar_job));
    pthread_t* tids = (pthread_t*)malloc((size_t)n_threads * sizeof(pthread_t));
    if (!jobs || !tids) {
        free(jobs);
        free(tids);
        return 2;
    }
    int status = 0;
    for (int k = 0; k < n_threads; ++k) {
        jobs[k] = proto;
        jobs[k].row_begin = n_tokens * k / n_threads;
        jobs[k].row_end = n_tokens * (k + 1) / n_threads;
        if (pthread_create(&tids[k], NULL, ar_thread, &jobs[k]) != 0) {
            ar_rows(&jobs[k]);
            tids[k] = 0;
        }
    }
    for (int k = 0; k < n_threads; ++k) {
        if (tids[k]) pthread_join(tids[k], NULL);
        if (jobs[k].status) status = jobs[k].status;
    }
    free(jobs);
    free(tids);
    return status;
}
